"""The shared-PRF activation mask on the GPU against the oracle: the mask is bit-exact, the masked gradient formed
from it matches the oracle's."""
import numpy as np
import pytest

from oracle import spectral_oracle as so
from parity_util import rel
from synth import generator as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


@pytest.mark.parametrize("tokens,features,keep", [(300, 264, 0.1), (1024, 4096, 0.05), (65, 8, 0.5), (16, 64, 1.0)])
def test_mask_is_bit_exact_and_values_pass_through(torch, tokens, features, keep):
    import paper_2609_14339_b200 as sc
    rng = np.random.default_rng(1)
    X = (rng.standard_normal((tokens, features)) + 3.0).astype(np.float32)       # no zeros: the mask is readable
    Xb = torch.from_numpy(X).cuda().to(torch.bfloat16)
    out = sc.apply_prf_mask(Xb, keep, seed=77, layer=3, step=12345, rescale=False)
    M = so.prf_keep_mask(77, 3, 12345, tokens, features, keep)
    got = out.float().cpu().numpy()
    assert np.array_equal(got != 0, M != 0)                                       # bit-exact mask
    assert np.array_equal(got, Xb.float().cpu().numpy() * M)                      # kept values untouched
    # rescaled form: one bf16 rounding of x * 65536 / threshold
    out2 = sc.apply_prf_mask(Xb, keep, seed=77, layer=3, step=12345, rescale=True)
    want = Xb.double().cpu().numpy() * M * (65536.0 / so.keep_threshold(keep))
    assert rel(out2.double().cpu().numpy(), want) < 3e-3
    # another step gives another mask; in-place works
    other = sc.apply_prf_mask(Xb, keep, seed=77, layer=3, step=12346, rescale=False)
    assert keep == 1.0 or not torch.equal(other, out)
    inplace = Xb.clone()
    sc.apply_prf_mask(inplace, keep, seed=77, layer=3, step=12345, rescale=False, out=inplace)
    assert torch.equal(inplace, out)


def test_masked_weight_gradient_from_the_gpu_mask(torch):
    import paper_2609_14339_b200 as sc
    spec = gen.GradSpec(m=96, n=128, tokens=256, keep=0.25, planted_rank=4, seed=5)
    X, dY = gen.batch(spec, 1)
    Xb = torch.from_numpy(X.astype(np.float32)).cuda().to(torch.bfloat16)
    dYb = torch.from_numpy(dY.astype(np.float32)).cuda().to(torch.bfloat16)
    Xm = sc.apply_prf_mask(Xb, 0.25, seed=9, layer=1, step=4, rescale=False)
    G = (dYb.double().T @ Xm.double()).cpu().numpy() * (65536.0 / so.keep_threshold(0.25))
    want = so.masked_weight_gradient(dYb.double().cpu().numpy(), Xb.double().cpu().numpy(),
                                     so.prf_keep_mask(9, 1, 4, 256, 128, 0.25), 0.25)
    assert rel(G, want) < 1e-12


def test_rejects_bad_arguments(torch):
    import paper_2609_14339_b200 as sc
    lib = sc.load_library()
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    assert lib.sc_apply_prf_mask(p, p, 4, 12, 0.5, 0, 0, 0, 0, None) == -2        # features % 8 != 0
    assert lib.sc_apply_prf_mask(p, p, 4, 16, 0.0, 0, 0, 0, 0, None) == -1
    assert lib.sc_apply_prf_mask(None, p, 4, 16, 0.5, 0, 0, 0, 0, None) == -1
    assert lib.sc_apply_prf_mask(p + 2, p, 4, 16, 0.5, 0, 0, 0, 0, None) == -4


# the last four cases sit on rounding ties of K = round(keep * features): halves round up, product in single precision
@pytest.mark.parametrize("tokens,features,keep", [(200, 264, 0.1), (64, 4096, 0.05), (33, 37, 0.5), (8, 16, 1.0),
                                                  (9, 8, 0.3125), (9, 10, 0.25), (9, 5, 0.7), (9, 6, 0.75)])
def test_exact_k_mask_is_bit_exact(torch, tokens, features, keep):
    import paper_2609_14339_b200 as sc
    rng = np.random.default_rng(2)
    X = (rng.standard_normal((tokens, features)) + 3.0).astype(np.float32)
    Xb = torch.from_numpy(X).cuda().to(torch.bfloat16)
    out = sc.apply_prf_mask(Xb, keep, seed=31, layer=2, step=7, rescale=False, exact_k=True)
    M = so.prf_exact_k_mask(31, 2, 7, tokens, features, keep)
    got = out.float().cpu().numpy()
    assert np.array_equal(got != 0, M != 0)
    assert np.all((got != 0).sum(axis=1) == so.exact_k(features, keep))
    assert np.array_equal(got, Xb.float().cpu().numpy() * M)
    out2 = sc.apply_prf_mask(Xb, keep, seed=31, layer=2, step=7, rescale=True, exact_k=True)
    want = Xb.double().cpu().numpy() * M * (features / so.exact_k(features, keep))
    assert rel(out2.double().cpu().numpy(), want) < 3e-3
