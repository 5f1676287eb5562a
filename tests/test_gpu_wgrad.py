"""sc_masked_weight_grad (mask pass + tensor-core GEMM over the tokens) against the oracle's masked_weight_gradient.
bf16 inputs multiply exactly, the sum is fp32 in the tensor core's accumulator: the fp32 output matches the fp64
oracle to accumulation error; the bf16 output adds one rounding (2^-9 per element)."""
import numpy as np
import pytest

from oracle import spectral_oracle as so
from parity_util import rel
from synth import generator as gen

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5      # task tolerance for fp32 results
TOL_BF16 = 2e-3     # task tolerance for bf16 results


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _inputs(torch, tokens, rows, cols, seed):
    spec = gen.GradSpec(m=rows, n=cols, tokens=tokens, keep=0.25, planted_rank=4, seed=seed)
    X, dY = gen.batch(spec, 1)
    Xb = torch.from_numpy(X.astype(np.float32)).cuda().to(torch.bfloat16)
    dYb = torch.from_numpy(dY.astype(np.float32)).cuda().to(torch.bfloat16)
    return Xb, dYb


# several 128 x 256 tiles with ragged edges in all three dimensions; one tile; K shorter than one stage; keep = 1
@pytest.mark.parametrize("tokens,rows,cols,keep", [(300, 264, 520, 0.1), (1024, 512, 1024, 0.25), (40, 8, 8, 0.5),
                                                   (257, 136, 256, 1.0), (4096, 128, 256, 0.05)])
def test_matches_the_oracle(torch, tokens, rows, cols, keep):
    import paper_2609_14339_b200 as sc
    Xb, dYb = _inputs(torch, tokens, rows, cols, seed=3)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    G32, Xm = sc.masked_weight_grad(dYb, Xb, keep, seed=21, layer=2, step=77, out_dtype=torch.float32, status=status)
    G16, _ = sc.masked_weight_grad(dYb, Xb, keep, seed=21, layer=2, step=77, out_dtype=torch.bfloat16, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    M = so.prf_keep_mask(21, 2, 77, tokens, cols, keep)
    Xd, dYd = Xb.double().cpu().numpy(), dYb.double().cpu().numpy()
    assert np.array_equal(Xm.double().cpu().numpy(), Xd * M)                      # the mask pass, bit-exact
    want = so.masked_weight_gradient(dYd, Xd, M, keep)
    assert rel(G32.double().cpu().numpy(), want) < TOL_F32
    assert rel(G16.double().cpu().numpy(), want) < TOL_BF16
    # element-wise on the fp32 result as well: no tile, row or column is out of place
    err = np.abs(G32.double().cpu().numpy() - want)
    assert err.max() <= 1e-4 * np.abs(want).max()


def test_full_size_ffn_layer_sampled(torch):
    """One 14336 x 4096 layer, 4096 tokens, as bench.py --wgrad times it: sampled rows and columns against the oracle."""
    import paper_2609_14339_b200 as sc
    tokens, rows, cols, keep = 4096, 14336, 4096, 0.1
    g = torch.Generator(device="cuda"); g.manual_seed(11)
    Xb = torch.randn((tokens, cols), generator=g, device="cuda").to(torch.bfloat16)
    dYb = torch.randn((tokens, rows), generator=g, device="cuda").to(torch.bfloat16)
    G, Xm = sc.masked_weight_grad(dYb, Xb, keep, seed=5, layer=9, step=1000, out_dtype=torch.float32)
    torch.cuda.synchronize()
    rs = np.array([0, 1, 127, 128, 5000, 14335])
    cs = np.array([0, 255, 256, 2049, 4095])
    M = so.prf_keep_mask(5, 9, 1000, tokens, cols, keep)[:, cs]
    Xs = Xb[:, cs].double().cpu().numpy()
    assert np.array_equal(Xm[:, cs].double().cpu().numpy(), Xs * M)
    want = so.masked_weight_gradient(dYb[:, rs].double().cpu().numpy(), Xs, M, keep)
    got = G[rs][:, cs].double().cpu().numpy()
    assert rel(got, want) < TOL_F32


def test_rejects_bad_arguments(torch):
    import paper_2609_14339_b200 as sc
    lib = sc.load_library()
    x = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    assert lib.sc_masked_weight_grad(p, p, p, p, 0, 16, 12, 8, 0.5, 0, 0, 0, None, None) == -2      # rows % 8 != 0
    assert lib.sc_masked_weight_grad(p, p, p, p, 7, 16, 8, 8, 0.5, 0, 0, 0, None, None) == -3       # dtype
    assert lib.sc_masked_weight_grad(p, p, p, p + 2, 0, 16, 8, 8, 0.5, 0, 0, 0, None, None) == -4   # alignment
    assert lib.sc_masked_weight_grad(p, p, p, p, 0, 16, 8, 8, 1.5, 0, 0, 0, None, None) == -1       # keep
    assert lib.sc_masked_weight_grad(None, p, p, p, 0, 16, 8, 8, 0.5, 0, 0, 0, None, None) == -1
