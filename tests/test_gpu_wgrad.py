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


def test_from_activations_to_the_corrected_step(torch):
    """Algorithm 1 lines 4-14 on the GPU from the activations on: masked weight gradients from sc_masked_weight_grad
    (anchor gradients from the same call with keep = 1 on an independent batch), then the anchor update and the
    corrected AdamW step; the oracle forms its own gradients in fp64 from the same X, dY and the oracle's mask."""
    import paper_2609_14339_b200 as sc
    from parity_util import Case, GpuRun, OracleRun, compare_step, make_inputs
    shapes = [(512, 256), (256, 512), (384, 384)]
    case = Case(shapes=shapes, rank=16, tokens=384, keep=0.25, planted=8, seed=7, tau_p=50.0, prescaled=True)
    inp_o = make_inputs(case)                     # optimizer state and specs; gradients are replaced below
    inp_g = dict(inp_o, anchors=[None] * len(shapes), G=[None] * len(shapes))
    inp_o = dict(inp_o, anchors=[None] * len(shapes), G=[None] * len(shapes))
    bits = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    for i, spec in enumerate(inp_o["specs"]):
        Xa, dYa = gen.batch(spec, 0)              # the anchor circuit's unmasked batch
        X, dY = gen.batch(spec, 2)                # the fast circuit's batch
        dev = lambda a: torch.from_numpy(a.astype(np.float32)).cuda().to(torch.bfloat16)
        Xab, dYab, Xb, dYb = dev(Xa), dev(dYa), dev(X), dev(dY)
        Ganc, _ = sc.masked_weight_grad(dYab, Xab, 1.0, seed=3, layer=i, step=0)
        G, _ = sc.masked_weight_grad(dYb, Xb, case.keep, seed=3, layer=i, step=2)
        torch.cuda.synchronize()
        inp_g["anchors"][i] = [bits(Ganc)]
        inp_g["G"][i] = bits(G)
        f64 = lambda t: t.double().cpu().numpy()
        M = so.prf_keep_mask(3, i, 2, case.tokens, spec.n, case.keep)
        inp_o["anchors"][i] = [gen.round_to(f64(dYab).T @ f64(Xab), "bf16")]
        inp_o["G"][i] = gen.round_to(so.masked_weight_gradient(f64(dYb), f64(Xb), M, case.keep), "bf16")
        # the two sides' stored gradients differ only where the fp32 sum lands on the other side of a bf16 rounding point
        assert rel(gen.stored_to_f64(inp_g["G"][i], "bf16"), gen.stored_to_f64(inp_o["G"][i], "bf16")) < 5e-4
    g = GpuRun(case, inp_g, torch)
    assert g.uses_tc and g.dev_status == 0
    o = OracleRun(case, inp_o, "mirror")
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL_BF16, es
