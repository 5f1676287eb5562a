"""GPU parity of the fp32 CUDA-core engine against the fp64 oracle (through the C ABI).

Tolerances: 1e-5 relative Frobenius error for fp32 gradients, 2e-3 for bf16 gradients (the task's bar);
bases are compared as projectors."""
import numpy as np
import pytest

from parity_util import Case, GpuRun, OracleRun, compare_basis, compare_step, make_inputs

pytestmark = pytest.mark.gpu
TOL32 = 1e-5
SIMT = 1


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def test_sketch_is_bit_exact(torch):
    from oracle import spectral_oracle as so
    case = Case(shapes=[(64, 64)], rank=8, dtype="fp32", seed=12345, engine=SIMT)
    from parity_util import make_plan
    plan = make_plan(case, torch)
    got = plan.export_sketch(777, 40).cpu().numpy()
    assert np.array_equal(got, so.rademacher_sketch(12345, 0, 777, 40))


def test_c1_single_256_fp32_mirror_and_exact(torch):
    """Config 1: one 256x256 fp32 matrix, T=512, keep 0.25, r=8, one cold step."""
    case = Case(shapes=[(256, 256)], rank=8, dtype="fp32", tokens=512, keep=0.25, seed=0, warmed=False, q=2, engine=SIMT)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.dev_status == 0 and g.step_status == 0 and not g.uses_tc
    o = OracleRun(case, inp, "mirror")
    eb = compare_basis(g, o)
    assert eb["M"] < 1e-6 and eb["PU"] < TOL32 and eb["PV"] < TOL32 and eb["s"] < TOL32 and eb["orth"] < 1e-5, eb
    es = compare_step(g, o, mask_small_g=True)
    assert es["gproj"] < TOL32 and es["m"] < TOL32 and es["v"] < TOL32 and es["dW"] < TOL32, es
    # rule parity on the oracle's exact basis (imported)
    oe = OracleRun(case, inp, "exact")
    g2 = GpuRun(case, inp, torch, import_bases=[(s.U, s.s, s.V) for s in oe.states])
    es = compare_step(g2, oe, mask_small_g=True)
    assert es["gproj"] < TOL32 and es["m"] < TOL32 and es["v"] < TOL32 and es["dW"] < TOL32, es


def test_c1_exact_parity_with_wide_sketch(torch):
    """With l=128, q=8 the iteration reaches the exact truncated SVD on the tiny config."""
    case = Case(shapes=[(256, 256)], rank=8, dtype="fp32", tokens=512, keep=0.25, seed=0, l=128, q=8, engine=SIMT,
                tau_p=50.0)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    oe = OracleRun(case, inp, "exact")
    es = compare_step(g, oe)
    assert es["gproj"] < TOL32 and es["m"] < TOL32 and es["v"] < TOL32 and es["dW"] < TOL32, es


@pytest.mark.parametrize("dtype,tol", [("fp32", TOL32), ("bf16", 2e-3)])
def test_ragged_shapes_warmed_state(torch, dtype, tol):
    shapes = [(200, 136), (72, 520), (200, 136), (130, 66)]
    case = Case(shapes=shapes, rank=5, dtype=dtype, tokens=192, keep=0.5, planted=3, seed=3, q=1, tau_p=40.0,
                n_anchor=2, engine=SIMT)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.dev_status == 0
    o = OracleRun(case, inp, "mirror")
    eb = compare_basis(g, o)
    assert eb["M"] < 1e-6 and max(eb["PU"], eb["PV"], eb["s"]) < tol, eb
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < tol, es
    assert es["Wb"] < 5e-3       # bf16 copy of the weights: one bf16 rounding


def test_rank_zero_is_plain_adamw(torch):
    case = Case(shapes=[(96, 80)], rank=0, dtype="fp32", alpha=1.0, engine=SIMT)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    o = OracleRun(case, inp, "exact")
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL32, es
    assert np.array_equal(g.gproj[0], inp["G"][0].astype(np.float64))


def test_no_anchor_yet_gives_alpha_g_and_a_warning(torch):
    case = Case(shapes=[(64, 48)], rank=4, dtype="fp32", n_anchor=0, engine=SIMT)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.step_status == 1                                     # SC_WARN_NO_ANCHOR
    assert np.allclose(g.gproj[0], 0.3 * inp["G"][0].astype(np.float64), rtol=1e-6, atol=0)


def test_clipping_rescale_and_stats(torch):
    from oracle import spectral_oracle as so
    case = Case(shapes=[(128, 96), (64, 160)], rank=6, dtype="fp32", keep=0.25, prescaled=False, max_grad_norm=0.2,
                tau_p=30.0, engine=SIMT)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    o = OracleRun(case, inp, "mirror")
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL32, es
    total = sum(np.sum(x * x) for x in g.gproj)
    assert abs(np.sqrt(total) - 0.2) < 1e-5
    for i, st in enumerate(o.states):
        gs = 1.0 / case.keep * o.G[i]
        X = so.project(st.U, gs, st.V)
        assert abs(g.stats[i]["g_sqnorm"] / np.sum(gs * gs) - 1) < 1e-4
        assert abs(g.stats[i]["x_sqnorm"] / np.sum(X * X) - 1) < 1e-4
        assert abs(g.stats[i]["r_eff"] / so.effective_rank(so.filter_weights(st.s, case.tau_p)) - 1) < 1e-4


def test_partial_anchor_arrival_and_stale_tag(torch):
    import paper_2609_14339_b200 as sc
    from parity_util import make_plan, to_dev
    case = Case(shapes=[(64, 64), (64, 64)], rank=4, dtype="fp32", engine=SIMT)
    inp = make_inputs(case)
    plan = make_plan(case, torch)
    a0 = to_dev(inp["anchors"][0][0], "fp32", torch, "cuda:0")
    plan.anchor_update([a0, None], 5)
    torch.cuda.synchronize()
    assert plan.get_anchor_info() == (5, 1)
    assert float(plan.export_anchor_momentum(1).abs().max()) == 0.0
    assert float(plan.export_anchor_momentum(0).abs().max()) > 0.0
    with pytest.raises(sc.SCError) as e:
        plan.anchor_update([a0, None], 4)
    assert e.value.status == -6
