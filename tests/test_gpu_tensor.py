"""GPU parity of the tensor-core (tcgen05) engine for bf16 gradients against the fp64 oracle.

Tolerance: 2e-3 relative Frobenius error (the bar for bf16 operands); bases compared as projectors."""
import numpy as np
import pytest

from oracle import spectral_oracle as so
from parity_util import Case, GpuRun, OracleRun, compare_basis, compare_step, make_inputs, rel
from synth import generator as gen

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _check(case, torch, tol=TOL):
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.uses_tc, "expected the tcgen05 engine"
    assert g.dev_status == 0 and g.status_after_anchor == 0
    o = OracleRun(case, inp, "mirror")
    # the two contractions on their own, against the oracle with the GPU's own basis
    for i in range(len(case.shapes)):
        U, s, V = g.basis[i]
        T, X = g.plan.export_projection(i)
        assert rel(T.double().cpu().numpy(), o.G[i] @ V) < 1e-4, "T = G V"
        # X = U^T T runs on tf32 tensor cores: per-element rounding 2^-11, averaged over the m rows; ~1.5e-4 at m = 512
        assert rel(X.double().cpu().numpy(), U.T @ o.G[i] @ V) < 5e-4, "X = U^T G V"
    eb = compare_basis(g, o)
    assert eb["M"] < 1e-6 and max(eb["PU"], eb["PV"], eb["s"]) < tol and eb["orth"] < 1e-4, eb
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < tol, es
    # rule parity on the oracle's exact basis
    oe = OracleRun(case, inp, "exact")
    g2 = GpuRun(case, inp, torch, import_bases=[(st.U, st.s, st.V) for st in oe.states])
    es2 = compare_step(g2, oe)
    assert max(es2["gproj"], es2["m"], es2["v"], es2["dW"]) < tol, es2
    return g, o, es, es2


def test_small_two_shapes(torch):
    case = Case(shapes=[(256, 384), (384, 256)], rank=16, tokens=256, keep=0.25, planted=8, seed=1, tau_p=50.0)
    _check(case, torch)


def test_rank64_several_tiles(torch):
    case = Case(shapes=[(512, 1024), (512, 1024), (1024, 512)], rank=64, tokens=512, keep=0.1, planted=32, seed=2,
                tau_p=100.0)
    _check(case, torch)


def test_ragged_tail_shapes(torch):
    # rows and columns that are not multiples of the 128 x 128 tile, rank not a multiple of 16
    case = Case(shapes=[(200, 136), (72, 520), (330, 264)], rank=5, tokens=192, keep=0.5, planted=3, seed=3, tau_p=40.0,
                n_anchor=2)
    _check(case, torch)


def test_rank_above_one_k_chunk(torch):
    case = Case(shapes=[(384, 640)], rank=96, tokens=512, keep=0.25, planted=48, seed=4, tau_p=80.0)
    _check(case, torch)


def test_split_k_single_matrix(torch):
    # one matrix with few row tiles and a long K: the projection splits K over several blocks
    case = Case(shapes=[(256, 4096)], rank=32, tokens=256, keep=0.25, planted=16, seed=5, tau_p=80.0)
    _check(case, torch)


def test_engines_agree(torch):
    case = Case(shapes=[(256, 384)], rank=16, tokens=256, keep=0.25, planted=8, seed=6, tau_p=50.0)
    inp = make_inputs(case)
    a = GpuRun(case, inp, torch)
    case2 = Case(**{**case.__dict__, "engine": 1})
    b = GpuRun(case2, inp, torch)
    assert a.uses_tc and not b.uses_tc
    assert rel(a.gproj[0], b.gproj[0]) < 1e-4 and rel(a.m[0], b.m[0]) < 1e-4 and rel(a.W[0], b.W[0]) < 1e-5


def test_host_gradient_entry_point_matches_device_path(torch):
    """sc_correct_and_step_host copies pinned host gradients class by class and must give the device path's bits."""
    from parity_util import make_plan, to_dev
    case = Case(shapes=[(256, 384), (384, 256), (256, 384)], rank=16, tokens=256, keep=0.25, planted=8, seed=7, tau_p=50.0)
    inp = make_inputs(case)
    outs = []
    for host in (False, True):
        plan = make_plan(case, torch)
        n = len(case.shapes)
        plan.anchor_update([to_dev(inp["anchors"][i][0], "bf16", torch, "cuda:0") for i in range(n)], 0)
        G = [to_dev(inp["G"][i], "bf16", torch, "cuda:0") for i in range(n)]
        W = [torch.from_numpy(inp["W"][i].copy()).cuda() for i in range(n)]
        m = [torch.from_numpy(inp["m"][i].copy()).cuda() for i in range(n)]
        v = [torch.from_numpy(inp["v"][i].copy()).cuda() for i in range(n)]
        if host:
            Gh = [g.cpu().pin_memory() for g in G]
            stage = [torch.zeros_like(g) for g in G]
            rc, stats, clip = plan.correct_and_step_host(Gh, stage, W, m, v, 100)
            assert rc == 0 and len(stats) == n and stats[0]["g_sqnorm"] > 0 and clip == 1.0
            assert all(torch.equal(a, b) for a, b in zip(stage, G))
        else:
            assert plan.correct_and_step(G, W, m, v, 100) == 0
        torch.cuda.synchronize()
        outs.append((W, m, v))
    for a, b in zip(outs[0], outs[1]):
        assert all(torch.equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("engine", [0, 1])
def test_warm_started_range_finder(torch, engine):
    """From the second anchor arrival on the range finder starts from the previous right basis (two sweeps per
    arrival); the oracle's MIRROR mode does the same."""
    case = Case(shapes=[(384, 512), (256, 384), (384, 512)], rank=16, l=24, tokens=256, keep=0.25, planted=8, seed=8,
                tau_p=60.0, n_anchor=3, warm=True, q_warm=0, engine=engine)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.dev_status == 0
    o = OracleRun(case, inp, "mirror")
    eb = compare_basis(g, o)
    assert eb["M"] < 1e-6 and max(eb["PU"], eb["PV"], eb["s"]) < TOL, eb
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL, es
    # and it is a better basis than a cold start with the same two sweeps: closer to the exact truncated SVD
    cold = Case(**{**case.__dict__, "warm": False, "q": 0})
    oc = OracleRun(cold, inp, "mirror")
    oe = OracleRun(case, inp, "exact")
    d_warm = so.projector_distance(o.states[0].V, oe.states[0].V)
    d_cold = so.projector_distance(oc.states[0].V, oe.states[0].V)
    assert d_warm < d_cold


@pytest.mark.parametrize("shape,k", [((1024, 1024), 16), ((512, 2048), 32)])
def test_exact_parity_where_the_rank_cut_is_well_posed(torch, shape, k):
    """Gate G3: with r equal to the planted rank there is a wide spectral gap at the cut, the truncated SVD is
    well conditioned, and the GPU path (l = 2r, q = 4) must match the oracle's EXACT mode."""
    case = Case(shapes=[shape], rank=k, tokens=1024, keep=0.1, planted=k, snr=4.0, seed=12, tau_p=1e-3, q=4, l=2 * k)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    oe = OracleRun(case, inp, "exact")
    s_all = np.linalg.svd(oe.states[0].M_anc, compute_uv=False)
    assert (s_all[k - 1] - s_all[k]) / s_all[k - 1] > 0.3            # the gap is really there
    eb, es = compare_basis(g, oe), compare_step(g, oe)
    assert max(eb["PU"], eb["PV"], eb["s"]) < TOL, eb
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL, es


@pytest.mark.parametrize("engine", [0, 1])
def test_factored_anchor_gradient(torch, engine):
    """Anchor gradients arriving as rank-rho factors P Q^T: Eq. 1 without densifying, then the usual basis."""
    from parity_util import make_plan
    rng = np.random.default_rng(21)
    case = Case(shapes=[(384, 256), (200, 136)], rank=8, tokens=128, tau_p=5.0, engine=engine)
    plan = make_plan(case, torch)
    hp = so.Hyper(beta_anc=float(np.float32(0.9)))
    states = [so.new_state(m, n) for m, n in case.shapes]
    for arrival, rho in enumerate((12, 5)):
        Ps = [rng.standard_normal((m, rho)).astype(np.float32) for m, n in case.shapes]
        Qs = [rng.standard_normal((n, rho)).astype(np.float32) for m, n in case.shapes]
        plan.anchor_update_factored([torch.from_numpy(x).cuda() for x in Ps], [torch.from_numpy(x).cuda() for x in Qs], arrival)
        for st, P, Q, (m, n) in zip(states, Ps, Qs, case.shapes):
            so.anchor_update(st, P.astype(np.float64) @ Q.astype(np.float64).T, hp, 8, mode="mirror",
                             Omega=so.rademacher_sketch(0, 0, n, 8), q=1)
    torch.cuda.synchronize()
    for i, st in enumerate(states):
        assert rel(plan.export_anchor_momentum(i).double().cpu().numpy(), st.M_anc) < 1e-6
        U, s, V = [x.double().cpu().numpy() for x in plan.export_basis(i)]
        tol = TOL if engine == 0 else 1e-4
        assert so.projector_distance(U, st.U) < tol and so.projector_distance(V, st.V) < tol and rel(s, st.s) < tol
    import paper_2609_14339_b200 as sc
    with pytest.raises(sc.SCError):
        plan.anchor_update_factored([None, torch.zeros((200, 4), device="cuda")], [torch.zeros((256, 4), device="cuda"), None], 9)


def test_global_clipping_and_in_step_rescale_on_the_tensor_engine(torch):
    """max_grad_norm on: projections of all classes first, one clip factor from the closed-form norms, then the
    updates; grads_prescaled = 0: the step applies 1/keep itself."""
    case = Case(shapes=[(256, 384), (384, 256), (256, 384)], rank=16, tokens=128, keep=0.25, prescaled=False,
                max_grad_norm=0.2, tau_p=30.0, planted=4)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.uses_tc and g.dev_status == 0
    o = OracleRun(case, inp, "mirror")
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL, es
    total = sum(np.sum(x * x) for x in g.gproj)
    assert abs(np.sqrt(total) - 0.2) < 2e-4
    assert 0.0 < g.clip < 1.0


def test_every_tile_of_every_matrix_is_updated_exactly_once(torch):
    """Thousands of work items over ten matrices of two shape classes (the update kernel hands them out through an
    atomic counter): every element of every matrix against the CUDA-core engine run from the same basis, and a second
    run of the tensor-core engine from the same state bit for bit."""
    import paper_2609_14339_b200 as sc
    dev = torch.device("cuda", 0)
    shapes = [(1024, 2048)] * 6 + [(1536, 1024)] * 4
    g = torch.Generator(device=dev); g.manual_seed(17)
    rnd = lambda s, scale=1.0: torch.randn(s, generator=g, device=dev) * scale
    # low-rank signal plus noise, so that the basis is well defined
    def grad(s, seed_rank=8):
        m, n = s
        return (rnd((m, seed_rank)) @ rnd((seed_rank, n)) * 3.0 + rnd(s)).to(torch.bfloat16)
    Ga = [grad(s) for s in shapes]
    G = [grad(s) for s in shapes]
    W0 = [rnd(s, 0.02) for s in shapes]
    m0 = [rnd(s, 0.1) for s in shapes]
    v0 = [torch.rand(s, generator=g, device=dev) * 4.0 + 0.1 for s in shapes]

    def run(engine, bases=None):
        hp = sc.Hparams.default(tau_p=60.0, lr=1e-2, weight_decay=0.01, engine=engine)
        plan = sc.Plan(shapes, 32, 0.25, hp, device=dev)
        plan.anchor_update(Ga, 0)
        if bases is not None:
            for i, (U, s, V) in enumerate(bases):
                plan.import_basis(i, U, s, V)
        W = [x.clone() for x in W0]; m = [x.clone() for x in m0]; v = [x.clone() for x in v0]
        Wb = [torch.zeros(s, dtype=torch.bfloat16, device=dev) for s in shapes]
        assert plan.correct_and_step(G, W, m, v, 50, params_bf16=Wb) == 0
        torch.cuda.synchronize()
        assert plan.get_device_status() == 0
        out_bases = [plan.export_basis(i) for i in range(len(shapes))]
        used_tc = plan.uses_tensor_cores()
        plan.close()
        return W, m, v, Wb, out_bases, used_tc

    W1, m1, v1, Wb1, bases, tc1 = run(sc.SC_ENGINE_AUTO)
    W2, m2, v2, Wb2, _, tc2 = run(sc.SC_ENGINE_AUTO)
    assert tc1 and tc2
    for a, b in zip(W1 + m1 + v1 + Wb1, W2 + m2 + v2 + Wb2):
        assert torch.equal(a, b)
    W3, m3, v3, Wb3, _, tc3 = run(sc.SC_ENGINE_SIMT, bases)
    assert not tc3
    for i in range(len(shapes)):
        dW1 = (W1[i] - W0[i]).double(); dW3 = (W3[i] - W0[i]).double()
        assert float((dW1 - dW3).norm() / dW3.norm()) < 1e-4, i
        assert float((m1[i] - m3[i]).double().norm() / m3[i].double().norm()) < 1e-5, i
        assert float((v1[i] - v3[i]).double().norm() / v3[i].double().norm()) < 1e-5, i
        # element-wise as well: a tile applied twice or not at all moves dW by its whole size there
        assert float((dW1 - dW3).abs().max()) < 2e-2 * float(dW3.abs().max()), i


@pytest.mark.parametrize("rank,tiles", [(96, 2), (128, 2), (128, 3), (256, 0), (200, 3)])
@pytest.mark.parametrize("optimizer", [0, 1])
def test_ranks_above_64_with_the_basis_panel_in_tensor_memory(torch, rank, tiles, optimizer, monkeypatch):
    """Ranks above 64 keep the U panel of a work item in tensor memory (runs of `tiles` column tiles per item; the
    library picks that path by itself for rank > 128 or large plans, here the run length is forced through its test
    hook so that small matrices take it too). Ragged edges in both dimensions, several matrices, a last run that is
    shorter than the others; AdamW and the dual-EMA optimizer."""
    if tiles:
        monkeypatch.setenv("SC_UT_TILES", str(tiles))
    case = Case(shapes=[(520, 712), (520, 712), (264, 1160)], rank=rank, tokens=768, keep=0.25, planted=rank // 2, seed=6,
                tau_p=120.0, optimizer=optimizer, beta3=0.99, mix_alpha=3.0)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.uses_tc and g.dev_status == 0
    o = OracleRun(case, inp, "mirror")
    eb = compare_basis(g, o)
    assert max(eb["PU"], eb["PV"], eb["s"]) < TOL, eb
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"], es.get("ms", 0.0)) < TOL, es
    # the same basis through the path that re-fetches U per tile: G_proj to rounding, everything else to 1e-6
    monkeypatch.setenv("SC_NO_TMEM_U", "1")
    g0 = GpuRun(case, inp, torch)
    for i in range(len(case.shapes)):
        assert rel(g.gproj[i], g0.gproj[i]) < 1e-6 and rel(g.W[i], g0.W[i]) < 1e-6
        assert float(np.abs(g.gproj[i] - g0.gproj[i]).max()) < 1e-4 * float(np.abs(g0.gproj[i]).max())


@pytest.mark.parametrize("rank", [8, 48, 64, 128])
def test_filter_and_ct_in_one_launch_match_the_separate_launches_bit_for_bit(torch, rank, monkeypatch):
    """Plans with few matrices form the r x r filter and C^T = V Xs^T in one launch; the batched launches that large
    plans use are forced through the library's test hook. Both add up the rank index in the same order, so the
    step's results agree bit for bit; the statistics (summed in another order) agree to rounding."""
    case = Case(shapes=[(520, 712), (520, 712), (264, 1160)], rank=rank, tokens=768, keep=0.25, planted=max(2, rank // 2),
                seed=11, tau_p=120.0)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.uses_tc and g.dev_status == 0
    o = OracleRun(case, inp, "mirror")
    es = compare_step(g, o)
    assert max(es["gproj"], es["m"], es["v"], es["dW"]) < TOL, es
    monkeypatch.setenv("SC_NO_FUSED_FILTER", "1")
    g0 = GpuRun(case, inp, torch)
    for i in range(len(case.shapes)):
        assert np.array_equal(g.gproj[i], g0.gproj[i]) and np.array_equal(g.W[i], g0.W[i]), i
        assert np.array_equal(g.m[i], g0.m[i]) and np.array_equal(g.v[i], g0.v[i]) and np.array_equal(g.Wb[i], g0.Wb[i]), i
    for a, b in zip(g.stats, g0.stats):
        for key in a:
            assert abs(a[key] - b[key]) <= 1e-5 * abs(b[key]), (key, a, b)
