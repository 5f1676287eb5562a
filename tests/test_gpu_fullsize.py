"""Parity at the full sizes of the benchmark's configs, in the launch configuration bench.py times.

Inputs come from the torch backend of the seeded generator (they only fit on the GPU); the matrices that are
checked are copied to the host and pushed through the fp64 oracle (MIRROR mode: same sketch, l, q, r), one matrix
per distinct shape; every matrix of the plan is checked through properties that hold at any size.
Tolerance: 2e-3 relative Frobenius (bf16 operands)."""
import numpy as np
import pytest

from oracle import spectral_oracle as so
from parity_util import rel
from synth import generator as gen

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _f32(x):
    return float(np.float32(x))


def _run_config(torch, name, layers=None, lr=1e-2, tau_p=None, n_arrivals=1, warm=False, q_warm=0):
    """n_arrivals anchor gradients (independent batches) arrive before the step; warm=True is the refresh bench.py
    times: cold start with one power iteration on the first arrival, then warm starts from the previous right basis
    with q_warm power iterations (two sweeps per arrival plus two per iteration)."""
    import paper_2609_14339_b200 as sc
    import bench
    cfg = dict(gen.CONFIGS[name])
    if layers is not None:
        cfg["layers"] = layers
    saved = gen.CONFIGS[name]
    gen.CONFIGS[name] = cfg
    try:
        device = torch.device("cuda", 0)
        cfg, shapes, buf = bench.build_workload(name, device, torch)
    finally:
        gen.CONFIGS[name] = saved
    r, keep = cfg["r"], cfg["keep"]
    # tau_p of the order of the singular values so that the soft filter is active (d well inside (0, 1))
    T = cfg["tokens"]
    m0, n0 = shapes[0]
    if tau_p is None:
        tau_p = 3.0 * 0.1 * np.sqrt(T) * (np.sqrt(m0) + np.sqrt(n0))
    hp = sc.Hparams.default(tau_p=tau_p, lr=lr, weight_decay=0.01, power_iters=1, collect_stats=1,
                            warm_start=int(warm), warm_power_iters=q_warm)
    plan = sc.Plan(shapes, r, keep, hp, device=device)
    assert plan.uses_tensor_cores()
    # one sampled matrix per distinct shape (the first of each)
    sampled = {}
    for i, s in enumerate(shapes):
        sampled.setdefault(s, i)
    idxs = sorted(sampled.values())
    host = {i: dict(G=buf["G"][i].double().cpu().numpy(), Ga=[buf["Ga"][i].double().cpu().numpy()],
                    W=buf["W"][i].double().cpu().numpy(), m=buf["M1"][i].double().cpu().numpy(),
                    v=buf["M2"][i].double().cpu().numpy()) for i in idxs}
    gp = [torch.empty(shapes[i], dtype=torch.float32, device=device) if i in host else None for i in range(len(shapes))]
    plan.set_debug_gproj_out(gp)
    plan.anchor_update(buf["Ga"], 0)
    per_layer = len(cfg["shapes"])
    for a in range(1, n_arrivals):
        anc = []
        for i, (m, n) in enumerate(shapes):
            spec = gen.GradSpec(m=m, n=n, tokens=cfg["tokens"], keep=keep, planted_rank=cfg["k"], snr=1.0, seed=0,
                                layer=i // per_layer, mat_id=i % per_layer)
            anc.append(gen.torch_gradients(spec, a, device, buf["Ga"][i].dtype, anchor=True))
            if i in host:
                host[i]["Ga"].append(anc[-1].double().cpu().numpy())
        plan.anchor_update(anc, a)
        torch.cuda.synchronize()
        del anc
    assert plan.correct_and_step(buf["G"], buf["W"], buf["M1"], buf["M2"], 100, params_bf16=buf["Wb"]) == 0
    torch.cuda.synchronize()
    assert plan.get_device_status() == 0
    stats, clip = plan.get_stats()

    ohp = so.Hyper(alpha=_f32(0.3), tau_p=_f32(tau_p), beta_anc=_f32(0.9), lr=_f32(lr), beta1=_f32(0.9), beta2=_f32(0.999),
                   eps=_f32(1e-8), weight_decay=_f32(0.01), keep=_f32(keep))
    worst = {}
    for i in idxs:
        m, n = shapes[i]
        h = host[i]
        st = so.new_state(m, n)
        for Ga in h["Ga"]:
            so.anchor_update(st, Ga, ohp, r, mode="mirror", Omega=so.rademacher_sketch(0, 0, n, r), q=1, warm=warm,
                             q_warm=q_warm)
        Wn, mn, vn, gpo = so.correct_and_step([st], [h["G"]], [h["W"]], [h["m"]], [h["v"]], 100, ohp)
        U, s, V = [x.double().cpu().numpy() for x in plan.export_basis(i)]
        orth = max(float(np.abs(U.T @ U - np.eye(r)).max()), float(np.abs(V.T @ V - np.eye(r)).max()))
        # (the projector distance below re-orthonormalises its inputs, so orthonormality is checked on its own; the
        # last Cholesky-QR round takes its Gram matrix from tf32 tensor cores, which bounds it near 1e-4)
        assert orth <= (1e-4 if r <= 128 else 2e-4), (name, shapes[i], orth)
        Mg = plan.export_anchor_momentum(i).double().cpu().numpy()
        assert rel(Mg, st.M_anc) < 1e-6, (name, shapes[i])
        del Mg
        worst["orth"] = max(worst.get("orth", 0.0), orth)
        e = dict(PU=so.projector_distance(U, st.U), PV=so.projector_distance(V, st.V), s=rel(s, st.s),
                 gproj=rel(gp[i].double().cpu().numpy(), gpo[0]),
                 m=rel(buf["M1"][i].double().cpu().numpy(), mn[0]), v=rel(buf["M2"][i].double().cpu().numpy(), vn[0]),
                 dW=rel(buf["W"][i].double().cpu().numpy() - h["W"], Wn[0] - h["W"]),
                 Wb=rel(buf["Wb"][i].double().cpu().numpy(), Wn[0]))
        d = so.filter_weights(st.s, ohp.tau_p)
        assert 0.05 < d.min() and d.max() < 0.98, (d.min(), d.max())       # the filter really is active
        for k, v_ in e.items():
            worst[k] = max(worst.get(k, 0.0), v_)
        assert max(e["PU"], e["PV"], e["s"], e["gproj"], e["m"], e["v"], e["dW"]) < TOL, (name, shapes[i], e)
        assert e["Wb"] < 5e-3
        # statistics against the oracle
        X = so.project(st.U, h["G"], st.V)
        assert abs(stats[i]["x_sqnorm"] / np.sum(X * X) - 1) < 5e-3
        assert abs(stats[i]["g_sqnorm"] / np.sum(h["G"] ** 2) - 1) < 1e-3
    # properties on every matrix: finite state, 0 <= eta_r <= 1, Lemma 1 via the closed-form norm, r_eff in (0, r)
    for i in range(len(shapes)):
        st_i = stats[i]
        eta = st_i["x_sqnorm"] / st_i["g_sqnorm"]
        assert 0.0 <= eta <= 1.0 + 1e-3
        assert st_i["gproj_sqnorm"] <= st_i["g_sqnorm"] * (1 + 1e-3)           # alpha g + (1-alpha) P g never grows
        assert 0.0 < st_i["r_eff"] < r
    for t in (buf["W"], buf["M1"], buf["M2"]):
        assert all(bool(torch.isfinite(x).all()) for x in t[:: max(1, len(t) // 16)])
    return worst


def test_llama8b_full_set_as_benchmarked(torch):
    """Config 3 exactly as bench.py launches it: 224 matrices, rank 64, keep 0.1, T = 4096."""
    worst = _run_config(torch, "llama8b")
    print("llama8b worst errors", worst)


def test_llama1b_two_layers_full_shapes(torch):
    worst = _run_config(torch, "llama1b", layers=2)
    print("llama1b worst errors", worst)


def test_llama70b_slice_one_layer_full_shapes(torch):
    """Config 5 shapes (8192 hidden, 28672 FFN, rank 128): two K chunks in the update kernel, 470 MB matrices."""
    worst = _run_config(torch, "llama70b_slice", layers=1)
    print("llama70b worst errors", worst)


@pytest.mark.parametrize("q_warm", [1, 0])
def test_llama8b_two_layers_warm_refresh_as_benchmarked(torch, q_warm):
    """The refresh bench.py times (cold q = 1 once, then warm starts with q = 1; q = 0 is the cheaper option), at full
    size: two 8B-shaped layers (all seven shapes), three arrivals of independent anchor batches, against the oracle's
    MIRROR mode with warm=True."""
    worst = _run_config(torch, "llama8b", layers=2, n_arrivals=3, warm=True, q_warm=q_warm)
    print("llama8b warm worst errors", q_warm, worst)


def test_planted_subspace_against_the_exact_oracle_at_the_benchmarked_settings(torch):
    """The well-posed part of the rule against the EXACT oracle (full fp64 SVD), at the range-finder settings bench.py
    times (l = r, cold q = 1, warm starts with q = 1), on the attention shapes of the 8B set after three arrivals of
    independent anchor batches: the planted rank-32 subspace (a wide spectral gap below it) and the filtered gradient
    restricted to it must meet the stated 2e-3. The other half of the rank-64 basis lies in a gapless noise bulk where
    the rank cut itself is ill-posed; that part is reported by bench.py, not gated."""
    import paper_2609_14339_b200 as sc
    import bench
    saved = gen.CONFIGS["llama8b"]
    gen.CONFIGS["llama8b"] = dict(saved, layers=1)
    try:
        device = torch.device("cuda", 0)
        cfg, shapes, buf = bench.build_workload("llama8b", device, torch)
    finally:
        gen.CONFIGS["llama8b"] = saved
    hp = sc.Hparams.default(power_iters=1, warm_start=1, warm_power_iters=1, tau_p=1e-3)
    plan = sc.Plan(shapes, cfg["r"], cfg["keep"], hp, device=device)
    plan.anchor_update(buf["Ga"], 0)
    for a in (1, 2):
        anc = []
        for i, (m, n) in enumerate(shapes):
            spec = gen.GradSpec(m=m, n=n, tokens=cfg["tokens"], keep=cfg["keep"], planted_rank=cfg["k"], snr=1.0, seed=0,
                                layer=0, mat_id=i)
            anc.append(gen.torch_gradients(spec, a, device, torch.bfloat16, anchor=True))
        plan.anchor_update(anc, a)
        torch.cuda.synchronize()
    assert plan.get_device_status() == 0
    for mat in (0, 1):                                     # 4096 x 4096 and 1024 x 4096
        rep = bench.exact_parity_report(plan, cfg, shapes, buf, mat, 0.3, 1e-3)
        print("exact-side report", rep)
        assert rep["relative_gap_at_k"] > 0.1                      # the planted subspace is well separated
        assert rep["top_k_projector_distance_U"] < TOL and rep["top_k_projector_distance_V"] < TOL, rep
        assert rep["gfilt_top_k_rel_vs_exact"] < TOL, rep


@pytest.mark.parametrize("rank,keep", [(8, 0.05), (16, 0.1), (32, 0.1), (128, 0.1), (256, 0.5)])
def test_ffn_sweep_corner_cells(torch, rank, keep):
    """Config 4: one 14336x4096 matrix; every rank class of the sweep (the smallest and largest at the extreme keep
    ratios; 16 and 32 exercise the padding of the basis to whole MMA K steps, 128 the two-chunk operand path)."""
    saved = dict(gen.CONFIGS["ffn_sweep"])
    gen.CONFIGS["ffn_sweep"] = dict(saved, r=rank, keep=keep, k=max(rank // 2, 1))
    try:
        worst = _run_config(torch, "ffn_sweep")
    finally:
        gen.CONFIGS["ffn_sweep"] = saved
    print("ffn_sweep", rank, keep, worst)
