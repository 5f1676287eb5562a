"""The dual-EMA (AdEMAMix) optimizer applied to the corrected gradient G_proj (appendix "On the Compatibility with
Dual-EMA Optimizers"), on both engines, against the fp64 oracle: G_proj, the fast and slow averages, the second
moment and the weight change.  Tolerances: 2e-3 for bf16 gradients on the tensor cores, 1e-5 for the fp32 engine."""
import numpy as np
import pytest

from parity_util import Case, GpuRun, OracleRun, compare_basis, compare_step, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _check(es, tol):
    assert max(es["gproj"], es["m"], es["ms"], es["v"], es["dW"]) < tol, es
    assert es["Wb"] < 5e-3


@pytest.mark.parametrize("engine,dtype,tol", [(0, "bf16", 2e-3), (1, "fp32", 1e-5), (1, "bf16", 1e-5)])
def test_dual_ema_step_matches_the_oracle(torch, engine, dtype, tol):
    # several tiles with ragged edges; two shape classes; active filter; clip on for one matrix pair
    shapes = [(384, 520), (200, 136), (384, 520)]
    case = Case(shapes=shapes, rank=12, dtype=dtype, tokens=192, keep=0.25, planted=4, seed=5, tau_p=40.0, engine=engine,
                optimizer=1, beta3=0.99, mix_alpha=5.0, max_grad_norm=0.0, n_anchor=2)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    assert g.dev_status == 0 and g.step_status == 0 and g.uses_tc == (engine == 0)
    o = OracleRun(case, inp, "mirror")
    eb = compare_basis(g, o)
    assert max(eb["PU"], eb["PV"], eb["s"]) < tol, eb
    _check(compare_step(g, o), tol)
    # the slow average really moved, and by (1 - beta3) (G_proj - m_slow)
    for i in range(len(shapes)):
        want = 0.99 * inp["ms"][i].astype(np.float64) + (1 - np.float64(np.float32(0.99))) * o.gproj[i]
        assert np.linalg.norm(g.ms[i] - want) / np.linalg.norm(want) < 1e-3


@pytest.mark.parametrize("engine", [0, 1])
def test_dual_ema_with_clipping_and_rescale(torch, engine):
    case = Case(shapes=[(256, 384), (129, 200)], rank=16, tokens=128, keep=0.25, prescaled=False, max_grad_norm=0.2,
                tau_p=30.0, engine=engine, optimizer=1, beta3=0.999, mix_alpha=2.0)
    inp = make_inputs(case)
    g = GpuRun(case, inp, torch)
    o = OracleRun(case, inp, "mirror")
    _check(compare_step(g, o), 2e-3 if engine == 0 else 1e-5)
    total = sum(np.sum(x * x) for x in g.gproj)
    assert abs(np.sqrt(total) - 0.2) < 1e-4


@pytest.mark.parametrize("engine", [0, 1])
def test_mix_alpha_zero_is_adamw_bit_for_bit_in_the_moments(torch, engine):
    """With mix_alpha = 0 the slow average is carried but unused: W, m, v equal the AdamW plan's to rounding."""
    base = dict(shapes=[(256, 384)], rank=16, tokens=128, tau_p=20.0, engine=engine)
    inp = make_inputs(Case(**base))
    a = GpuRun(Case(**base), inp, torch)
    b = GpuRun(Case(**base, optimizer=1, mix_alpha=0.0), inp, torch)
    assert np.array_equal(a.m[0], b.m[0]) and np.array_equal(a.v[0], b.v[0]) and np.array_equal(a.gproj[0], b.gproj[0])
    assert np.linalg.norm(a.W[0] - b.W[0]) / np.linalg.norm(a.W[0]) < 1e-6


def test_dual_ema_needs_its_state_array(torch):
    import paper_2609_14339_b200 as sc
    from parity_util import make_plan, to_dev
    case = Case(shapes=[(64, 64)], rank=4, dtype="fp32", engine=1, optimizer=1)
    inp = make_inputs(case)
    plan = make_plan(case, torch)
    G = [to_dev(inp["G"][0], "fp32", torch, "cuda:0")]
    W = [torch.from_numpy(inp["W"][0].copy()).cuda()]
    with pytest.raises(sc.SCError) as e:
        plan.correct_and_step(G, W, [W[0].clone()], [W[0].clone()], 1)
    assert e.value.status == -1
    with pytest.raises(sc.SCError):
        sc.Plan([(64, 64)], 4, 0.5, sc.Hparams.default(optimizer=1, beta3=1.0))


def test_dual_ema_full_size_ffn_matrix_sampled(torch):
    """One 14336 x 4096 bf16 matrix (the launch configuration the dual-EMA bench line times): every tile of the
    persistent kernel, checked on the whole matrix against the oracle."""
    import paper_2609_14339_b200 as sc
    from oracle import spectral_oracle as so
    from synth import generator as gen
    from parity_util import rel
    m, n, r, T = 14336, 4096, 64, 4096
    dev = torch.device("cuda", 0)
    spec = gen.GradSpec(m=m, n=n, tokens=T, keep=0.1, planted_rank=32, snr=1.0, seed=0)
    G = gen.torch_gradients(spec, 1, dev, torch.bfloat16)
    Ga = gen.torch_gradients(spec, 0, dev, torch.bfloat16, anchor=True)
    gg = torch.Generator(device=dev); gg.manual_seed(77)
    W = torch.randn((m, n), generator=gg, device=dev) * 0.02
    m1 = torch.randn((m, n), generator=gg, device=dev) * 10.0
    m2 = torch.rand((m, n), generator=gg, device=dev) * 4000.0 + 100.0
    ms = torch.randn((m, n), generator=gg, device=dev) * 5.0
    Wb = torch.empty((m, n), device=dev, dtype=torch.bfloat16)
    tau = 3.0 * 0.1 * np.sqrt(T) * (np.sqrt(m) + np.sqrt(n))
    hp = sc.Hparams.default(tau_p=tau, lr=1e-2, weight_decay=0.01, optimizer=1, beta3=0.9999, mix_alpha=5.0)
    plan = sc.Plan([(m, n)], r, 0.1, hp, device=dev)
    host = [x.double().cpu().numpy() for x in (G, Ga, W, m1, m2, ms)]
    plan.anchor_update([Ga], 0)
    assert plan.correct_and_step([G], [W], [m1], [m2], 100, params_bf16=[Wb], exp_avg_slow=[ms]) == 0
    torch.cuda.synchronize()
    assert plan.get_device_status() == 0
    f = lambda x: float(np.float32(x))
    ohp = so.Hyper(alpha=f(0.3), tau_p=f(tau), beta_anc=f(0.9), lr=f(1e-2), beta1=f(0.9), beta2=f(0.999), eps=f(1e-8),
                   weight_decay=f(0.01), keep=f(0.1), beta3=f(0.9999), mix_alpha=f(5.0))
    st = so.new_state(m, n)
    so.anchor_update(st, host[1], ohp, r, mode="mirror", Omega=so.rademacher_sketch(0, 0, n, r), q=1)
    Wn, an, bn, vn, _ = so.correct_and_step_ademamix([st], [host[0]], [host[2]], [host[3]], [host[5]], [host[4]], 100, ohp)
    e = dict(m=rel(m1.double().cpu().numpy(), an[0]), ms=rel(ms.double().cpu().numpy(), bn[0]),
             v=rel(m2.double().cpu().numpy(), vn[0]), dW=rel(W.double().cpu().numpy() - host[2], Wn[0] - host[2]),
             Wb=rel(Wb.double().cpu().numpy(), Wn[0]))
    print("dual-EMA full-size errors", e)
    assert max(e["m"], e["ms"], e["v"], e["dW"]) < 2e-3 and e["Wb"] < 5e-3, e
