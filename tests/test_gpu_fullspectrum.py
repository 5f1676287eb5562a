"""Full-spectrum soft filter (the main-text form of Section 3.2: d_i = s_i / (s_i + tau_p) on ALL singular directions,
no rank cut) on the GPU against the plain definition in the fp64 oracle (full SVD): G_proj, AdamW moments and the
weight change.  Here nothing is ill-posed (the operator is a smooth function of the anchor momentum), so the
comparison is against the exact oracle, at the stated 2e-3 for bf16 operands."""
import numpy as np
import pytest

from oracle import spectral_oracle as so
from parity_util import Case, make_inputs, oracle_hyper, rel, to_dev
from synth import generator as gen

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def _run(torch, shapes, tau_p, n_anchor=2, tokens=192, planted=4, sqrt_iters=24, inv_iters=12, alpha=0.3, prescaled=True,
         keep=0.25):
    import paper_2609_14339_b200 as sc
    case = Case(shapes=shapes, rank=0, tokens=tokens, keep=keep, planted=planted, seed=7, tau_p=tau_p, n_anchor=n_anchor,
                alpha=alpha, prescaled=prescaled)
    inp = make_inputs(case)
    hp = sc.Hparams.default(alpha=alpha, tau_p=tau_p, lr=case.lr, weight_decay=case.weight_decay, full_spectrum=1,
                            fs_sqrt_iters=sqrt_iters, fs_inv_iters=inv_iters, grads_prescaled=int(prescaled))
    plan = sc.Plan(shapes, 0, keep, hp)
    assert plan.uses_tensor_cores()
    n = len(shapes)
    for a in range(n_anchor):
        plan.anchor_update([to_dev(inp["anchors"][i][a], "bf16", torch, "cuda:0") for i in range(n)], a)
    G = [to_dev(inp["G"][i], "bf16", torch, "cuda:0") for i in range(n)]
    W = [torch.from_numpy(inp["W"][i].copy()).cuda() for i in range(n)]
    m = [torch.from_numpy(inp["m"][i].copy()).cuda() for i in range(n)]
    v = [torch.from_numpy(inp["v"][i].copy()).cuda() for i in range(n)]
    Wb = [torch.zeros(s, dtype=torch.bfloat16, device="cuda:0") for s in shapes]
    gp = [torch.zeros(s, dtype=torch.float32, device="cuda:0") for s in shapes]
    plan.set_debug_gproj_out(gp)
    status = plan.correct_and_step(G, W, m, v, case.t0, params_bf16=Wb)
    torch.cuda.synchronize()
    assert plan.get_device_status() == 0
    ohp = oracle_hyper(case)
    out = []
    for i, (mm, nn) in enumerate(shapes):
        M = np.zeros((mm, nn))
        for a in range(n_anchor):
            M = so.anchor_ema(M, gen.stored_to_f64(inp["anchors"][i][a], "bf16"), ohp.beta_anc)
        Gi = gen.stored_to_f64(inp["G"][i], "bf16")
        gproj = so.correct_full_spectrum(M, Gi, ohp) if n_anchor else ohp.alpha * Gi * (1.0 if prescaled else 1.0 / ohp.keep)
        W0 = inp["W"][i].astype(np.float64)
        Wn, mn, vn = so.adamw_step(W0, inp["m"][i].astype(np.float64), inp["v"][i].astype(np.float64), gproj, case.t0,
                                   ohp.lr, ohp.beta1, ohp.beta2, ohp.eps, ohp.weight_decay)
        s = np.linalg.svd(M, compute_uv=False) if n_anchor else np.zeros(1)
        out.append(dict(gproj=rel(gp[i].double().cpu().numpy(), gproj), m=rel(m[i].double().cpu().numpy(), mn),
                        v=rel(v[i].double().cpu().numpy(), vn), dW=rel(W[i].double().cpu().numpy() - W0, Wn - W0),
                        Wb=rel(Wb[i].double().cpu().numpy(), Wn), d=so.filter_weights(s, ohp.tau_p),
                        gfilt_share=rel(gproj, ohp.alpha * Gi)))
    return status, out, plan


def test_two_matrices_against_the_exact_oracle(torch):
    # tau_p of the order of the singular values: d spreads over (0, 1), i.e. the filter does something on every direction
    status, out, _ = _run(torch, [(256, 384), (512, 256)], tau_p=60.0)
    assert status == 0
    for e in out:
        assert e["d"].max() > 0.6 and np.median(e["d"]) < 0.5 and e["gfilt_share"] > 0.1, (e["d"].max(), np.median(e["d"]))
        assert max(e["gproj"], e["m"], e["v"], e["dW"]) < TOL, e
        assert e["Wb"] < 5e-3
    print("full-spectrum errors", [{k: v for k, v in e.items() if k != "d"} for e in out])


def test_rescale_inside_and_alpha_limits(torch):
    _, out, _ = _run(torch, [(256, 256)], tau_p=40.0, prescaled=False, alpha=0.0)
    assert max(out[0]["gproj"], out[0]["m"], out[0]["dW"]) < TOL, out[0]
    _, out, _ = _run(torch, [(256, 256)], tau_p=40.0, alpha=1.0)
    assert out[0]["gproj"] < 1e-6                     # alpha = 1: the gradient passes through


def test_before_the_first_anchor(torch):
    status, out, _ = _run(torch, [(256, 320)], tau_p=10.0, n_anchor=0)
    assert status == 1                                 # SC_WARN_NO_ANCHOR; G_proj = alpha g
    assert out[0]["gproj"] < 1e-6 and out[0]["dW"] < 1e-5


def test_fewer_iterations_only_under_weight(torch):
    """Directions whose square root has not converged get a smaller weight, never a larger one: the result moves
    towards alpha g, and the error against the exact operator falls as iterations are added."""
    errs = []
    for it in (4, 10, 24):
        _, out, _ = _run(torch, [(256, 384)], tau_p=60.0, sqrt_iters=it)
        errs.append(out[0]["gproj"])
    assert errs[0] > errs[1] > errs[2] and errs[2] < TOL, errs


def test_attention_kv_shape_full_size(torch):
    """One 1024 x 4096 matrix (the k/v projection of the 8B-shaped layer): P_U is 1024^2, P_V 4096^2."""
    T = 1024
    tau = 3.0 * 0.1 * np.sqrt(T) * (np.sqrt(1024) + np.sqrt(4096))
    status, out, _ = _run(torch, [(1024, 4096)], tau_p=tau, n_anchor=1, tokens=T, planted=16, keep=0.1)
    e = out[0]
    print("full-spectrum 1024x4096", {k: v for k, v in e.items() if k != "d"}, "d range", e["d"].min(), e["d"].max())
    assert e["d"].max() > 0.5 and max(e["gproj"], e["m"], e["v"], e["dW"]) < TOL, e


def test_attention_qo_shape_full_size(torch):
    """One 4096 x 4096 matrix (the q / o projection of the 8B-shaped layer), as bench.py --full-spectrum launches it:
    both soft projectors are 4096^2, every contraction runs 256 tiles of 256 x 256 over the 74 pairs of SMs."""
    T = 1024
    tau = 3.0 * 0.1 * np.sqrt(T) * (np.sqrt(4096) + np.sqrt(4096))
    status, out, _ = _run(torch, [(4096, 4096)], tau_p=tau, n_anchor=1, tokens=T, planted=16, keep=0.1)
    e = out[0]
    print("full-spectrum 4096x4096", {k: v for k, v in e.items() if k != "d"}, "d range", e["d"].min(), e["d"].max())
    assert e["d"].max() > 0.5 and max(e["gproj"], e["m"], e["v"], e["dW"]) < TOL, e


def test_checkpoint_rebuilds_the_soft_projectors(torch):
    """The checkpoint blob carries the anchor momentum only; an importing full-spectrum plan rebuilds P_U and P_V from
    it, and a step afterwards is bit-identical to the exporting plan's."""
    import paper_2609_14339_b200 as sc
    shapes = [(256, 384), (256, 256)]
    case = Case(shapes=shapes, rank=0, tokens=192, keep=0.25, planted=4, seed=9, tau_p=50.0)
    inp = make_inputs(case)
    hp = sc.Hparams.default(tau_p=50.0, lr=1e-2, full_spectrum=1)
    a, b = sc.Plan(shapes, 0, 0.25, hp), sc.Plan(shapes, 0, 0.25, hp)
    anc = [to_dev(inp["anchors"][i][0], "bf16", torch, "cuda:0") for i in range(2)]
    a.anchor_update([anc[0], None], 3)                    # the second matrix has no anchor yet
    b.state_import(a.state_export())
    assert b.get_anchor_info() == (3, 1)
    G = [to_dev(inp["G"][i], "bf16", torch, "cuda:0") for i in range(2)]
    outs = []
    for plan in (a, b):
        W = [torch.from_numpy(inp["W"][i].copy()).cuda() for i in range(2)]
        m = [torch.from_numpy(inp["m"][i].copy()).cuda() for i in range(2)]
        v = [torch.from_numpy(inp["v"][i].copy()).cuda() for i in range(2)]
        assert plan.correct_and_step(G, W, m, v, 100) == 0
        torch.cuda.synchronize()
        outs.append(W + m + v)
    assert all(torch.equal(x, y) for x, y in zip(*outs))


def test_rejects_unsupported_configurations(torch):
    import paper_2609_14339_b200 as sc
    hp = sc.Hparams.default(full_spectrum=1, tau_p=1.0)
    with pytest.raises(sc.SCError) as e:
        sc.Plan([(256, 256)], 4, 0.5, hp)              # a rank makes no sense without a rank cut
    assert e.value.status == -1
    with pytest.raises(sc.SCError) as e:
        sc.Plan([(200, 256)], 0, 0.5, hp)
    assert e.value.status in (-1, -2)
    for bad in (dict(tau_p=0.0), dict(max_grad_norm=1.0), dict(optimizer=1), dict(grad_dtype=1), dict(fs_sqrt_iters=0)):
        with pytest.raises(sc.SCError):
            sc.Plan([(256, 256)], 0, 0.5, sc.Hparams.default(**{**dict(full_spectrum=1, tau_p=1.0), **bad}))
