"""Shared driver for the GPU parity tests: same seeded inputs to the CUDA path (through the C ABI
binding) and to the fp64 oracle, then element-wise / projector comparisons."""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from oracle import spectral_oracle as so
from synth import generator as gen


def rel(a, b) -> float:
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


@dataclass
class Case:
    shapes: list
    rank: int
    dtype: str = "bf16"            # gradient storage type
    tokens: int = 256
    keep: float = 0.25
    planted: int = 0
    snr: float = 1.0
    seed: int = 0
    l: int = 0                     # sketch width (0 = rank)
    q: int = 1
    alpha: float = 0.3
    tau_p: float = 1e-3
    beta_anc: float = 0.9
    lr: float = 1e-2               # large enough that fp32 storage rounding of W does not hide the update
    weight_decay: float = 0.01
    eps: float = 1e-8
    max_grad_norm: float = 0.0
    prescaled: bool = True
    warmed: bool = True
    t0: int = 100                  # optimizer step count used with a warmed state
    engine: int = 0
    n_anchor: int = 1              # anchor arrivals before the step
    warm: bool = False             # warm-started range finder from the second arrival on
    q_warm: int = 0
    optimizer: int = 0             # 0 AdamW, 1 dual EMA (AdEMAMix) on G_proj
    beta3: float = 0.99
    mix_alpha: float = 5.0
    extra: dict = field(default_factory=dict)


def specs(case: Case):
    return [gen.GradSpec(m=m, n=n, tokens=case.tokens, keep=case.keep, planted_rank=case.planted, snr=case.snr,
                         seed=case.seed, layer=i // 7, mat_id=i % 7 + 10 * (i // 7)) for i, (m, n) in enumerate(case.shapes)]


def make_inputs(case: Case):
    """Stored arrays (exact bits both sides see) for anchors, masked gradient and optimizer state."""
    sp = specs(case)
    out = dict(specs=sp, anchors=[], G=[], W=[], m=[], v=[], ms=[])
    for s in sp:
        out["anchors"].append([gen.round_to(gen.anchor_gradient(s, a), case.dtype) for a in range(case.n_anchor)])
        out["G"].append(gen.round_to(gen.masked_gradient(s, case.n_anchor + 1, rescale=case.prescaled), case.dtype))
        W, m, v = gen.optimizer_state(s, warmed=case.warmed)
        out["W"].append(W); out["m"].append(m); out["v"].append(v)
        # slow EMA of the dual-EMA optimizer: a seeded array of its own (a shifted, rescaled copy of the fast moment)
        out["ms"].append(np.ascontiguousarray(np.roll(m, 1, axis=1) * np.float32(0.5)))
    return out


def oracle_hyper(case: Case) -> so.Hyper:
    """The hyper-parameters as the C ABI receives them: the ABI's fields are C floats, so both sides get the
    fp32-rounded values (0.999 as a float is 0.99900001287..., which moves 1 - beta2 by 1.3e-5 relative)."""
    f = lambda x: float(np.float32(x))
    return so.Hyper(alpha=f(case.alpha), tau_p=f(case.tau_p), beta_anc=f(case.beta_anc), lr=f(case.lr), eps=f(case.eps),
                    weight_decay=f(case.weight_decay), max_grad_norm=f(case.max_grad_norm),
                    beta1=f(0.9), beta2=f(0.999), grads_prescaled=case.prescaled, keep=f(case.keep),
                    beta3=f(case.beta3), mix_alpha=f(case.mix_alpha))


def to_dev(arr, dtype: str, torch, device):
    if dtype == "bf16":
        return torch.from_numpy(arr.view(np.int16).copy()).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr, np.float32)).to(device)


def make_plan(case: Case, torch, device="cuda:0"):
    import paper_2609_14339_b200 as sc
    hp = sc.Hparams.default(alpha=case.alpha, tau_p=case.tau_p, beta_anc=case.beta_anc, lr=case.lr, eps=case.eps,
                            weight_decay=case.weight_decay, max_grad_norm=case.max_grad_norm,
                            grads_prescaled=int(case.prescaled),
                            grad_dtype=sc.SC_DTYPE_BF16 if case.dtype == "bf16" else sc.SC_DTYPE_FP32,
                            sketch_width=case.l, power_iters=case.q, engine=case.engine, collect_stats=1,
                            warm_start=int(case.warm), warm_power_iters=case.q_warm,
                            optimizer=case.optimizer, beta3=case.beta3, mix_alpha=case.mix_alpha,
                            seed=case.seed)
    return sc.Plan(case.shapes, case.rank, case.keep, hp, device=device)


class GpuRun:
    """Runs the CUDA path for a Case and keeps everything needed for comparisons on the host (fp64)."""

    def __init__(self, case: Case, inputs, torch, device="cuda:0", import_bases=None):
        self.case = case
        self.plan = make_plan(case, torch, device)
        n = len(case.shapes)
        for a in range(case.n_anchor):
            anc = [to_dev(inputs["anchors"][i][a], case.dtype, torch, device) for i in range(n)]
            self.plan.anchor_update(anc, a)
        self.status_after_anchor = self.plan.get_device_status()
        if import_bases is not None:
            for i, (U, s, V) in enumerate(import_bases):
                self.plan.import_basis(i, torch.from_numpy(U), torch.from_numpy(s), torch.from_numpy(V))
        self.M_anc = [self.plan.export_anchor_momentum(i).double().cpu().numpy() for i in range(n)]
        self.basis = []
        for i in range(n):
            U, s, V = self.plan.export_basis(i)
            self.basis.append((U.double().cpu().numpy(), s.double().cpu().numpy(), V.double().cpu().numpy()))
        G = [to_dev(inputs["G"][i], case.dtype, torch, device) for i in range(n)]
        W = [torch.from_numpy(inputs["W"][i].copy()).to(device) for i in range(n)]
        m = [torch.from_numpy(inputs["m"][i].copy()).to(device) for i in range(n)]
        v = [torch.from_numpy(inputs["v"][i].copy()).to(device) for i in range(n)]
        ms = [torch.from_numpy(inputs["ms"][i].copy()).to(device) for i in range(n)] if case.optimizer == 1 else None
        Wb = [torch.zeros(s, dtype=torch.bfloat16, device=device) for s in case.shapes]
        gp = [torch.zeros(s, dtype=torch.float32, device=device) for s in case.shapes]
        self.plan.set_debug_gproj_out(gp)
        t = case.t0 if case.warmed else 1
        self.step_status = self.plan.correct_and_step(G, W, m, v, t, params_bf16=Wb, exp_avg_slow=ms)
        torch.cuda.synchronize()
        self.dev_status = self.plan.get_device_status()
        self.stats, self.clip = self.plan.get_stats()
        self.W = [x.double().cpu().numpy() for x in W]
        self.m = [x.double().cpu().numpy() for x in m]
        self.v = [x.double().cpu().numpy() for x in v]
        self.ms = [x.double().cpu().numpy() for x in ms] if ms is not None else None
        self.Wb = [x.float().double().cpu().numpy() for x in Wb]
        self.gproj = [x.double().cpu().numpy() for x in gp]
        self.uses_tc = self.plan.uses_tensor_cores()


class OracleRun:
    """The same sequence through the oracle. basis_mode: 'mirror' (same sketch, l, q), 'exact', or a list of bases."""

    def __init__(self, case: Case, inputs, basis_mode="mirror"):
        hp = oracle_hyper(case)
        n = len(case.shapes)
        self.states = []
        l = case.l if case.l > 0 else case.rank
        for i, (mm, nn) in enumerate(case.shapes):
            st = so.new_state(mm, nn)
            for a in range(case.n_anchor):
                Ga = gen.stored_to_f64(inputs["anchors"][i][a], case.dtype)
                if isinstance(basis_mode, str) and basis_mode == "mirror":
                    Om = so.rademacher_sketch(case.seed, 0, nn, l) if case.rank > 0 else None
                    so.anchor_update(st, Ga, hp, case.rank, mode="mirror", Omega=Om, q=case.q, warm=case.warm,
                                     q_warm=case.q_warm)
                elif isinstance(basis_mode, str):
                    so.anchor_update(st, Ga, hp, case.rank, mode="exact")
                else:
                    st.M_anc = so.anchor_ema(st.M_anc, Ga, hp.beta_anc)
            if not isinstance(basis_mode, str):
                st.U, st.s, st.V = basis_mode[i]
            self.states.append(st)
        G = [gen.stored_to_f64(inputs["G"][i], case.dtype) for i in range(n)]
        t = case.t0 if case.warmed else 1
        self.W0 = [np.asarray(w, np.float64) for w in inputs["W"]]
        f64 = lambda key: [np.asarray(x, np.float64) for x in inputs[key]]
        if case.optimizer == 1:
            self.W, self.m, self.ms, self.v, self.gproj = so.correct_and_step_ademamix(
                self.states, G, self.W0, f64("m"), f64("ms"), f64("v"), t, hp)
        else:
            self.ms = None
            self.W, self.m, self.v, self.gproj = so.correct_and_step(self.states, G, self.W0, f64("m"), f64("v"), t, hp)
        self.G = G
        self.hp = hp


def compare_step(g: GpuRun, o: OracleRun, mask_small_g=False):
    """Relative Frobenius errors of G_proj, m, v and the weight update, worst over matrices."""
    errs = dict(gproj=0.0, m=0.0, v=0.0, dW=0.0, W=0.0, Wb=0.0)
    for i in range(len(o.W)):
        errs["gproj"] = max(errs["gproj"], rel(g.gproj[i], o.gproj[i]))
        errs["m"] = max(errs["m"], rel(g.m[i], o.m[i]))
        errs["v"] = max(errs["v"], rel(g.v[i], o.v[i]))
        if o.ms is not None:
            errs["ms"] = max(errs.get("ms", 0.0), rel(g.ms[i], o.ms[i]))
        dWg = g.W[i] - o.W0[i]
        dWo = o.W[i] - o.W0[i]
        if mask_small_g:
            gp = o.gproj[i]
            keep = np.abs(gp) >= 1e-3 * np.sqrt(np.mean(gp * gp))
            dWg = dWg * keep; dWo = dWo * keep
        errs["dW"] = max(errs["dW"], rel(dWg, dWo))
        errs["W"] = max(errs["W"], rel(g.W[i], o.W[i]))
        errs["Wb"] = max(errs["Wb"], rel(g.Wb[i], o.W[i]))
    return errs


def compare_basis(g: GpuRun, o: OracleRun):
    errs = dict(M=0.0, PU=0.0, PV=0.0, s=0.0, orth=0.0)
    for i, st in enumerate(o.states):
        errs["M"] = max(errs["M"], rel(g.M_anc[i], st.M_anc))
        U, s, V = g.basis[i]
        if st.U.shape[1] == 0:
            continue
        r = U.shape[1]
        errs["orth"] = max(errs["orth"], float(np.abs(U.T @ U - np.eye(r)).max()), float(np.abs(V.T @ V - np.eye(r)).max()))
        errs["PU"] = max(errs["PU"], so.projector_distance(U, st.U))
        errs["PV"] = max(errs["PV"], so.projector_distance(V, st.V))
        errs["s"] = max(errs["s"], rel(s, st.s))
    return errs
