"""fp64 CPU oracle for the spectral-correction optimizer step.

THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no
code with the CUDA path and never imports it.

Every function is the plain definition of one step of the method (Section 3.2
"Anchor Priors and Spectral Correction", Eq. 1-3, Algorithm 1 lines 7-14 and
the operator P_t of the convergence appendix), written in NumPy fp64 with no
blocking, fusion or reordering.  A library routine (LAPACK SVD / QR / matmul)
is used as a step where the paper just says "SVD".

Two basis modes exist because the paper only says "SVD" while the GPU path
uses a randomized subspace iteration:

* EXACT  - full thin SVD of the anchor momentum, keep the leading r triplets
           (the operator D_t = diag(d_1..d_r) of the appendix).
* MIRROR - the documented randomized range finder written out in fp64:
           Q = orth(M W); q x { Z = orth(M^T Q); Q = orth(M Z) };
           B = Q^T M; thin SVD of B; U = Q U_B[:, :r], V = V_B[:, :r].
           In exact arithmetic it depends only on (M, W, q, r), not on how
           orth() is realised.

Pins (tests/test_oracle_pins.py): hand-derived 2x2 worked example, brute-force
one-sided Jacobi SVD, rank-1 / diagonal closed forms, Lemma 1 and Lemma 2,
idempotence at tau_p = 0, the alpha / rank / keep limit cases, torch AdamW in
fp64, the closed-form global norm, MIRROR == EXACT for rank(M) <= r; the dual-EMA
step by a one-element hand calculation, its mix_alpha = 0 and beta3 = beta1 special
cases (both reduce to adamw_step) and the fixed point of the slow EMA; the low-rank
compressor by exact recovery of rank <= rho inputs, orthogonality of the error to
the transmitted range, linearity over workers, the telescoping identity of error
feedback and convergence to the truncated SVD (Eckart-Young) under repetition;
the full-spectrum filter by its equality with the rank-min(m,n) basis form, closed
forms on diagonal input, and the product-only iteration by convergence to it.
Parity unpinned: end-to-end MIRROR vs EXACT on inputs with no spectral gap at r
(the cut is ill-posed there; it is reported, not gated).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Eq. 1 / Algorithm 1 line 8: anchor momentum
# --------------------------------------------------------------------------
def anchor_ema(M_anc: np.ndarray, G_anc: np.ndarray, beta_anc: float) -> np.ndarray:
    """M <- beta_anc * M + (1 - beta_anc) * G_anc  (Eq. 1; zero init, no bias correction)."""
    return beta_anc * np.asarray(M_anc, F64) + (1.0 - beta_anc) * np.asarray(G_anc, F64)


# --------------------------------------------------------------------------
# "M = U S V^T" (Section 3.2, "From momentum to a denoising operator")
# --------------------------------------------------------------------------
def svd_exact(M: np.ndarray):
    """Thin SVD through LAPACK, singular values descending.  Returns (U, s, V) with M = U diag(s) V^T."""
    U, s, Vt = np.linalg.svd(np.asarray(M, F64), full_matrices=False)
    return U, s, Vt.T


def svd_jacobi(M: np.ndarray, sweeps: int = 60, tol: float = 1e-15):
    """Brute-force one-sided (Hestenes) Jacobi SVD, pure loops; for tiny matrices only.

    Used to pin svd_exact to something that is not LAPACK.  Returns (U, s, V)
    sorted by descending s.  Columns of U belonging to zero singular values are
    left as zero vectors (callers compare only the non-null part).
    """
    A = np.array(M, F64)
    transposed = A.shape[0] < A.shape[1]
    if transposed:
        A = A.T.copy()
    m, n = A.shape
    V = np.eye(n)
    for _ in range(sweeps):
        off = 0.0
        for p in range(n - 1):
            for q in range(p + 1, n):
                a = A[:, p] @ A[:, p]
                b = A[:, q] @ A[:, q]
                c = A[:, p] @ A[:, q]
                if abs(c) <= tol * np.sqrt(a * b) or c == 0.0:
                    continue
                off = max(off, abs(c) / np.sqrt(a * b))
                zeta = (b - a) / (2.0 * c)
                t = np.sign(zeta) / (abs(zeta) + np.sqrt(1.0 + zeta * zeta)) if zeta != 0 else 1.0
                cs = 1.0 / np.sqrt(1.0 + t * t)
                sn = cs * t
                Ap = A[:, p].copy()
                A[:, p] = cs * Ap - sn * A[:, q]
                A[:, q] = sn * Ap + cs * A[:, q]
                Vp = V[:, p].copy()
                V[:, p] = cs * Vp - sn * V[:, q]
                V[:, q] = sn * Vp + cs * V[:, q]
        if off <= tol:
            break
    s = np.sqrt(np.sum(A * A, axis=0))
    order = np.argsort(-s)
    s = s[order]
    A = A[:, order]
    V = V[:, order]
    U = np.zeros_like(A)
    nz = s > 0
    U[:, nz] = A[:, nz] / s[nz]
    if transposed:
        U, V = V, U
    return U, s, V


def truncate(U, s, V, r: int):
    """Keep the leading r singular triplets (D_t = diag(d_1..d_r)); r = 0 gives an empty basis."""
    r = int(r)
    return U[:, :r], s[:r], V[:, :r]


# --------------------------------------------------------------------------
# Eq. 2: soft spectral filter
# --------------------------------------------------------------------------
def filter_weights(s: np.ndarray, tau_p: float) -> np.ndarray:
    """d_i = s_i / (s_i + tau_p)  (Eq. 2).  0/0 (s_i = tau_p = 0) is taken as 0: an unsupported direction."""
    s = np.asarray(s, F64)
    den = s + tau_p
    out = np.zeros_like(s)
    np.divide(s, den, out=out, where=den > 0)
    return out


# --------------------------------------------------------------------------
# "Two-sided application"
# --------------------------------------------------------------------------
def project(U, G, V):
    """X = U^T G V."""
    return U.T @ np.asarray(G, F64) @ V


def filtered_gradient(U, d, G, V):
    """G_filt = U diag(d) (U^T G V) diag(d) V^T  ==  P_t(G)."""
    X = project(U, G, V)
    X_filt = (d[:, None] * X) * d[None, :]
    return U @ X_filt @ V.T


def blend(G, G_filt, alpha: float):
    """G_proj = alpha G + (1 - alpha) G_filt  (Eq. 3)."""
    return alpha * np.asarray(G, F64) + (1.0 - alpha) * G_filt


def corrected_gradient(U, s, V, G, alpha: float, tau_p: float, scale: float = 1.0):
    """Eq. 2 + two-sided filter + Eq. 3 on g = scale * G (scale = 1/keep for un-rescaled inputs)."""
    g = scale * np.asarray(G, F64)
    d = filter_weights(s, tau_p)
    return blend(g, filtered_gradient(U, d, g, V), alpha)


# --------------------------------------------------------------------------
# Diagnostics that the appendix defines
# --------------------------------------------------------------------------
def alignment_eta(U, G, V) -> float:
    """eta_r = ||U^T g V||_F^2 / ||g||_F^2 (Alignment Trajectory appendix)."""
    G = np.asarray(G, F64)
    den = float(np.sum(G * G))
    return float(np.sum(project(U, G, V) ** 2) / den) if den > 0 else 0.0


def effective_rank(d) -> float:
    """r_eff = ||D_t||_F^2 = sum_i d_i^2  (Lemma 2)."""
    d = np.asarray(d, F64)
    return float(np.sum(d * d))


def gproj_sqnorm_closed_form(g_sqnorm: float, X, d, alpha: float) -> float:
    """||G_proj||_F^2 from ||g||^2 and X = U^T g V only.

    <g, U A V^T> = <U^T g V, A> and ||U A V^T||_F = ||A||_F for orthonormal U, V,
    so with A = D X D:  ||alpha g + (1-alpha) U A V^T||^2
      = alpha^2 ||g||^2 + 2 alpha (1-alpha) sum d_i d_j X_ij^2 + (1-alpha)^2 sum d_i^2 d_j^2 X_ij^2.
    """
    X = np.asarray(X, F64)
    dd = np.outer(d, d)
    return float(alpha * alpha * g_sqnorm
                 + 2.0 * alpha * (1.0 - alpha) * np.sum(dd * X * X)
                 + (1.0 - alpha) ** 2 * np.sum(dd * dd * X * X))


def clip_factor(total_sqnorm: float, max_norm: float) -> float:
    """Global-norm clipping factor min(1, c_max / ||G_proj||) over all matrices; max_norm <= 0 switches it off."""
    if max_norm is None or max_norm <= 0.0:
        return 1.0
    nrm = float(np.sqrt(total_sqnorm))
    return 1.0 if nrm <= max_norm else max_norm / nrm


# --------------------------------------------------------------------------
# Algorithm 1 line 13: AdamW with G_proj
# --------------------------------------------------------------------------
def adamw_step(W, m, v, g, t: int, lr: float, beta1: float, beta2: float, eps: float, weight_decay: float):
    """One decoupled-weight-decay Adam step, step count t >= 1.

    m <- b1 m + (1-b1) g ; v <- b2 v + (1-b2) g^2 ;
    W <- W - lr*wd*W - lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps).
    Returns new (W, m, v).
    """
    W = np.asarray(W, F64)
    g = np.asarray(g, F64)
    m = beta1 * np.asarray(m, F64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, F64) + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** t)
    v_hat = v / (1.0 - beta2 ** t)
    W = W - lr * weight_decay * W - lr * m_hat / (np.sqrt(v_hat) + eps)
    return W, m, v


def ademamix_step(W, m1, m2, v, g, t: int, lr: float, beta1: float, beta2: float, beta3: float, mix_alpha: float,
                  eps: float, weight_decay: float):
    """One dual-EMA (AdEMAMix) step on the corrected gradient (appendix "On the Compatibility with Dual-EMA
    Optimizers": the composition applies the dual-EMA dynamics to G_proj instead of the raw masked gradient).

    fast EMA  m1 <- b1 m1 + (1-b1) g   (bias-corrected in the update, as Adam's first moment)
    slow EMA  m2 <- b3 m2 + (1-b3) g   (b3 close to 1, no bias correction)
    second    v  <- b2 v  + (1-b2) g^2 (bias-corrected)
    theta <- theta - lr*wd*theta - lr * (m1/(1-b1^t) + mix_alpha * m2) / (sqrt(v/(1-b2^t)) + eps).
    The appendix prints the update without a decay term; decay is decoupled here exactly as in adamw_step, so
    that mix_alpha = 0 is that function.  Returns new (W, m1, m2, v).
    """
    W = np.asarray(W, F64)
    g = np.asarray(g, F64)
    m1 = beta1 * np.asarray(m1, F64) + (1.0 - beta1) * g
    m2 = beta3 * np.asarray(m2, F64) + (1.0 - beta3) * g
    v = beta2 * np.asarray(v, F64) + (1.0 - beta2) * g * g
    m1_hat = m1 / (1.0 - beta1 ** t)
    v_hat = v / (1.0 - beta2 ** t)
    W = W - lr * weight_decay * W - lr * (m1_hat + mix_alpha * m2) / (np.sqrt(v_hat) + eps)
    return W, m1, m2, v


# --------------------------------------------------------------------------
# Randomized range finder (MIRROR mode)
# --------------------------------------------------------------------------
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_MIX1 = np.uint64(0xBF58476D1CE4E5B9)
_MIX2 = np.uint64(0x94D049BB133111EB)


def mix64(x: np.ndarray) -> np.ndarray:
    """The 64-bit finaliser of the SplitMix64 generator (wrap-around uint64 arithmetic)."""
    x = np.asarray(x, np.uint64)
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * _MIX1
        x = (x ^ (x >> np.uint64(27))) * _MIX2
        x = x ^ (x >> np.uint64(31))
    return x


def rademacher_sketch(seed: int, mat_id: int, n: int, l: int) -> np.ndarray:
    """Sketch matrix W in {-1,+1}^{n x l}, a pure function of (seed, mat_id, row j, column c).

    counter = mat_id * 2^44 + j * 2^10 + c ; h = mix64(seed XOR (counter + 1) * golden) ;
    W[j, c] = +1 if the top bit of h is 0 else -1.
    """
    j = np.arange(n, dtype=np.uint64)[:, None]
    c = np.arange(l, dtype=np.uint64)[None, :]
    with np.errstate(over="ignore"):
        counter = np.uint64(mat_id) * np.uint64(1 << 44) + j * np.uint64(1 << 10) + c
        h = mix64(np.uint64(seed) ^ ((counter + np.uint64(1)) * _GOLDEN))
    return np.where((h >> np.uint64(63)) == 0, 1.0, -1.0).astype(F64)


def _orth(Y):
    """Orthonormal basis of range(Y) by Householder QR."""
    Q, _ = np.linalg.qr(Y)
    return Q


def mirror_basis(M, Omega, q: int, r: int):
    """Rank-r basis by randomized subspace iteration with sketch Omega (n x l), q power iterations."""
    M = np.asarray(M, F64)
    if r == 0:
        return np.zeros((M.shape[0], 0)), np.zeros(0), np.zeros((M.shape[1], 0))
    Q = _orth(M @ Omega)
    for _ in range(int(q)):
        Z = _orth(M.T @ Q)
        Q = _orth(M @ Z)
    B = Q.T @ M
    Ub, s, Vbt = np.linalg.svd(B, full_matrices=False)
    U = Q @ Ub
    return U[:, :r], s[:r], Vbt.T[:, :r]


def projector_distance(Ua, Ub) -> float:
    """||Pa - Pb||_F / sqrt(2 r) for the orthogonal projectors onto span(Ua), span(Ub) (sign/rotation free).

    For equal ranks ||Pa - Pb||_F^2 = 2 ||(I - Pa) Qb||_F^2 with Qb an orthonormal basis of span(Ub); the
    residual form is used because 2r - 2||Ua^T Ub||_F^2 cancels catastrophically (it cannot resolve
    distances below ~sqrt(machine eps of the inputs)).  Inputs are re-orthonormalised first, so
    a slightly non-unit column norm of an fp32 basis does not register as a subspace error.
    """
    ra, rb = Ua.shape[1], Ub.shape[1]
    if ra == 0 and rb == 0:
        return 0.0
    if ra != rb:
        return 1.0
    Qa, _ = np.linalg.qr(np.asarray(Ua, F64))
    Qb, _ = np.linalg.qr(np.asarray(Ub, F64))
    res = Qb - Qa @ (Qa.T @ Qb)
    return float(np.linalg.norm(res) / np.sqrt(ra))


# --------------------------------------------------------------------------
# Whole step for one matrix, and a small state holder (Algorithm 1 lines 7-14)
# --------------------------------------------------------------------------
@dataclass
class Hyper:
    alpha: float = 0.3
    tau_p: float = 1e-3
    beta_anc: float = 0.9
    lr: float = 2e-5
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    max_grad_norm: float = 0.0      # 0 = no clipping
    grads_prescaled: bool = True    # False: the step multiplies the masked gradient by 1/keep
    keep: float = 1.0
    beta3: float = 0.9999           # slow EMA of the dual-EMA composition
    mix_alpha: float = 5.0          # weight of the slow EMA in the update


@dataclass
class MatrixState:
    """Per-matrix oracle state: anchor momentum, cached basis, AdamW moments."""
    M_anc: np.ndarray
    U: np.ndarray = None
    s: np.ndarray = None
    V: np.ndarray = None
    have_anchor: bool = False
    extra: dict = field(default_factory=dict)


def new_state(m: int, n: int) -> MatrixState:
    return MatrixState(M_anc=np.zeros((m, n), F64), U=np.zeros((m, 0)), s=np.zeros(0), V=np.zeros((n, 0)))


def anchor_update(state: MatrixState, G_anc, hp: Hyper, r: int, mode: str = "exact",
                  Omega=None, q: int = 1, warm: bool = False, q_warm: int = 0) -> MatrixState:
    """Anchor arrival: Eq. 1 then the rank-r basis of the new momentum (cached until the next arrival).

    mirror mode with warm=True: a matrix that already has a basis starts the range finder from
    [previous V | sketch columns r..l-1] instead of the sketch and runs q_warm power iterations.
    """
    state.M_anc = anchor_ema(state.M_anc, G_anc, hp.beta_anc)
    if mode == "exact":
        state.U, state.s, state.V = truncate(*svd_exact(state.M_anc), r)
    elif mode == "mirror":
        if warm and state.have_anchor and r > 0:
            start = np.concatenate([state.V[:, :r], Omega[:, r:]], axis=1)
            state.U, state.s, state.V = mirror_basis(state.M_anc, start, q_warm, r)
        else:
            state.U, state.s, state.V = mirror_basis(state.M_anc, Omega, q, r)
    else:
        raise ValueError(mode)
    state.have_anchor = True
    return state


def correct(state: MatrixState, G_mask, hp: Hyper):
    """G_proj for one matrix (before optional clipping).  Also returns X and ||g||^2 for the closed-form norm."""
    scale = 1.0 if hp.grads_prescaled else 1.0 / hp.keep
    g = scale * np.asarray(G_mask, F64)
    d = filter_weights(state.s, hp.tau_p)
    X = project(state.U, g, state.V)
    G_proj = blend(g, state.U @ ((d[:, None] * X) * d[None, :]) @ state.V.T, hp.alpha)
    return G_proj, X, float(np.sum(g * g)), d


def correct_and_step(states, G_masks, Ws, ms, vs, t: int, hp: Hyper):
    """One fast-circuit step over a list of matrices: correction, optional global clip, AdamW.

    Returns (new Ws, new ms, new vs, list of G_proj after clipping).
    """
    projs = [correct(st, G, hp)[0] for st, G in zip(states, G_masks)]
    total = sum(float(np.sum(P * P)) for P in projs)
    c = clip_factor(total, hp.max_grad_norm)
    outW, outm, outv, outg = [], [], [], []
    for P, W, m, v in zip(projs, Ws, ms, vs):
        g = c * P
        W2, m2, v2 = adamw_step(W, m, v, g, t, hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay)
        outW.append(W2); outm.append(m2); outv.append(v2); outg.append(g)
    return outW, outm, outv, outg


def correct_and_step_ademamix(states, G_masks, Ws, m1s, m2s, vs, t: int, hp: Hyper):
    """The same fast-circuit step with the dual-EMA optimizer in place of AdamW: correction, optional global clip,
    then ademamix_step on G_proj.  Returns (new Ws, new m1s, new m2s, new vs, list of G_proj after clipping)."""
    projs = [correct(st, G, hp)[0] for st, G in zip(states, G_masks)]
    total = sum(float(np.sum(P * P)) for P in projs)
    c = clip_factor(total, hp.max_grad_norm)
    outW, out1, out2, outv, outg = [], [], [], [], []
    for P, W, m1, m2, v in zip(projs, Ws, m1s, m2s, vs):
        g = c * P
        W2, a, b, v2 = ademamix_step(W, m1, m2, v, g, t, hp.lr, hp.beta1, hp.beta2, hp.beta3, hp.mix_alpha, hp.eps,
                                     hp.weight_decay)
        outW.append(W2); out1.append(a); out2.append(b); outv.append(v2); outg.append(g)
    return outW, out1, out2, outv, outg


# --------------------------------------------------------------------------
# In-graph activation mask from a shared pseudo-random function (Section 3.1, Algorithm 1 line 4:
# M_l = g(l, t, B, S, H)) and the masked weight gradient it leads to.  Nothing here is part of the
# optimizer step; it is the producer of the step's input, kept beside it for the fused GPU producer.
# --------------------------------------------------------------------------
def lowbias32(x: np.ndarray) -> np.ndarray:
    """A 32-bit integer finaliser (xorshift-multiply, two rounds), wrap-around uint32 arithmetic."""
    x = np.asarray(x, np.uint32).copy()
    with np.errstate(over="ignore"):
        x ^= x >> np.uint32(16)
        x *= np.uint32(0x21F0AAAD)
        x ^= x >> np.uint32(15)
        x *= np.uint32(0x735A2D97)
        x ^= x >> np.uint32(15)
    return x


def keep_threshold(keep: float) -> int:
    """keep ratio quantised to 16 bits: an element is kept iff its 16 random bits are below this."""
    x = np.float32(keep) * np.float32(65536.0)           # the keep ratio crosses the C ABI as a float
    return int(min(65536, max(1, int(np.floor(np.float64(x) + 0.5)))))


def prf_keep_mask(seed: int, layer: int, step: int, tokens: int, features: int, keep: float) -> np.ndarray:
    """Mask in {0,1}^{tokens x features}: a pure function of (seed, layer, step, token, feature).

    row key   k_t = low 32 bits of mix64(seed XOR ((layer * 2^40 + step) * golden) XOR (t + 1) * 0xD1B54A32D192ED03)
    pair hash h   = lowbias32(k_t + (j // 2) * 0x9E3779B9)
    bits          = low 16 bits of h for even j, high 16 bits for odd j;  kept iff bits < keep_threshold(keep)
    """
    t = np.arange(tokens, dtype=np.uint64)
    with np.errstate(over="ignore"):
        base = np.uint64(seed) ^ ((np.uint64(layer) * np.uint64(1 << 40) + np.uint64(step)) * _GOLDEN)
        key = mix64(base ^ ((t + np.uint64(1)) * np.uint64(0xD1B54A32D192ED03)))
    k32 = (key & np.uint64(0xFFFFFFFF)).astype(np.uint32)[:, None]
    pairs = (np.arange((features + 1) // 2, dtype=np.uint64) * np.uint64(0x9E3779B9) & np.uint64(0xFFFFFFFF)).astype(np.uint32)[None, :]
    with np.errstate(over="ignore"):
        h = lowbias32(k32 + pairs)
    bits = np.empty((tokens, 2 * h.shape[1]), np.uint32)
    bits[:, 0::2] = h & np.uint32(0xFFFF)
    bits[:, 1::2] = h >> np.uint32(16)
    return (bits[:, :features] < np.uint32(keep_threshold(keep))).astype(F64)


def masked_weight_gradient(dY, X, mask, keep: float, rescale: bool = True) -> np.ndarray:
    """G_mask = dY^T (X * mask) / keep_q, keep_q the 16-bit quantised keep ratio (so that E_mask[G_mask] = dY^T X)."""
    G = np.asarray(dY, F64).T @ (np.asarray(X, F64) * mask)
    return G * (65536.0 / keep_threshold(keep)) if rescale else G


def prf_exact_k_mask(seed: int, layer: int, step: int, tokens: int, features: int, keep: float) -> np.ndarray:
    """The per-token variant of the shared-PRF mask (Section 3.1, K = round(keep * H) features kept per token):
    every token keeps exactly K features, those with the K smallest composite keys
        key(t, j) = lowbias32(k_t + j * 0x9E3779B9) * 2^16 + j        (k_t as in prf_keep_mask; j < 65536),
    which are distinct by construction, so the selection is unique.
    """
    K = exact_k(features, keep)
    t = np.arange(tokens, dtype=np.uint64)
    with np.errstate(over="ignore"):
        base = np.uint64(seed) ^ ((np.uint64(layer) * np.uint64(1 << 40) + np.uint64(step)) * _GOLDEN)
        key = mix64(base ^ ((t + np.uint64(1)) * np.uint64(0xD1B54A32D192ED03)))
    k32 = (key & np.uint64(0xFFFFFFFF)).astype(np.uint32)[:, None]
    j = np.arange(features, dtype=np.uint64)
    jm = ((j * np.uint64(0x9E3779B9)) & np.uint64(0xFFFFFFFF)).astype(np.uint32)[None, :]
    with np.errstate(over="ignore"):
        h = lowbias32(k32 + jm)
    comp = (h.astype(np.uint64) << np.uint64(16)) | j[None, :]
    kth = np.partition(comp, K - 1, axis=1)[:, K - 1:K]
    return (comp <= kth).astype(F64)


def exact_k(features: int, keep: float) -> int:
    """K = round(keep * H) (halves round up; the product is formed in fp32 as the C ABI does), at least 1, at most H."""
    x = np.float32(keep) * np.float32(features)
    return int(min(features, max(1, int(np.floor(np.float64(x) + 0.5)))))


# --------------------------------------------------------------------------
# Full-spectrum soft filter: the main-text form of Section 3.2 ("Filtering d_i = s_i / (s_i + tau_p)"), where the
# soft weights apply to ALL singular directions of the anchor momentum and there is no rank cut.  With
# M = U S V^T (thin, all min(m, n) directions):
#     P_U = U diag(d) U^T = A (A + tau I)^-1,  A = (M M^T)^(1/2)        (m x m)
#     P_V = V diag(d) V^T = B (B + tau I)^-1,  B = (M^T M)^(1/2)        (n x n)
#     G_filt = P_U G P_V
# which is filtered_gradient() with r = min(m, n), written without an explicit basis.
# --------------------------------------------------------------------------
def full_spectrum_projectors(M, tau_p: float):
    """(P_U, P_V) by the plain definition: full thin SVD, Eq. 2 on every singular value."""
    U, s, V = svd_exact(M)
    d = filter_weights(s, tau_p)
    return (U * d) @ U.T, (V * d) @ V.T


def full_spectrum_filtered(M, G, tau_p: float):
    """G_filt = P_U G P_V."""
    PU, PV = full_spectrum_projectors(M, tau_p)
    return PU @ np.asarray(G, F64) @ PV


def soft_projector_iterative(A, tau_p: float, n_sqrt: int, n_inv: int):
    """f(A) = A^(1/2) (A^(1/2) + tau I)^-1 for a symmetric positive semi-definite A (a Gram matrix of the anchor
    momentum) by products only - the iteration the GPU path runs, restated in fp64 step by step:

      square root (coupled Newton-Schulz):  Y_0 = A / c, Z_0 = I, c = ||A||_F (an upper bound of the largest eigenvalue)
                                            T = (3 I - Z Y) / 2 ;  Y <- Y T ;  Z <- T Z          (n_sqrt times)
                                            S = sqrt(c) Y   ->  A^(1/2)
      inverse (Newton-Schulz):              B = S + tau I, X_0 = I / (||S||_F + tau)
                                            X <- X (2 I - B X)                                   (n_inv times)
      result                                I - tau X       ->  S (S + tau I)^-1

    An eigenvalue lam of A moves as p <- p (3 - p)^2 / 4 from p_0 = lam / c, y = sqrt(lam p / c): directions far
    below the threshold converge last and are UNDER-estimated until then (y < sqrt(lam / c)), which only pushes their
    filter weight further towards 0.  On the null space of A the companion iterate Z grows by 3/2 per
    iteration and drags rounding noise with it, so n_sqrt is a few dozen, not hundreds (fp64: the result is
    good to 1e-9 at 40 iterations on a singular Gram matrix and breaks down past about 70).  tau_p must be
    positive (for tau_p = 0 the operator is a projector and B is singular)."""
    A = np.asarray(A, F64)
    k = A.shape[0]
    I = np.eye(k)
    c = np.linalg.norm(A)
    if c == 0.0:
        return np.zeros_like(A)
    Y, Z = A / c, I.copy()
    for _ in range(int(n_sqrt)):
        T = 1.5 * I - 0.5 * (Z @ Y)
        Y, Z = Y @ T, T @ Z
    S = np.sqrt(c) * Y
    B = S + tau_p * I
    X = I / (np.linalg.norm(S) + tau_p)
    for _ in range(int(n_inv)):
        X = X @ (2.0 * I - B @ X)
    return I - tau_p * X


def full_spectrum_filtered_iterative(M, G, tau_p: float, n_sqrt: int, n_inv: int):
    """G_filt with both soft projectors from soft_projector_iterative (mirror of the GPU path)."""
    M = np.asarray(M, F64)
    PU = soft_projector_iterative(M @ M.T, tau_p, n_sqrt, n_inv)
    PV = soft_projector_iterative(M.T @ M, tau_p, n_sqrt, n_inv)
    return PU @ np.asarray(G, F64) @ PV


def correct_full_spectrum(M_anc, G_mask, hp: Hyper):
    """G_proj (Eq. 3) with the full-spectrum filter, before clipping."""
    scale = 1.0 if hp.grads_prescaled else 1.0 / hp.keep
    g = scale * np.asarray(G_mask, F64)
    return blend(g, full_spectrum_filtered(M_anc, g, hp.tau_p), hp.alpha)


# --------------------------------------------------------------------------
# Low-rank gradient compressor with error feedback (DP-compression appendix, "Low-rank factorization (F3)":
# rank-1..4 factors from one subspace-iteration step per gradient, a linear map so that it commutes with the
# sum over workers, error feedback for what the factors miss).  Plain definition, one matrix:
#     M = G + E                       gradient plus the error memory
#     P = M Q_prev                    (sum over workers here)
#     P_hat = orthonormalise(P)       Gram-Schmidt, column by column
#     Q = M^T P_hat                   (sum over workers here)
#     G_hat = P_hat Q^T ;  E <- M - G_hat
# Q is carried to the next step as the start of its subspace iteration.
# --------------------------------------------------------------------------
def gram_schmidt(P, drop_tol: float = 1e-3) -> np.ndarray:
    """Columns of P orthonormalised in order (modified Gram-Schmidt, fp64).  A column whose remainder is below
    drop_tol times its original norm lies in the span of the earlier ones and is dropped (left as zeros); the
    default is the level at which a single-precision implementation can still tell the remainder from rounding."""
    P = np.array(P, F64)
    out = np.zeros_like(P)
    for k in range(P.shape[1]):
        v = P[:, k].copy()
        n0 = np.linalg.norm(v)
        for j in range(k):
            v -= (out[:, j] @ v) * out[:, j]
        nv = np.linalg.norm(v)
        if n0 > 0.0 and nv > drop_tol * n0:
            out[:, k] = v / nv
    return out


def lowrank_compress(G, E, Q_prev):
    """One compression step.  Returns (P_hat m x rho, Q n x rho, E_new m x n); the transmitted approximation is
    P_hat Q^T.  E may be None (no error feedback: the error is returned but nothing was added to G)."""
    M = np.asarray(G, F64) + (0.0 if E is None else np.asarray(E, F64))
    P_hat = gram_schmidt(M @ np.asarray(Q_prev, F64))
    Q = M.T @ P_hat
    return P_hat, Q, M - P_hat @ Q.T
