"""Pins for the fp64 oracle: each part is tied to something other than itself.

Hand-derived worked example, brute force, closed forms, the paper's lemmas, and
library special cases.  A dropped term, a wrong sign or index, or a transposed
operand in the oracle fails at least one of these.
"""
import numpy as np
import pytest

from conftest import read_golden
from oracle import spectral_oracle as so
from synth import generator as gen

RNG = np.random.default_rng(1234)


def rel(a, b):
    return float(np.linalg.norm(np.asarray(a) - np.asarray(b)) / max(np.linalg.norm(b), 1e-300))


# ----------------------------------------------------------------- worked example
def test_worked_2x2_example():
    g = read_golden("worked_2x2.txt")
    hp = so.Hyper(alpha=0.3, tau_p=1.0, beta_anc=0.5)
    G_anc = np.array([[6.0, 0.0], [0.0, 2.0]])
    G = np.array([[1.0, 2.0], [3.0, 4.0]])
    for r, key in ((2, "gproj_rank2"), (1, "gproj_rank1")):
        st = so.anchor_update(so.new_state(2, 2), G_anc, hp, r, mode="exact")
        assert np.allclose(st.M_anc.ravel(), g["M_anc"], atol=1e-15)
        assert np.allclose(so.filter_weights(st.s, hp.tau_p), g["d"][:r], atol=1e-15)
        P, X, gg, d = so.correct(st, G, hp)
        assert np.allclose(P.ravel(), g[key], atol=1e-14)
    # AdamW from a cold state is sign-like; weight decay is decoupled
    st = so.anchor_update(so.new_state(2, 2), G_anc, hp, 2, mode="exact")
    one = np.ones((2, 2)); z = np.zeros((2, 2))
    for wd, key in ((0.0, "w_after_nodecay"), (0.5, "w_after_decay")):
        hp2 = so.Hyper(alpha=0.3, tau_p=1.0, beta_anc=0.5, lr=0.1, eps=0.0, weight_decay=wd)
        W, m, v, _ = so.correct_and_step([st], [G], [one], [z], [z], 1, hp2)
        assert np.allclose(W[0].ravel(), g[key], atol=1e-14)


def test_adamw_one_element_hand_calc():
    g = read_golden("adamw_one_element.txt")
    W, m, v = so.adamw_step(np.array([2.0]), np.array([0.5]), np.array([0.04]), np.array([-1.0]),
                            t=3, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
    assert abs(m[0] - g["m"][0]) < 1e-15
    assert abs(v[0] - g["v"][0]) < 1e-15
    assert abs(W[0] - g["W"][0]) < 1e-14


def test_adamw_matches_torch_fp64():
    torch = pytest.importorskip("torch")
    W0 = RNG.standard_normal((7, 5)); m = np.zeros((7, 5)); v = np.zeros((7, 5))
    p = torch.nn.Parameter(torch.tensor(W0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=3e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.05)
    W = W0.copy()
    for t in range(1, 6):
        g = RNG.standard_normal((7, 5))
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        W, m, v = so.adamw_step(W, m, v, g, t, 3e-3, 0.9, 0.999, 1e-8, 0.05)
        assert rel(W, p.detach().numpy()) < 1e-13


# ----------------------------------------------------------------- SVD
@pytest.mark.parametrize("shape", [(24, 24), (40, 17), (13, 31), (64, 48)])
def test_svd_lapack_vs_bruteforce_jacobi(shape):
    A = RNG.standard_normal(shape)
    U, s, V = so.svd_exact(A)
    Uj, sj, Vj = so.svd_jacobi(A)
    assert np.allclose(s, sj, rtol=1e-11, atol=1e-12)
    assert rel((Uj * sj) @ Vj.T, A) < 1e-12
    assert rel((U * s) @ V.T, A) < 1e-12
    # same leading subspaces, compared as projectors
    for r in (1, 3, 8):
        assert so.projector_distance(U[:, :r], Uj[:, :r]) < 1e-6
        assert so.projector_distance(V[:, :r], Vj[:, :r]) < 1e-6
    assert abs(np.sum(A * A) - np.sum(s * s)) < 1e-10 * np.sum(A * A)


def test_svd_rank_one_and_diagonal_closed_forms():
    a = RNG.standard_normal(9); b = RNG.standard_normal(6)
    U, s, V = so.svd_exact(np.outer(a, b))
    assert abs(s[0] - np.linalg.norm(a) * np.linalg.norm(b)) < 1e-12
    assert np.all(s[1:] < 1e-12)
    assert abs(abs(U[:, 0] @ a) - np.linalg.norm(a)) < 1e-12
    assert abs(abs(V[:, 0] @ b) - np.linalg.norm(b)) < 1e-12
    # orientation: U spans the row index (out features), V the column index (in features)
    assert U.shape == (9, 6) and V.shape == (6, 6)
    D = np.diag([5.0, 0.5, 2.0])
    U, s, V = so.svd_exact(D)
    assert np.allclose(s, [5.0, 2.0, 0.5])
    assert np.allclose(np.abs(U[:, 1]), [0, 0, 1]) and np.allclose(np.abs(V[:, 2]), [0, 1, 0])


# ----------------------------------------------------------------- filter (Eq. 2), P_t
def _basis(m=20, n=14, r=5, tau=0.7):
    M = RNG.standard_normal((m, n))
    U, s, V = so.truncate(*so.svd_exact(M), r)
    return M, U, s, V, so.filter_weights(s, tau)


def test_filter_weights_range_and_limits():
    s = np.array([1e6, 1.0, 1e-6, 0.0])
    d = so.filter_weights(s, 1e-3)
    assert np.all(d >= 0) and np.all(d < 1)
    assert d[0] > 1 - 1e-8 and d[2] < 1e-2 and d[3] == 0
    assert np.allclose(so.filter_weights(np.array([3.0, 1.0]), 1.0), [0.75, 0.5])
    assert np.all(so.filter_weights(np.array([0.0, 0.0]), 0.0) == 0)      # before any anchor: d = 0
    # 1/tau-Lipschitz
    a, b = RNG.random(50) * 3, RNG.random(50) * 3
    assert np.all(np.abs(so.filter_weights(a, 0.2) - so.filter_weights(b, 0.2)) <= np.abs(a - b) / 0.2 + 1e-15)


def test_filter_on_basis_dyads_and_on_anchor():
    M, U, s, V, d = _basis(r=14)           # full rank so that P(M) closed form holds
    for i, j in ((0, 0), (1, 4), (3, 2)):
        dy = np.outer(U[:, i], V[:, j])
        assert rel(so.filtered_gradient(U, d, dy, V), d[i] * d[j] * dy) < 1e-12
    assert rel(so.filtered_gradient(U, d, M, V), (U * (d * d * s)) @ V.T) < 1e-12


def test_lemma1_nonexpansive_and_composition():
    M, U, s, V, d = _basis()
    for _ in range(5):
        G = RNG.standard_normal(M.shape)
        PG = so.filtered_gradient(U, d, G, V)
        assert np.linalg.norm(PG) <= np.linalg.norm(G) + 1e-12
        # P o P is the filter with weights d^2
        assert rel(so.filtered_gradient(U, d, PG, V), so.filtered_gradient(U, d * d, G, V)) < 1e-12


def test_projector_idempotent_at_tau_zero():
    M, U, s, V, _ = _basis()
    d = so.filter_weights(s, 0.0)
    assert np.all(d == 1.0)
    G = RNG.standard_normal(M.shape)
    PG = so.filtered_gradient(U, d, G, V)
    assert rel(so.filtered_gradient(U, d, PG, V), PG) < 1e-13
    assert rel(PG, U @ U.T @ G @ V @ V.T) < 1e-13
    # a transposed operand would fail here: shapes differ and U^T G V is r x r
    assert so.project(U, G, V).shape == (5, 5)


def test_lemma2_noise_contraction_monte_carlo():
    m, n, r = 30, 22, 6
    M, U, s, V, d = _basis(m, n, r, tau=0.9)
    sigma2 = 3.0
    rng = np.random.default_rng(5)
    acc = 0.0
    trials = 4000
    for _ in range(trials):
        eps = rng.standard_normal((m, n)) * np.sqrt(sigma2 / (m * n))
        acc += np.sum(so.filtered_gradient(U, d, eps, V) ** 2)
    want = sigma2 * so.effective_rank(d) ** 2 / (m * n)
    assert abs(acc / trials - want) / want < 0.05


# ----------------------------------------------------------------- blend (Eq. 3) and named limits
def test_blend_limits():
    M, U, s, V, d = _basis()
    G = RNG.standard_normal(M.shape)
    assert np.array_equal(so.corrected_gradient(U, s, V, G, 1.0, 0.7), G)
    assert rel(so.corrected_gradient(U, s, V, G, 0.0, 0.7), so.filtered_gradient(U, d, G, V)) < 1e-14
    mid = so.corrected_gradient(U, s, V, G, 0.3, 0.7)
    assert rel(mid, 0.3 * G + 0.7 * so.filtered_gradient(U, d, G, V)) < 1e-14


def test_rank_zero_is_plain_adamw_on_alpha_g():
    hp = so.Hyper(alpha=1.0, tau_p=1e-3, lr=1e-2)
    G_anc = RNG.standard_normal((6, 4)); G = RNG.standard_normal((6, 4))
    st = so.anchor_update(so.new_state(6, 4), G_anc, hp, 0, mode="exact")
    W0 = RNG.standard_normal((6, 4)); z = np.zeros((6, 4))
    W, m, v, gp = so.correct_and_step([st], [G], [W0], [z], [z], 1, hp)
    Wp, mp, vp = so.adamw_step(W0, z, z, G, 1, hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay)
    assert np.array_equal(W[0], Wp) and np.array_equal(gp[0], G)
    # alpha < 1 with rank 0: G_proj = alpha g, the same as before any anchor has arrived
    hp.alpha = 0.3
    _, _, _, gp = so.correct_and_step([st], [G], [W0], [z], [z], 1, hp)
    assert rel(gp[0], 0.3 * G) < 1e-15
    st0 = so.new_state(6, 4)
    assert rel(so.correct(st0, G, hp)[0], 0.3 * G) < 1e-15


def test_keep_one_full_rank_tau_zero_is_identity():
    spec = gen.GradSpec(m=10, n=10, tokens=40, keep=1.0, seed=3)
    G = gen.masked_gradient(spec, 1)
    assert np.array_equal(G, gen.dense_gradient(spec, 1))                 # mask all ones, /1 exact
    hp = so.Hyper(alpha=0.3, tau_p=0.0, keep=1.0)
    st = so.anchor_update(so.new_state(10, 10), gen.anchor_gradient(spec, 0), hp, 10, mode="exact")
    assert rel(so.correct(st, G, hp)[0], G) < 1e-12                       # square: P = I for any alpha
    # rectangular (m > n): V V^T = I_n but U U^T is only the rank-n projector onto range(M)
    spec = gen.GradSpec(m=12, n=9, tokens=40, keep=1.0, seed=3)
    G = gen.masked_gradient(spec, 1)
    st = so.anchor_update(so.new_state(12, 9), gen.anchor_gradient(spec, 0), hp, 9, mode="exact")
    assert rel(so.correct(st, G, hp)[0], 0.3 * G + 0.7 * st.U @ st.U.T @ G) < 1e-12


def test_rescale_inside_equals_prescaled():
    spec = gen.GradSpec(m=10, n=8, tokens=64, keep=0.25, seed=1)
    hp_a = so.Hyper(keep=0.25, grads_prescaled=True, tau_p=0.5)
    hp_b = so.Hyper(keep=0.25, grads_prescaled=False, tau_p=0.5)
    st = so.anchor_update(so.new_state(10, 8), gen.anchor_gradient(spec, 0), hp_a, 3, mode="exact")
    a = so.correct(st, gen.masked_gradient(spec, 1, rescale=True), hp_a)[0]
    b = so.correct(st, gen.masked_gradient(spec, 1, rescale=False), hp_b)[0]
    assert rel(a, b) < 1e-14


def test_closed_form_norm_and_clipping():
    M, U, s, V, d = _basis(tau=0.4)
    G = RNG.standard_normal(M.shape)
    P = so.corrected_gradient(U, s, V, G, 0.3, 0.4)
    X = so.project(U, G, V)
    cf = so.gproj_sqnorm_closed_form(float(np.sum(G * G)), X, d, 0.3)
    assert abs(cf - np.sum(P * P)) < 1e-11 * cf
    assert so.clip_factor(4.0, 0.0) == 1.0 and so.clip_factor(4.0, 5.0) == 1.0
    assert abs(so.clip_factor(4.0, 0.2) - 0.1) < 1e-15
    # global clip over two matrices
    hp = so.Hyper(alpha=0.3, tau_p=0.4, max_grad_norm=0.2)
    st = so.MatrixState(M_anc=M, U=U, s=s, V=V, have_anchor=True)
    z = np.zeros_like(M)
    _, _, _, gp = so.correct_and_step([st, st], [G, 2 * G], [z, z], [z, z], [z, z], 1, hp)
    assert abs(np.sqrt(sum(np.sum(x * x) for x in gp)) - 0.2) < 1e-12


def test_alignment_eta():
    M, U, s, V, d = _basis()
    inside = U @ RNG.standard_normal((5, 5)) @ V.T
    assert abs(so.alignment_eta(U, inside, V) - 1.0) < 1e-12
    G = RNG.standard_normal(M.shape)
    eta = so.alignment_eta(U, G, V)
    assert 0.0 < eta < 1.0
    assert abs(eta - np.linalg.norm(U @ U.T @ G @ V @ V.T) ** 2 / np.linalg.norm(G) ** 2) < 1e-12


# ----------------------------------------------------------------- Eq. 1
def test_anchor_ema_zero_init_no_bias_correction():
    hp = so.Hyper(beta_anc=0.9)
    st = so.new_state(3, 2)
    G1 = RNG.standard_normal((3, 2)); G2 = RNG.standard_normal((3, 2))
    so.anchor_update(st, G1, hp, 1)
    assert rel(st.M_anc, 0.1 * G1) < 1e-15
    so.anchor_update(st, G2, hp, 1)
    assert rel(st.M_anc, 0.09 * G1 + 0.1 * G2) < 1e-15


# ----------------------------------------------------------------- sketch + MIRROR
def test_mix64_published_vector():
    want = [int(x, 16) for x in read_golden("splitmix64.txt")]
    g = np.uint64(0x9E3779B97F4A7C15)
    with np.errstate(over="ignore"):
        got = [int(so.mix64(g * np.uint64(i))) for i in (1, 2, 3)]
    assert got == want


def test_rademacher_sketch_is_a_pure_balanced_function():
    W = so.rademacher_sketch(11, 5, 512, 64)
    assert set(np.unique(W)) == {-1.0, 1.0}
    assert abs(W.mean()) < 0.02
    assert np.array_equal(W[:100, :16], so.rademacher_sketch(11, 5, 100, 16))      # prefix-stable in n and l
    assert not np.array_equal(W, so.rademacher_sketch(11, 6, 512, 64))
    assert not np.array_equal(W, so.rademacher_sketch(12, 5, 512, 64))
    # columns are nearly orthogonal: Gram/n close to identity
    Gm = W.T @ W / 512
    assert np.max(np.abs(Gm - np.eye(64))) < 0.25


def test_mirror_equals_exact_when_rank_le_r():
    m, n, r = 60, 44, 6
    M = RNG.standard_normal((m, r)) @ RNG.standard_normal((r, n))
    Om = so.rademacher_sketch(0, 0, n, r)
    U, s, V = so.mirror_basis(M, Om, 0, r)
    Ue, se, Ve = so.truncate(*so.svd_exact(M), r)
    assert np.allclose(s, se, rtol=1e-10)
    assert so.projector_distance(U, Ue) < 1e-7 and so.projector_distance(V, Ve) < 1e-7
    G = RNG.standard_normal((m, n))
    assert rel(so.corrected_gradient(U, s, V, G, 0.3, 1.0), so.corrected_gradient(Ue, se, Ve, G, 0.3, 1.0)) < 1e-10


def test_mirror_converges_to_exact_on_gapped_input():
    m, n, r = 80, 64, 5
    A, _ = np.linalg.qr(RNG.standard_normal((m, n)))
    B, _ = np.linalg.qr(RNG.standard_normal((n, n)))
    s = np.concatenate([np.linspace(10, 6, r), np.linspace(1.0, 0.1, n - r)])
    M = (A * s) @ B.T
    G = RNG.standard_normal((m, n))
    Ue, se, Ve = so.truncate(*so.svd_exact(M), r)
    want = so.corrected_gradient(Ue, se, Ve, G, 0.3, 2.0)
    errs = []
    for q in (0, 2, 8):
        U, sv, V = so.mirror_basis(M, so.rademacher_sketch(1, 0, n, r), q, r)
        errs.append(rel(so.corrected_gradient(U, sv, V, G, 0.3, 2.0), want))
    assert errs[0] > errs[1] > errs[2] and errs[2] < 1e-8
    # oversampling: l > r with truncation also converges
    U, sv, V = so.mirror_basis(M, so.rademacher_sketch(1, 0, n, 4 * r), 4, r)
    assert rel(so.corrected_gradient(U, sv, V, G, 0.3, 2.0), want) < 1e-8


# ----------------------------------------------------------------- input generator statistics
def test_masked_gradient_unbiased_with_variance_factor():
    keep = 0.25
    base = gen.GradSpec(m=6, n=5, tokens=48, keep=keep, seed=0)
    X, dY = gen.batch(base, 3)
    dense = dY.T @ X
    # hold the batch fixed, redraw only the mask: E_m[G_mask] = dY^T X ; Var = (1-keep)/keep * sum_t dY_ti^2 X_tj^2
    rng = np.random.default_rng(9)
    acc = np.zeros_like(dense); acc2 = np.zeros_like(dense)
    trials = 6000
    for _ in range(trials):
        Mk = (rng.random(X.shape) < keep).astype(float)
        G = dY.T @ (X * Mk) / keep
        acc += G; acc2 += (G - dense) ** 2
    var_want = (1 - keep) / keep * (dY ** 2).T @ (X ** 2)
    assert np.max(np.abs(acc / trials - dense)) < 5 * np.sqrt(var_want.max() / trials)
    assert abs((acc2 / trials).sum() / var_want.sum() - 1.0) < 0.05
    # the generator's own mask has the right density and is deterministic
    Mk = gen.keep_mask(gen.GradSpec(m=6, n=500, tokens=400, keep=keep, seed=0), 3)
    assert abs(Mk.mean() - keep) < 0.01
    assert np.array_equal(gen.masked_gradient(base, 3), gen.masked_gradient(base, 3))


def test_bf16_rounding_helpers():
    torch = pytest.importorskip("torch")
    x = (RNG.standard_normal(4096) * np.exp(RNG.standard_normal(4096) * 5)).astype(np.float32)
    bits = gen.f32_to_bf16_bits(x)
    want = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    back = gen.bf16_bits_to_f64(bits)
    assert np.array_equal(back, torch.tensor(x).to(torch.bfloat16).to(torch.float64).numpy())


def test_planted_component_has_requested_snr():
    spec = gen.GradSpec(m=96, n=80, tokens=256, keep=1.0, planted_rank=4, snr=1.0, seed=2)
    Px, Py = gen.planted_directions(spec)
    assert rel(Px.T @ Px, np.eye(4)) < 1e-12 and rel(Py.T @ Py, np.eye(4)) < 1e-12
    G = gen.dense_gradient(spec, 1)
    inside = np.linalg.norm(Py.T @ G @ Px) ** 2 / np.linalg.norm(G) ** 2
    assert 0.2 < inside < 0.9       # planted energy comparable to the noise energy at SNR 1


def test_projector_distance_matches_explicit_projectors():
    A, _ = np.linalg.qr(RNG.standard_normal((40, 6)))
    for th in (1e-7, 1e-3, 0.3):
        x = RNG.standard_normal(40); x -= A @ (A.T @ x); x /= np.linalg.norm(x)
        B = A.copy(); B[:, 2] = np.cos(th) * A[:, 2] + np.sin(th) * x
        explicit = np.sin(th) / np.sqrt(6)           # ||Pa-Pb||_F = sqrt(2) sin(theta) for one rotated direction
        assert abs(so.projector_distance(A, B) - explicit) < 1e-12 + 1e-9 * explicit
        assert abs(so.projector_distance(A, B @ np.diag([1, -1, 2, 1, 1, 0.5])) - explicit) < 1e-12 + 1e-9 * explicit
    if True:
        Pa, Pb = A @ A.T, B @ B.T
        assert abs(so.projector_distance(A, B) - np.linalg.norm(Pa - Pb) / np.sqrt(12)) < 1e-12


def test_mirror_warm_start_reduces_to_cold_on_first_arrival_and_improves_later():
    m, n, r = 70, 50, 4
    A, _ = np.linalg.qr(RNG.standard_normal((m, n)))
    B, _ = np.linalg.qr(RNG.standard_normal((n, n)))
    s = np.concatenate([np.linspace(10, 7, r), np.linspace(2.0, 0.1, n - r)])
    G1 = (A * s) @ B.T
    hp = so.Hyper(beta_anc=0.5)
    Om = so.rademacher_sketch(3, 0, n, r)
    cold = so.anchor_update(so.new_state(m, n), G1, hp, r, mode="mirror", Omega=Om, q=0)
    warm = so.anchor_update(so.new_state(m, n), G1, hp, r, mode="mirror", Omega=Om, q=0, warm=True)
    assert np.array_equal(cold.V, warm.V)                              # no basis yet: same as a cold start
    Ve = so.truncate(*so.svd_exact(G1), r)[2]
    errs = []
    for _ in range(6):                                                 # same gradient again and again: M -> G1
        so.anchor_update(warm, G1, hp, r, mode="mirror", Omega=Om, q=0, warm=True)
        errs.append(so.projector_distance(warm.V, Ve))
    assert errs[-1] < 1e-2 * errs[0] and all(b <= a * 1.0001 for a, b in zip(errs, errs[1:]))


def test_prf_mask_is_a_balanced_independent_pure_function():
    keep = 0.1
    M = so.prf_keep_mask(5, 3, 17, 512, 384, keep)
    assert set(np.unique(M)) <= {0.0, 1.0}
    assert abs(M.mean() - so.keep_threshold(keep) / 65536.0) < 0.004
    assert np.array_equal(M, so.prf_keep_mask(5, 3, 17, 512, 384, keep))
    assert np.array_equal(M[:100, :37], so.prf_keep_mask(5, 3, 17, 100, 37, keep))       # prefix-stable, odd width
    for other in ((6, 3, 17), (5, 4, 17), (5, 3, 18)):
        assert abs((M * so.prf_keep_mask(*other, 512, 384, keep)).mean() - M.mean() ** 2) < 0.003   # independent draws
    # neighbours inside a pair, across pairs and across tokens are uncorrelated
    c = lambda a, b: abs(np.mean(a * b) - a.mean() * b.mean())
    assert c(M[:, 0::2], M[:, 1::2]) < 0.003 and c(M[:, :-2], M[:, 2:]) < 0.003 and c(M[:-1], M[1:]) < 0.003
    assert so.keep_threshold(1.0) == 65536 and so.prf_keep_mask(1, 0, 0, 8, 8, 1.0).all()
    assert so.keep_threshold(0.25) == 16384 and so.keep_threshold(0.5) == 32768


def test_masked_weight_gradient_is_unbiased_over_steps():
    rng = np.random.default_rng(3)
    dY = rng.standard_normal((64, 6)); X = rng.standard_normal((64, 10))
    dense = dY.T @ X
    acc = np.zeros_like(dense)
    steps = 3000
    for s in range(steps):
        acc += so.masked_weight_gradient(dY, X, so.prf_keep_mask(1, 2, s, 64, 10, 0.25), 0.25)
    var = (1 - 0.25) / 0.25 * (dY ** 2).T @ (X ** 2)                 # per-entry variance of one masked draw
    assert np.max(np.abs(acc / steps - dense) / np.sqrt(var / steps)) < 5.0
    assert np.array_equal(so.masked_weight_gradient(dY, X, np.ones_like(X), 1.0), dense)


def test_exact_k_mask_keeps_exactly_k_per_token_and_is_unbiased():
    H, T, keep = 200, 300, 0.1
    M = so.prf_exact_k_mask(4, 1, 9, T, H, keep)
    K = so.exact_k(H, keep)
    assert K == 20 and np.all(M.sum(axis=1) == K)                       # exactly K per token
    assert np.array_equal(M, so.prf_exact_k_mask(4, 1, 9, T, H, keep))
    assert not np.array_equal(M, so.prf_exact_k_mask(4, 1, 10, T, H, keep))
    # every feature is kept with probability K/H: column means over many tokens
    big = so.prf_exact_k_mask(4, 1, 9, 4000, H, keep)
    assert np.max(np.abs(big.mean(axis=0) - K / H)) < 5 * np.sqrt(0.1 * 0.9 / 4000)
    assert so.exact_k(4096, 0.05) == 205 and so.exact_k(8, 0.01) == 1 and so.exact_k(8, 1.0) == 8
    assert so.prf_exact_k_mask(1, 0, 0, 5, 8, 1.0).all()


def _golden_lines(name):
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
    return [l.split() for l in open(path) if l.strip() and not l.startswith("#")]


def test_exact_k_and_keep_threshold_at_ties_hand_computed():
    """Halves round up and the product is formed in single precision (tests/golden/rounding_ties.txt, by hand)."""
    n = 0
    for parts in _golden_lines("rounding_ties.txt"):
        if parts[0] == "exact_k":
            assert so.exact_k(int(parts[1]), float(parts[2])) == int(parts[3]), parts
        else:
            assert parts[0] == "keep_threshold"
            assert so.keep_threshold(float(parts[1])) == int(parts[2]), parts
        n += 1
    assert n == 12
    # the single-precision product is what separates 5 * 0.7 from a double-precision evaluation
    assert int(np.floor(np.float64(np.float32(0.7)) * 5 + 0.5)) == 3 and so.exact_k(5, 0.7) == 4
    # the mask built from it keeps exactly that many
    assert np.all(so.prf_exact_k_mask(1, 0, 0, 9, 8, 0.3125).sum(axis=1) == 3)


def test_prf_hash_and_masks_match_stored_vectors():
    """Regression pins written by tests/golden/make_prf_vectors.py (which imports only the oracle)."""
    lines = _golden_lines("prf_vectors.txt")
    hashes = [(int(p[1], 16), int(p[2], 16)) for p in lines if p[0] == "lowbias32"]
    assert len(hashes) == 16
    got = so.lowbias32(np.array([a for a, _ in hashes], np.uint32))
    assert [int(x) for x in got] == [b for _, b in hashes]
    args = dict(seed=0x5EED, layer=3, step=17, tokens=4, features=16)
    want = np.array([[int(c) for c in p[1]] for p in lines if p[0] == "keep_mask"], float)
    assert want.shape == (4, 16) and np.array_equal(so.prf_keep_mask(keep=0.5, **args), want)
    want = np.array([[int(c) for c in p[1]] for p in lines if p[0] == "exact_k_mask"], float)
    assert want.shape == (4, 16) and np.array_equal(so.prf_exact_k_mask(keep=0.25, **args), want)
    assert np.all(want.sum(axis=1) == 4)


# ----------------------------------------------------------------- dual-EMA step on G_proj
def test_ademamix_one_element_hand_calc():
    g = read_golden("ademamix_one_element.txt")
    W, m1, m2, v = so.ademamix_step(np.array([2.0]), np.array([0.5]), np.array([0.2]), np.array([0.04]),
                                    np.array([-1.0]), 3, 0.01, 0.9, 0.999, 0.99, 5.0, 1e-8, 0.1)
    assert abs(m1[0] - g["m1"][0]) < 1e-15 and abs(m2[0] - g["m2"][0]) < 1e-15 and abs(v[0] - g["v"][0]) < 1e-15
    assert abs(W[0] - g["W"][0]) < 1e-14


def test_ademamix_reduces_to_adamw():
    rng = np.random.default_rng(11)
    W, m, v, g = (rng.standard_normal((5, 7)) for _ in range(4))
    v = np.abs(v)
    m2 = rng.standard_normal((5, 7))
    # mix_alpha = 0: the slow EMA is carried but unused, everything else is AdamW
    Wa, ma, va = so.adamw_step(W, m, v, g, 7, 1e-2, 0.9, 0.999, 1e-8, 0.05)
    Wx, m1x, m2x, vx = so.ademamix_step(W, m, m2, v, g, 7, 1e-2, 0.9, 0.999, 0.9999, 0.0, 1e-8, 0.05)
    assert np.array_equal(Wa, Wx) and np.array_equal(ma, m1x) and np.array_equal(va, vx)
    assert np.allclose(m2x, 0.9999 * m2 + (1.0 - 0.9999) * g, rtol=1e-14, atol=0)
    # beta3 = beta1 from a zero state: m2 == m1 at every step, so the parameter change is AdamW's times
    # (1 + mix_alpha (1 - beta1^t)), without decay
    Wm, Wd = W.copy(), W.copy()
    m1 = m2 = mm = np.zeros_like(W); v1 = v2 = np.zeros_like(W)
    for t in range(1, 6):
        gt = rng.standard_normal(W.shape)
        W_new, m1, m2, v1 = so.ademamix_step(Wm, m1, m2, v1, gt, t, 1e-2, 0.9, 0.999, 0.9, 3.0, 1e-8, 0.0)
        Wd_new, mm, v2 = so.adamw_step(Wm, mm, v2, gt, t, 1e-2, 0.9, 0.999, 1e-8, 0.0)
        assert np.allclose(m1, m2, rtol=0, atol=1e-16)
        assert rel(W_new - Wm, (Wd_new - Wm) * (1.0 + 3.0 * (1.0 - 0.9 ** t))) < 1e-12
        Wm = W_new


def test_ademamix_slow_ema_fixed_point_and_memory():
    g = np.array([[0.7, -1.3]])
    m1 = m2 = v = np.zeros_like(g); W = np.zeros_like(g)
    for t in range(1, 4001):
        W, m1, m2, v = so.ademamix_step(W, m1, m2, v, g, t, 1e-3, 0.9, 0.999, 0.99, 5.0, 1e-8, 0.0)
        if t == 10:      # closed form of an EMA of a constant from zero: g (1 - beta^t)
            assert np.allclose(m2, g * (1 - 0.99 ** 10), rtol=1e-12) and np.allclose(m1, g * (1 - 0.9 ** 10), rtol=1e-12)
    assert np.allclose(m2, g, rtol=1e-12) and np.allclose(v, g * g * (1 - 0.999 ** 4000), rtol=1e-12)
    # at the fixed point one step moves theta by lr (1 + mix_alpha) sign(g) (up to eps and the bias correction of v)
    W2, *_ = so.ademamix_step(W, m1, m2, v, g, 4001, 1e-3, 0.9, 0.999, 0.99, 5.0, 0.0, 0.0)
    assert np.allclose(W2 - W, -1e-3 * 6.0 * np.sign(g), rtol=1e-6)


def test_correct_and_step_ademamix_composes_correction_and_dual_ema():
    rng = np.random.default_rng(5)
    m, n, r = 12, 9, 3
    st = so.new_state(m, n)
    hp = so.Hyper(tau_p=0.5, max_grad_norm=0.3, beta3=0.99, mix_alpha=2.0, lr=1e-2)
    so.anchor_update(st, rng.standard_normal((m, n)), hp, r, mode="exact")
    G = rng.standard_normal((m, n)); W = rng.standard_normal((m, n))
    z = np.zeros((m, n))
    Wn, a, b, vn, gp = so.correct_and_step_ademamix([st], [G], [W], [z], [z], [z], 1, hp)
    # the gradient fed to the optimizer is exactly what the AdamW form of the step feeds (same correction and clip)
    _, _, _, gp_adam = so.correct_and_step([st], [G], [W], [z], [z], 1, hp)
    assert np.array_equal(gp[0], gp_adam[0]) and abs(np.linalg.norm(gp[0]) - 0.3) < 1e-12
    W_ref, a_ref, b_ref, v_ref = so.ademamix_step(W, z, z, z, gp[0], 1, hp.lr, hp.beta1, hp.beta2, hp.beta3, hp.mix_alpha,
                                                  hp.eps, hp.weight_decay)
    assert np.array_equal(Wn[0], W_ref) and np.array_equal(b[0], b_ref)


# ----------------------------------------------------------------- low-rank compressor with error feedback
def test_gram_schmidt_against_library_qr_and_on_dependent_columns():
    rng = np.random.default_rng(21)
    P = rng.standard_normal((40, 4))
    Qn, Rn = np.linalg.qr(P)
    assert rel(so.gram_schmidt(P), Qn * np.sign(np.diag(Rn))) < 1e-12        # QR with a positive diagonal is unique
    P[:, 2] = 2.0 * P[:, 0] - P[:, 1]                                         # third column in the span of the first two
    Ph = so.gram_schmidt(P)
    assert np.all(Ph[:, 2] == 0) and abs(np.linalg.norm(Ph[:, 3]) - 1) < 1e-12
    G = Ph.T @ Ph
    assert np.allclose(G, np.diag([1, 1, 0, 1]), atol=1e-12)


def test_lowrank_compress_is_exact_on_low_rank_input_and_orthogonal_otherwise():
    rng = np.random.default_rng(22)
    m, n, rho = 30, 24, 3
    M = rng.standard_normal((m, rho)) @ rng.standard_normal((rho, n))         # rank 3
    Q0 = rng.standard_normal((n, rho))
    Ph, Q, E = so.lowrank_compress(M, None, Q0)
    assert rel(Ph @ Q.T, M) < 1e-12 and np.linalg.norm(E) < 1e-12 * np.linalg.norm(M)
    G = rng.standard_normal((m, n)); E0 = 0.1 * rng.standard_normal((m, n))
    Ph, Q, E = so.lowrank_compress(G, E0, Q0)
    assert np.allclose(Ph.T @ Ph, np.eye(rho), atol=1e-12)
    assert rel(Ph @ Q.T, Ph @ (Ph.T @ (G + E0))) < 1e-12                      # orthogonal projection of M onto range(P_hat)
    assert np.linalg.norm(Ph.T @ E) < 1e-12 * np.linalg.norm(E)               # what is left is orthogonal to what was sent
    assert abs(np.linalg.norm(G + E0) ** 2 - np.linalg.norm(Ph @ Q.T) ** 2 - np.linalg.norm(E) ** 2) < 1e-9


def test_lowrank_compress_commutes_with_the_sum_over_workers():
    rng = np.random.default_rng(23)
    m, n, rho = 20, 16, 2
    Gs = [rng.standard_normal((m, n)) for _ in range(3)]
    Q0 = rng.standard_normal((n, rho))
    Ph, Q, _ = so.lowrank_compress(sum(Gs), None, Q0)
    P_sum = sum(G @ Q0 for G in Gs)                                            # each worker's P, summed
    Ph2 = so.gram_schmidt(P_sum)
    Q_sum = sum(G.T @ Ph2 for G in Gs)                                         # each worker's Q, summed
    assert rel(Ph2, Ph) < 1e-12 and rel(Q_sum, Q) < 1e-12


def test_lowrank_error_feedback_telescopes_and_repetition_reaches_the_truncated_svd():
    rng = np.random.default_rng(24)
    m, n, rho = 25, 18, 2
    E = np.zeros((m, n)); Q = rng.standard_normal((n, rho))
    sent, given = np.zeros((m, n)), np.zeros((m, n))
    for t in range(6):
        G = rng.standard_normal((m, n))
        Ph, Q, E = so.lowrank_compress(G, E, Q)
        sent += Ph @ Q.T; given += G
    assert rel(sent + E, given) < 1e-12                                        # nothing is lost, only delayed
    M = rng.standard_normal((m, n)) * np.logspace(0, -2, n)[None, :]
    Q = rng.standard_normal((n, rho))
    for _ in range(200):                                                       # same matrix again and again, no feedback
        Ph, Q, Err = so.lowrank_compress(M, None, Q)
    s = np.linalg.svd(M, compute_uv=False)
    assert abs(np.linalg.norm(Err) - np.sqrt(np.sum(s[rho:] ** 2))) < 1e-8 * np.linalg.norm(M)


# ----------------------------------------------------------------- full-spectrum soft filter (no rank cut)
def test_full_spectrum_filter_is_the_rank_min_mn_basis_form():
    rng = np.random.default_rng(31)
    for m, n in ((9, 14), (14, 9), (11, 11)):
        M = rng.standard_normal((m, n)); G = rng.standard_normal((m, n)); tau = 0.7
        U, s, V = so.svd_exact(M)
        want = so.filtered_gradient(U, so.filter_weights(s, tau), G, V)            # r = min(m, n)
        assert rel(so.full_spectrum_filtered(M, G, tau), want) < 1e-12
        PU, PV = so.full_spectrum_projectors(M, tau)
        assert np.allclose(PU, PU.T, atol=1e-13) and np.allclose(PV, PV.T, atol=1e-13)
        ev = np.linalg.eigvalsh(PU)
        assert ev.min() > -1e-12 and ev.max() < 1.0                                 # 0 <= d < 1
        assert rel(PU @ M, M @ PV) < 1e-12                                          # both equal U diag(d s) V^T
        assert rel(PU @ M, (U * (s * so.filter_weights(s, tau))) @ V.T) < 1e-12
        hp = so.Hyper(alpha=0.3, tau_p=tau)
        assert rel(so.correct_full_spectrum(M, G, hp), 0.3 * G + 0.7 * want) < 1e-12
    # diagonal momentum: P_U = P_V = diag(s / (s + tau)), elementwise closed form
    sv = np.array([3.0, 1.0, 0.25, 0.0])
    G = rng.standard_normal((4, 4))
    d = sv / (sv + 0.5)
    assert rel(so.full_spectrum_filtered(np.diag(sv), G, 0.5), d[:, None] * G * d[None, :]) < 1e-13


def test_product_only_iteration_converges_to_the_soft_projector():
    rng = np.random.default_rng(32)
    m, n, tau = 24, 40, 1.5
    M = rng.standard_normal((m, n)) @ np.diag(np.logspace(0, -1.5, n))
    PU, PV = so.full_spectrum_projectors(M, tau)
    errs = [rel(so.soft_projector_iterative(M @ M.T, tau, q, 30), PU) for q in (2, 4, 8, 16)]
    assert all(b < a for a, b in zip(errs, errs[1:])) and errs[-1] < 1e-12, errs
    errs = [rel(so.soft_projector_iterative(M.T @ M, tau, 20, q), PV) for q in (2, 4, 8, 16)]       # n > m: singular Gram
    assert all(b < a for a, b in zip(errs, errs[1:])) and errs[-1] < 1e-9, errs
    G = rng.standard_normal((m, n))
    assert rel(so.full_spectrum_filtered_iterative(M, G, tau, 20, 16), so.full_spectrum_filtered(M, G, tau)) < 1e-9
    # a direction that has not converged yet is under-weighted, never over-weighted
    few = so.soft_projector_iterative(M @ M.T, tau, 6, 30)
    assert np.all(np.linalg.eigvalsh(few) <= np.linalg.eigvalsh(PU) + 1e-9)
    assert np.array_equal(so.soft_projector_iterative(np.zeros((5, 5)), tau, 10, 10), np.zeros((5, 5)))
