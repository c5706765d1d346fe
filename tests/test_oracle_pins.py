"""Pins for the CPU oracle: every check here is against something the paper or
the mathematics fixes (closed forms, LAPACK's SVD, hand-derived small cases,
brute-force expansion, symmetries), never against the oracle itself."""

import math

import numpy as np
import pytest

from oracle import muon_oracle as orc

A_, B_, C_ = 3.4445, -4.7750, 2.0315


def f_scalar(x):
    return A_ * x + B_ * x**3 + C_ * x**5


def f_iter(x, n):
    for _ in range(n):
        x = f_scalar(x)
    return x


def householder_orthonormal(rng, rows, k):
    """rows x k matrix with orthonormal columns built as a product of
    Householder reflectors applied to the first k columns of the identity."""
    Q = np.eye(rows)
    for _ in range(3):
        v = rng.standard_normal(rows)
        v /= np.linalg.norm(v)
        Q = Q - 2.0 * np.outer(v, v @ Q)
    return Q[:, :k]


def step1_hyper(**kw):
    base = dict(lr=2e-2, wd=0.1, mu=0.95, nesterov=True, ns_steps=5, eps=0.0)
    base.update(kw)
    return orc.Hyper(**base)


# --- P1: closed form through a chosen SVD (Sec. 2.1: the iteration is an odd
# polynomial, so it acts on singular values only) ---------------------------
@pytest.mark.parametrize("rows,cols", [(12, 20), (20, 12), (16, 16), (1, 9), (9, 1)])
@pytest.mark.parametrize("steps", [1, 5, 10])
def test_closed_form_chosen_singular_values(rows, cols, steps):
    rng = np.random.default_rng(rows * 100 + cols)
    k = min(rows, cols)
    U = householder_orthonormal(rng, rows, k)
    V = householder_orthonormal(rng, cols, k)
    s = np.sort(rng.uniform(0.01, 3.0, size=k))[::-1].copy()
    G = (U * s) @ V.T
    X0 = G / np.linalg.norm(s)
    O = orc.newton_schulz(X0, steps)
    expect = (U * f_iter(s / np.linalg.norm(s), steps)) @ V.T
    assert np.max(np.abs(O - expect)) < 1e-10


def test_closed_form_with_a_coefficient_schedule():
    """One (a, b, c) per step: the singular values go through the composition
    of the per-step scalar polynomials."""
    rng = np.random.default_rng(77)
    rows, cols, k = 10, 14, 10
    U = householder_orthonormal(rng, rows, k)
    V = householder_orthonormal(rng, cols, k)
    s = rng.uniform(0.05, 2.0, size=k)
    sched = [(3.4445, -4.7750, 2.0315), (3.0, -3.5, 1.2), (2.0, -1.5, 0.5)]
    x = s / np.linalg.norm(s)
    for (a, b, c) in sched:
        x = a * x + b * x**3 + c * x**5
    O = orc.newton_schulz(((U * s) @ V.T) / np.linalg.norm(s), 3, coeffs=sched)
    assert np.max(np.abs(O - (U * x) @ V.T)) < 1e-10
    with pytest.raises(ValueError):
        orc.newton_schulz(np.eye(3), 2, coeffs=sched)


def test_closed_form_full_step_matches_scaled_update():
    rng = np.random.default_rng(7)
    rows, cols = 10, 24
    U = householder_orthonormal(rng, rows, rows)
    V = householder_orthonormal(rng, cols, rows)
    s = rng.uniform(0.1, 2.0, size=rows)
    G = (U * s) @ V.T
    W = rng.standard_normal((rows, cols))
    hp = step1_hyper(lr=3e-3, wd=0.05)
    out = orc.muon_step(W, G, np.zeros_like(G), hp)
    # step 1, M_0 = 0: the input is (1+mu) G, a positive multiple of G.
    O = (U * f_iter(s / np.linalg.norm(s), 5)) @ V.T
    Wexp = W - hp.lr * (0.2 * math.sqrt(24) * O + hp.wd * W)
    assert np.allclose(out["nu"], 1.95 * np.linalg.norm(s), rtol=1e-13)
    assert np.max(np.abs(out["W"] - Wexp)) < 1e-11
    assert np.array_equal(out["M"], G)


# --- P2: LAPACK SVD on tiny random inputs; polar-factor band ----------------
@pytest.mark.parametrize("rows,cols", [(8, 8), (24, 40), (64, 96), (48, 17)])
def test_svd_band_and_diagonalisation(rows, cols):
    rng = np.random.default_rng(rows + 3 * cols)
    G = rng.standard_normal((rows, cols))
    Us, s, Vt = np.linalg.svd(G, full_matrices=False)
    sn = s / np.linalg.norm(G)
    out = orc.muon_step(np.zeros_like(G), G, np.zeros_like(G), step1_hyper())
    D = Us.T @ out["O"] @ Vt.T
    off = D - np.diag(np.diag(D))
    assert np.max(np.abs(off)) < 1e-9
    assert np.max(np.abs(np.diag(D) - f_iter(sn, 5))) < 1e-9
    band = np.diag(D)[sn >= 0.003]
    assert band.size > 0
    assert band.min() >= 0.6818 - 1e-4 and band.max() <= 1.2024 + 1e-4
    # the result approximates the polar factor U V^T: same singular vectors,
    # singular values inside the band around 1
    polar = Us @ Vt
    assert np.linalg.norm(out["O"] - polar, 2) <= max(abs(band - 1).max(), 1 - np.diag(D).min()) + 1e-9


# --- P3 / P4: hand-derived 2x2 cases ---------------------------------------
def test_golden_dense_2x2_one_step(golden):
    g = golden("ns_2x2_one_step.txt")
    G = np.array([[1.0, 2.0], [3.0, 4.0]])
    for nesterov in (True, False):
        hp = step1_hyper(ns_steps=1, nesterov=nesterov)
        out = orc.muon_step(np.zeros((2, 2)), G, np.zeros((2, 2)), hp, trace=True)
        A, B, X1 = out["stages"][0]
        assert np.max(np.abs(out["X0"] - g["X0"])) < 1e-14
        assert np.max(np.abs(A - g["A"])) < 1e-14
        assert np.max(np.abs(B - g["B"])) < 1e-13
        assert np.max(np.abs(X1 - g["X1"])) < 1e-13
        assert np.allclose(np.linalg.svd(X1, compute_uv=False), g["SV1"][0], atol=1e-12)
    out5 = orc.muon_step(np.zeros((2, 2)), G, np.zeros((2, 2)), step1_hyper())
    assert np.allclose(np.sort(np.linalg.svd(out5["O"], compute_uv=False)), np.sort(g["SV5"][0]), atol=1e-12)


def test_golden_diagonal_2x2_full_step(golden):
    g = golden("diag_2x2_full_step.txt")
    G = np.diag([3.0, 4.0])
    W = np.array([[1.0, 2.0], [3.0, 4.0]])
    hp = step1_hyper(ns_steps=5)
    out = orc.muon_step(W, G, np.zeros((2, 2)), hp, trace=True)
    assert np.array_equal(out["M"], g["M1"])
    assert abs(out["nu"] - g["NU"][0, 0]) < 1e-13
    assert np.max(np.abs(out["X0"] - g["X0"])) < 1e-15
    for k in range(5):
        assert np.max(np.abs(out["stages"][k][2] - g["X%d" % (k + 1)])) < 1e-12
    assert np.max(np.abs(out["W"] - g["W_N5"])) < 1e-13
    out1 = orc.muon_step(W, G, np.zeros((2, 2)), step1_hyper(ns_steps=1))
    assert np.max(np.abs(out1["W"] - g["W_N1"])) < 1e-13


def test_rank_one_keeps_null_space(golden):
    g = golden("rank_one_iterates.txt")["F1"][0]
    rng = np.random.default_rng(11)
    u = rng.standard_normal(7)
    v = rng.standard_normal(13)
    G = np.outer(u, v)
    for n in range(1, 6):
        O = orc.newton_schulz(G / np.linalg.norm(G), n)
        expect = g[n - 1] * np.outer(u / np.linalg.norm(u), v / np.linalg.norm(v))
        assert np.max(np.abs(O - expect)) < 1e-12


# --- P5: Lemma 1 (update RMS) ------------------------------------------------
@pytest.mark.parametrize("rows,cols,r", [(6, 15, 6), (15, 6, 4), (9, 9, 9)])
def test_lemma1_rms_of_partial_isometry(rows, cols, r):
    rng = np.random.default_rng(rows * cols + r)
    U = householder_orthonormal(rng, rows, r)
    V = householder_orthonormal(rng, cols, r)
    O = U @ V.T
    # Lemma 1 / Appendix A: RMS(U V^T) = sqrt(r / (A*B)); full rank gives sqrt(1/max(A,B))
    rms = orc.update_rms(O, rms_scale=1.0) / math.sqrt(max(rows, cols))
    assert abs(rms - math.sqrt(r / (rows * cols))) < 1e-14
    if r == min(rows, cols):
        assert abs(rms - math.sqrt(1.0 / max(rows, cols))) < 1e-14


def test_lemma1_band_for_oracle_output():
    rng = np.random.default_rng(5)
    for rows, cols in [(32, 80), (80, 32), (40, 40)]:
        G = rng.standard_normal((rows, cols))
        sn = np.linalg.svd(G, compute_uv=False) / np.linalg.norm(G)
        out = orc.muon_step(np.zeros_like(G), G, np.zeros_like(G), step1_hyper())
        ratio = math.sqrt(np.mean(out["O"] ** 2)) * math.sqrt(max(rows, cols))
        if sn.min() >= 0.003:
            assert 0.6818 - 1e-4 <= ratio <= 1.2024 + 1e-4
        assert abs(out["rms"] - 0.2 * ratio) < 1e-13


# --- P6: symmetries -----------------------------------------------------------
def test_scale_invariance_and_step1_independence_of_mu():
    rng = np.random.default_rng(3)
    G = rng.standard_normal((9, 14))
    Z = np.zeros_like(G)
    ref = orc.muon_step(Z, G, Z, step1_hyper())["O"]
    for alpha in (1e-6, 17.0):
        assert np.max(np.abs(orc.muon_step(Z, alpha * G, Z, step1_hyper())["O"] - ref)) < 1e-10
    for mu, nest in ((0.5, True), (0.95, False), (0.0, True)):
        o = orc.muon_step(Z, G, Z, step1_hyper(mu=mu, nesterov=nest))["O"]
        assert np.max(np.abs(o - ref)) < 1e-10


def test_transpose_equivariance_and_internal_transpose_is_a_no_op():
    rng = np.random.default_rng(4)
    G = rng.standard_normal((21, 8))  # rows > cols: the oracle transposes inside
    X0 = G / np.linalg.norm(G)
    O = orc.newton_schulz(X0, 5)
    Ot = orc.newton_schulz(np.ascontiguousarray(X0.T), 5)
    assert np.max(np.abs(O - Ot.T)) < 1e-12
    # the same iteration written without any transposition (Eq. 2 literally)
    X = X0.copy()
    for _ in range(5):
        XXt = X @ X.T
        X = A_ * X + B_ * XXt @ X + C_ * XXt @ XXt @ X
    assert np.max(np.abs(O - X)) < 1e-12


def test_signed_permutation_equivariance():
    rng = np.random.default_rng(8)
    rows, cols = 6, 10
    G = rng.standard_normal((rows, cols))
    P1 = np.eye(rows)[rng.permutation(rows)] * rng.choice([-1.0, 1.0], size=rows)[:, None]
    P2 = np.eye(cols)[rng.permutation(cols)] * rng.choice([-1.0, 1.0], size=cols)[None, :]
    X0 = G / np.linalg.norm(G)
    lhs = orc.newton_schulz(P1 @ X0 @ P2, 5)
    rhs = P1 @ orc.newton_schulz(X0, 5) @ P2
    assert np.max(np.abs(lhs - rhs)) < 1e-12


# --- P7: element-wise parts against hand formulas ---------------------------
def test_momentum_nesterov_and_zero_ns_steps():
    rng = np.random.default_rng(9)
    rows, cols = 5, 3
    W = rng.standard_normal((rows, cols))
    G = rng.standard_normal((rows, cols))
    M = rng.standard_normal((rows, cols))
    mu, lr, wd, eps = 0.9, 0.01, 0.2, 1e-7
    hp = orc.Hyper(lr=lr, wd=wd, mu=mu, nesterov=True, ns_steps=0, eps=eps)
    out = orc.muon_step(W, G, M, hp)
    for i in range(rows):
        for j in range(cols):
            m1 = mu * M[i, j] + G[i, j]
            assert out["M"][i, j] == m1
    U = np.array([[mu * (mu * M[i, j] + G[i, j]) + G[i, j] for j in range(cols)] for i in range(rows)])
    nu = math.sqrt(sum(U[i, j] ** 2 for i in range(rows) for j in range(cols)))
    assert abs(out["nu"] - nu) < 1e-14
    Wexp = W - lr * (0.2 * math.sqrt(5) * U / (nu + eps) + wd * W)
    assert np.max(np.abs(out["W"] - Wexp)) < 1e-15
    out2 = orc.muon_step(W, G, M, orc.Hyper(lr=lr, wd=wd, mu=mu, nesterov=False, ns_steps=0, eps=eps))
    U2 = mu * M + G
    assert np.max(np.abs(out2["X0"] - U2 / (np.linalg.norm(U2) + eps))) < 1e-15


def test_zero_gradient_and_zero_momentum_only_decays():
    W = np.arange(6, dtype=np.float64).reshape(2, 3)
    Z = np.zeros_like(W)
    out = orc.muon_step(W, Z, Z, orc.Hyper(lr=0.1, wd=0.5))
    assert np.array_equal(out["O"], Z)
    assert np.allclose(out["W"], (1 - 0.05) * W, rtol=0, atol=1e-15)


def test_nonfinite_input_leaves_weight_unchanged():
    W = np.ones((2, 2))
    G = np.array([[1.0, np.inf], [0.0, 1.0]])
    out = orc.muon_step(W, G, np.zeros((2, 2)), orc.Hyper())
    assert out["nonfinite"] and np.array_equal(out["W"], W)


def test_protected_momentum_on_a_nonfinite_gradient():
    """The other reading of a non-finite gradient: weight AND momentum are left as
    they were; a finite gradient gives exactly the default step."""
    rng = np.random.default_rng(13)
    W, M = rng.standard_normal((3, 4)), rng.standard_normal((3, 4))
    G = rng.standard_normal((3, 4))
    hp = orc.Hyper(protect_momentum=True)
    same = orc.muon_step(W, G, M, hp)
    ref = orc.muon_step(W, G, M, orc.Hyper())
    assert np.array_equal(same["W"], ref["W"]) and np.array_equal(same["M"], ref["M"]) and not same["nonfinite"]
    for bad in (np.nan, np.inf, -np.inf):
        Gb = G.copy()
        Gb[2, 1] = bad
        out = orc.muon_step(W, Gb, M, hp)
        assert out["nonfinite"] and np.array_equal(out["W"], W) and np.array_equal(out["M"], M)
        plain = orc.muon_step(W, Gb, M, orc.Hyper())
        assert plain["nonfinite"] and np.array_equal(plain["W"], W) and not np.all(np.isfinite(plain["M"]))


def test_multi_step_momentum_chain():
    rng = np.random.default_rng(12)
    W = rng.standard_normal((4, 6))
    M = np.zeros((4, 6))
    Gs = [rng.standard_normal((4, 6)) for _ in range(3)]
    hp = orc.Hyper()
    for G in Gs:
        out = orc.muon_step(W, G, M, hp)
        W, M = out["W"], out["M"]
    # closed form of the momentum recursion: M_3 = mu^2 G1 + mu G2 + G3
    assert np.max(np.abs(M - (0.95**2 * Gs[0] + 0.95 * Gs[1] + Gs[2]))) < 1e-14


# --- P8: brute force on tiny inputs -----------------------------------------
@pytest.mark.parametrize("rows,cols", [(3, 5), (5, 3), (8, 8), (2, 7)])
def test_brute_force_explicit_polynomial(rows, cols):
    rng = np.random.default_rng(rows * 31 + cols)
    X = rng.standard_normal((rows, cols))
    X /= np.linalg.norm(X)
    O = orc.newton_schulz(X, 1)

    def mat(P, Q):
        out = np.zeros((len(P), len(Q[0])))
        for i in range(len(P)):
            for j in range(len(Q[0])):
                acc = 0.0
                for k in range(len(Q)):
                    acc += P[i][k] * Q[k][j]
                out[i, j] = acc
        return out

    Xt = X.T
    XXtX = mat(mat(X, Xt), X)
    XXtXXtX = mat(mat(X, Xt), XXtX)
    expect = A_ * X + B_ * XXtX + C_ * XXtXXtX
    assert np.max(np.abs(O - expect)) < 1e-13


def test_fixed_points_and_band_of_the_scalar_map():
    # facts about f used as test bounds elsewhere: the band [0.6818, 1.2024]
    # is invariant and attracts (0, 0.868)
    xs = np.linspace(0.6818, 1.2024, 20001)
    fx = f_scalar(xs)
    assert fx.min() >= 0.6818 - 1e-4 and fx.max() <= 1.2024 + 1e-4
    assert abs(f_scalar(0.8680) - 0.8680) < 2e-4
    for x0 in (0.003, 0.01, 0.1, 0.5, 1.0):
        assert 0.6818 - 1e-4 <= f_iter(x0, 5) <= 1.2024 + 1e-4


# --- sensitivity: the pins above would notice a plausible mistake ------------
def test_pins_are_sensitive_to_planted_mistakes(monkeypatch):
    rng = np.random.default_rng(21)
    rows, cols = 6, 11
    U = householder_orthonormal(rng, rows, rows)
    V = householder_orthonormal(rng, cols, rows)
    s = rng.uniform(0.2, 2.0, size=rows)
    G = (U * s) @ V.T
    X0 = G / np.linalg.norm(s)
    expect = (U * f_iter(s / np.linalg.norm(s), 5)) @ V.T
    good = orc.newton_schulz(X0, 5)
    assert np.max(np.abs(good - expect)) < 1e-10
    # swapped b and c, a dropped quintic term, a wrong sign: each must show
    for a, b, c in ((A_, C_, B_), (A_, B_, 0.0), (A_, -B_, C_), (-A_, B_, C_)):
        bad = orc.newton_schulz(X0, 5, a, b, c)
        assert np.max(np.abs(bad - expect)) > 1e-3
    # a transposed operand in the Gram product (X^T X instead of X X^T) cannot
    # even be formed for a non-square input, and for a square one it breaks
    # the closed form:
    Xs = rng.standard_normal((5, 5))
    Xs /= np.linalg.norm(Xs)
    wrong = A_ * Xs + (B_ * (Xs.T @ Xs) + C_ * (Xs.T @ Xs) @ (Xs.T @ Xs)) @ Xs
    assert np.max(np.abs(wrong - orc.newton_schulz(Xs, 1))) > 1e-3
    # Nesterov flag and the decay term are visible in a second step
    W = rng.standard_normal((rows, cols))
    M = rng.standard_normal((rows, cols))
    o1 = orc.muon_step(W, G, M, orc.Hyper(nesterov=True))
    o2 = orc.muon_step(W, G, M, orc.Hyper(nesterov=False))
    assert np.max(np.abs(o1["O"] - o2["O"])) > 1e-3
    o3 = orc.muon_step(W, G, M, orc.Hyper(wd=0.0))
    assert np.max(np.abs(o1["W"] - o3["W"])) > 1e-4


# ---------------------------------------------------------------------------
# Sec. 3.1: the three ways of scaling the update
# ---------------------------------------------------------------------------
def test_scale_variants_against_hand_formulas():
    """With ns_steps = 0 and eps = 0 the orthogonalised update is O = U/||U||_F,
    so every variant of Sec. 3.1 is closed-form element-wise arithmetic:
      Adjusted LR:  W - lr*(0.2*sqrt(max(A,B)) * U/||U|| + wd*W)
      Baseline:     W - lr*(0.2*sqrt(H)        * U/||U|| + wd*W)
      Update Norm:  RMS(O) = ||O||_F/sqrt(A*B) = 1/sqrt(A*B), hence
                    W - lr*(0.2*sqrt(A*B)      * U/||U|| + wd*W)."""
    rng = np.random.default_rng(5)
    rows, cols = 6, 10
    W = rng.standard_normal((rows, cols))
    G = rng.standard_normal((rows, cols))
    M = rng.standard_normal((rows, cols))
    mu, lr, wd = 0.9, 0.03, 0.2
    Mn = mu * M + G
    U = mu * Mn + G
    unit = U / np.sqrt((U ** 2).sum())
    for mode, dim, fac in (("adjusted_lr", 0.0, 0.2 * np.sqrt(10.0)),
                           ("fixed_dim", 49.0, 0.2 * 7.0),
                           ("update_norm", 0.0, 0.2 * np.sqrt(60.0))):
        hp = orc.Hyper(lr=lr, wd=wd, mu=mu, nesterov=True, ns_steps=0, eps=0.0, scale_mode=mode, scale_dim=dim)
        out = orc.muon_step(W, G, M, hp)
        expect = W - lr * (fac * unit + wd * W)
        assert np.allclose(out["W"], expect, rtol=1e-13, atol=1e-15), mode
        assert abs(out["rms"] - fac / np.sqrt(60.0)) <= 1e-13, mode


def test_update_norm_has_rms_exactly_point_two_after_the_iteration():
    rng = np.random.default_rng(6)
    W = rng.standard_normal((12, 7))
    G = rng.standard_normal((12, 7))
    hp = orc.Hyper(lr=0.01, wd=0.0, scale_mode="update_norm")
    out = orc.muon_step(W, G, np.zeros_like(G), hp)
    u = (W - out["W"]) / hp.lr
    assert abs(np.sqrt(np.mean(u ** 2)) - 0.2) <= 1e-12
    assert abs(out["rms"] - 0.2) <= 1e-12
    # the direction is still O
    assert np.allclose(u / np.linalg.norm(u), out["O"] / np.linalg.norm(out["O"]), atol=1e-12)


# ---------------------------------------------------------------------------
# bf16 storage model
# ---------------------------------------------------------------------------
def test_round_to_bf16_known_values_and_ties():
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: even significand wins (1.0);
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 and 1 + 2^-6: even wins (1 + 2^-6)
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -3.4445, 0.0, 2.0 ** -130])
    r = orc.round_to_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2.0 ** -6 and r[3] == 1.0 + 2.0 ** -7
    assert r[4] == -3.4375 and r[5] == 0.0
    # agrees with an independent implementation on random values
    import torch
    y = np.random.default_rng(3).standard_normal(10000) * 10.0 ** np.random.default_rng(4).uniform(-6, 6, 10000)
    assert np.array_equal(orc.round_to_bf16(y), torch.from_numpy(y).to(torch.float32).to(torch.bfloat16).double().numpy())


def test_bf16_storage_model_is_the_iteration_with_rounding_only():
    """The model is the float64 iteration plus bf16 rounding of the stored
    matrices: it stays within a few bf16 roundings (2^-9 each) amplified by the
    map of the float64 result, but not closer than one rounding; it follows the
    same orientation rule, and with no iteration it is bf16(U)/||U||_F."""
    rng = np.random.default_rng(8)
    G = rng.standard_normal((24, 40))
    ref = orc.newton_schulz(orc.frobenius_normalise(G, 1e-7)[1], 5)
    mod = orc.newton_schulz_bf16_storage(G, 1e-7, 5)
    err = np.linalg.norm(mod - ref) / np.linalg.norm(ref)
    assert 1e-4 < err < 5e-2
    # orientation rule and the no-iteration case
    assert np.allclose(orc.newton_schulz_bf16_storage(G.T, 1e-7, 5), mod.T, rtol=0, atol=0)
    x0 = orc.newton_schulz_bf16_storage(G, 0.0, 0)
    assert np.allclose(x0, orc.round_to_bf16(G) / np.linalg.norm(G), rtol=1e-15)


def test_bf16_storage_model_against_the_hand_derived_2x2_example(golden):
    """Two iterations on a 2x2 input whose every stored value was rounded to 8
    significant bits by hand (exact rational arithmetic, each decision listed in
    the fixture): the model must reproduce every stored matrix exactly, also when
    the input is embedded in a wide or a tall matrix (orientation rule)."""
    g = golden("bf16_storage_2x2_two_steps.txt")
    tr = []
    out = orc.newton_schulz_bf16_storage(g["U"], 0.0, 2, trace=tr)
    assert np.array_equal(tr[0], g["XB"])
    for k, names in ((1, ("A", "B", "X1")), (2, ("A2", "B2", "X2"))):
        for got, name in zip(tr[k], names):
            assert np.array_equal(got, g[name]), name
    assert np.array_equal(out, g["X2"])
    assert np.array_equal(orc.newton_schulz_bf16_storage(g["U"], 0.0, 1), g["X1"])
    # the reading with a*I folded into the stored polynomial
    tr = []
    out = orc.newton_schulz_bf16_storage(g["U"], 0.0, 2, trace=tr, fold_identity=True)
    assert np.array_equal(tr[0], g["XB"])
    for k, names in ((1, ("A", "BI", "X1F")), (2, ("A2F", "BI2", "X2F"))):
        for got, name in zip(tr[k], names):
            assert np.array_equal(got, g[name]), name
    assert np.array_equal(out, g["X2F"]) and not np.array_equal(g["X2F"], g["X2"])
    # a wide (2 x 3) and a tall (3 x 2) embedding of the same input: a zero column (row) changes no
    # stored value, and the tall one must come back transposed
    wide = np.concatenate([g["U"], np.zeros((2, 1))], axis=1)
    assert np.array_equal(orc.newton_schulz_bf16_storage(wide, 0.0, 2)[:, :2], g["X2"])
    tall = np.ascontiguousarray(np.concatenate([g["U"].T, np.zeros((1, 2))], axis=0))
    assert np.array_equal(orc.newton_schulz_bf16_storage(tall, 0.0, 2)[:2, :], g["X2"].T)


def _bf16_model_with_a_planted_mistake(U, kind):
    """One iteration of the bf16 storage model with one plausible mistake planted
    (a copy of the model's few lines, each variant changing one of them)."""
    r = orc.round_to_bf16
    a, b, c = A_, B_, C_
    s = 1.0 / math.sqrt(float(np.sum(U * U)))
    if kind == "s_before_rounding":
        X, sa, sx = r(s * U), 1.0, 1.0
    else:
        X, sa, sx = r(U), s * s, s
    gram = X.T @ X if kind == "transposed_gram" else X @ X.T
    A = sa * gram if kind == "A_not_rounded" else r(sa * gram)
    if kind == "bA_rounded_first":
        B = r(r(b * A) + c * (A @ A))
    elif kind == "B_not_rounded":
        B = b * A + c * (A @ A)
    elif kind == "b_and_c_swapped":
        B = r(c * A + b * (A @ A))
    else:
        B = r(b * A + c * (A @ A))
    Y = a * X + B @ X
    if kind == "rounded_then_scaled":
        return B, r(sx * r(Y))
    if kind == "X_not_rounded":
        return B, sx * Y
    if kind == "s_squared_on_X":
        return B, r(sa * Y)
    return B, r(sx * Y)


def test_bf16_storage_pin_notices_planted_mistakes(golden, monkeypatch):
    """The 2x2 example separates the model from its plausible wrong versions:
    a rounding left out (A, B, X), done twice or too early (b*A, s*U), the factor
    s misapplied, a transposed Gram product, swapped coefficients.  The values a
    wrong model stores are the ones listed in the fixture's comment."""
    g = golden("bf16_storage_2x2_two_steps.txt")
    B, X1 = _bf16_model_with_a_planted_mistake(g["U"], "none")
    assert np.array_equal(B, g["B"]) and np.array_equal(X1, g["X1"])  # the copy itself is faithful
    for kind in ("A_not_rounded", "s_before_rounding", "bA_rounded_first", "B_not_rounded", "rounded_then_scaled",
                 "transposed_gram", "X_not_rounded", "s_squared_on_X", "b_and_c_swapped"):
        B, X1 = _bf16_model_with_a_planted_mistake(g["U"], kind)
        assert not np.array_equal(X1, g["X1"]), kind
    B, X1 = _bf16_model_with_a_planted_mistake(g["U"], "A_not_rounded")
    assert B[0, 1] == -1.2890625 and np.array_equal(X1, [[0.51171875, 0.1904296875], [0.06494140625, 0.609375]])
    B, X1 = _bf16_model_with_a_planted_mistake(g["U"], "s_before_rounding")
    assert X1[0, 1] == 0.19140625 and X1[1, 0] == 0.0625
    B, X1 = _bf16_model_with_a_planted_mistake(g["U"], "rounded_then_scaled")
    assert X1[1, 0] == 0.068359375
    # the same, planted in the oracle itself: leaving out its n-th rounding (input, A, B, X1, A2, B2, X2)
    real = orc.round_to_bf16
    for skip in range(7):
        calls = {"n": 0}

        def skipping(x, _skip=skip):
            calls["n"] += 1
            return np.asarray(x, dtype=np.float64) if calls["n"] - 1 == _skip else real(x)

        monkeypatch.setattr(orc, "round_to_bf16", skipping)
        out = orc.newton_schulz_bf16_storage(g["U"], 0.0, 2)
        monkeypatch.setattr(orc, "round_to_bf16", real)
        assert calls["n"] == 7
        assert not np.array_equal(out, g["X2"]), skip


@pytest.mark.parametrize("rows,cols", [(6, 20), (12, 12), (9, 40)])
def test_two_iterations_equal_one_pass_with_the_product_of_their_polynomials(rows, cols):
    """Eq. 2 is X_{k+1} = P_k X_k with P_k = a I + b A_k + c A_k^2, A_k = X_k X_k^T.
    P_k is a polynomial in A_k, so A_{k+1} = P_k A_k P_k = P_k^2 A_k, and two
    iterations are X_{k+2} = P_{k+1} P_k X_k with P_{k+1} formed from A_{k+1}
    alone.  The GPU path uses this for wide matrices; here the oracle's plain
    iteration is the reference, with a different coefficient triple per
    iteration so that a swapped pair of triples would show."""
    rng = np.random.default_rng(rows * 100 + cols)
    X0 = orc.frobenius_normalise(rng.standard_normal((rows, cols)), 0.0)[1]
    coeffs = [(3.4445, -4.7750, 2.0315), (3.0, -4.0, 1.9), (2.5, -3.0, 1.5), (3.4445, -4.7750, 2.0315)]
    ref = orc.newton_schulz(X0, 4, coeffs=coeffs)
    I = np.eye(rows)
    X = X0
    for k in (0, 2):
        (a1, b1, c1), (a2, b2, c2) = coeffs[k], coeffs[k + 1]
        A = X @ X.T
        P1 = a1 * I + b1 * A + c1 * (A @ A)
        A1 = P1 @ P1 @ A
        P2 = a2 * I + b2 * A1 + c2 * (A1 @ A1)
        X = (P2 @ P1) @ X
    assert np.linalg.norm(X - ref) <= 1e-11 * np.linalg.norm(ref)
