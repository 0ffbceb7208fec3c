"""Pins of the float64 oracle against what the paper and the mathematics fix.

None of these retype the oracle's formulas: they use closed forms, brute-force definitions,
finite differences of the *forward* map, invariants and equivariances.
"""
import numpy as np
import pytest

from oracle import dense
from oracle import idkm_ref as R

RNG = np.random.default_rng(12345)


def rand_problem(m, d, k, scale=0.05, seed=0):
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((m, d)) * scale
    C = W[rng.choice(m, k, replace=False)] + rng.standard_normal((k, d)) * scale * 0.05
    G = rng.standard_normal((m, d))
    return W, C, G


# ----------------------------------------------------------------------------------------
# E-step: Eq. for a_j(w_i, C)
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("d,k", [(1, 2), (1, 4), (2, 4), (4, 8), (3, 5)])
def test_attention_rows_are_probabilities_and_match_bruteforce(d, k):
    W, C, _ = rand_problem(50, d, k, seed=d * 10 + k)
    tau = 0.03
    A = R.attention(W, C, tau)
    assert np.all(A >= 0) and np.all(A <= 1)
    np.testing.assert_allclose(A.sum(1), 1.0, rtol=0, atol=1e-14)
    # the definition, element by element, without any max-subtraction
    for i in range(W.shape[0]):
        e = np.array([np.exp(-np.linalg.norm(W[i] - C[j]) / tau) for j in range(k)])
        np.testing.assert_allclose(A[i], e / e.sum(), rtol=1e-12, atol=0)


def test_attention_survives_tiny_tau_without_nan():
    W, C, _ = rand_problem(20, 2, 4, seed=3)
    A = R.attention(W, C, 1e-9)
    assert np.all(np.isfinite(A))
    np.testing.assert_allclose(A.sum(1), 1.0, atol=1e-14)
    # tau -> 0 is the hard quantiser q (Section 3.2, "if tau = 0 then r_tau = q")
    nearest = np.argmin(((W[:, None] - C[None]) ** 2).sum(-1), 1)
    assert np.array_equal(np.argmax(A, 1), nearest)
    assert np.allclose(A.max(1), 1.0)


# ----------------------------------------------------------------------------------------
# M-step invariants (Eq. c_j^+)
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("d,k", [(1, 4), (2, 3), (4, 16)])
def test_step_invariants(d, k):
    W, C, _ = rand_problem(200, d, k, seed=7 + d)
    Cp, S, dead = R.step(W, C, 0.02)
    assert dead == 0
    np.testing.assert_allclose(S.sum(), W.shape[0], rtol=1e-13)
    np.testing.assert_allclose((S[:, None] * Cp).sum(0), W.sum(0), rtol=1e-11, atol=1e-13)
    assert np.all(Cp >= W.min(0) - 1e-15) and np.all(Cp <= W.max(0) + 1e-15)
    Wq, A, S2, F = R.final(W, Cp, 0.02, want_A=True)
    np.testing.assert_allclose(Wq, A @ Cp, rtol=1e-13, atol=1e-16)
    assert np.all(Wq >= Cp.min(0) - 1e-15) and np.all(Wq <= Cp.max(0) + 1e-15)
    np.testing.assert_allclose(S2, A.sum(0), rtol=1e-13)
    np.testing.assert_allclose(F, (A.T @ W) / A.sum(0)[:, None], rtol=1e-12, atol=1e-16)


def test_step_matches_matrix_form_of_eq_centers():
    # C+ = diag(A^T 1)^-1 A^T W, with A materialised by brute force
    W, C, _ = rand_problem(64, 2, 4, seed=11)
    tau = 0.04
    D = np.linalg.norm(W[:, None] - C[None], axis=-1)
    E = np.exp(-D / tau)
    A = E / E.sum(1, keepdims=True)
    expect = np.diag(1.0 / (A.T @ np.ones(64))) @ A.T @ W
    Cp, _, _ = R.step(W, C, tau)
    np.testing.assert_allclose(Cp, expect, rtol=1e-12, atol=1e-16)


# ----------------------------------------------------------------------------------------
# closed form, k = 1: A = 1, C* = mean(W), Wq_i = mean, J_C = 0, dW_i = mean_i(G)
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("d", [1, 2, 4])
def test_single_centroid_closed_form(d):
    rng = np.random.default_rng(d)
    W = rng.standard_normal((37, d))
    G = rng.standard_normal((37, d))
    C0 = rng.standard_normal((1, d))
    Ct, it, res, dead = R.forward(W, C0, 0.1, 0.0, 3)
    np.testing.assert_allclose(Ct[0], W.mean(0), rtol=1e-13)
    Wq, _, S, F = R.final(W, Ct, 0.1)
    np.testing.assert_allclose(Wq, np.tile(W.mean(0), (37, 1)), rtol=1e-13)
    for mode in ("implicit", "jfb"):
        dW, dC, _, _ = R.backward(W, G, Ct, 0.1, S, F, mode=mode, adj_max_iter=5)
        np.testing.assert_allclose(dW, np.tile(G.mean(0), (37, 1)), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(dC[0], G.sum(0), rtol=1e-12)


# ----------------------------------------------------------------------------------------
# closed form, symmetric two-point data: W = {-a, +a} repeated, k = 2, C0 = {-c0, +c0}.
# The iterate stays symmetric and c+ = a tanh(c / tau); non-trivial fixed point iff a/tau > 1.
# ----------------------------------------------------------------------------------------
def _tanh_fixed_point(a, tau):
    lo, hi = 1e-12, a
    f = lambda c: a * np.tanh(c / tau) - c
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if f(mid) > 0:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def test_two_point_closed_form_forward_and_gradients():
    a, tau, reps = 0.05, 0.02, 8
    W = np.array([[-a], [a]] * reps)
    C0 = np.array([[-0.03], [0.03]])
    # one step: c+ = a tanh(c/tau)
    Cp, _, _ = R.step(W, C0, tau)
    np.testing.assert_allclose(Cp[:, 0], [-a * np.tanh(0.03 / tau), a * np.tanh(0.03 / tau)], rtol=1e-13)
    cs = _tanh_fixed_point(a, tau)
    Ct, it, res, _ = R.forward(W, C0, tau, 1e-15, 2000)
    np.testing.assert_allclose(Ct[:, 0], [-cs, cs], rtol=1e-11)
    Wq, _, S, F = R.final(W, Ct, tau)
    th = np.tanh(cs / tau)
    np.testing.assert_allclose(Wq[:, 0], np.array([-1, 1] * reps) * cs * th, rtol=1e-11)
    # L = <G, Wq> with G = (-1, +1, ...)/1: by symmetry only the antisymmetric direction matters.
    # Wq(+a) = c tanh(c/tau) with c = c*(a): dWq/da = c' [tanh + (c/tau) sech^2],
    # implicit c' = tanh / (1 - (a/tau) sech^2), JFB c' = tanh.
    G = np.array([[-1.0], [1.0]] * reps)
    sech2 = 1.0 / np.cosh(cs / tau) ** 2
    direction = np.array([[-1.0], [1.0]] * reps)
    for mode, cprime in (("implicit", th / (1 - (a / tau) * sech2)), ("jfb", th)):
        dW, dC, _, _ = R.backward(W, G, Ct, tau, S, F, mode=mode, adj_tol=1e-15, adj_max_iter=5000)
        # dL/da along the antisymmetric direction: L(a) = 2 reps * Wq(+a)
        dL_da = float((dW * direction).sum())
        expect = 2 * reps * cprime * (th + (cs / tau) * sech2)
        np.testing.assert_allclose(dL_da, expect, rtol=1e-9)


def test_two_point_collapse_when_a_over_tau_below_one():
    a, tau = 0.01, 0.02
    W = np.array([[-a], [a]] * 4)
    Ct, _, _, _ = R.forward(W, np.array([[-0.009], [0.009]]), tau, 0.0, 400)
    assert np.all(np.abs(Ct) < 1e-12)


# ----------------------------------------------------------------------------------------
# tau -> 0: one soft step equals one Lloyd step; fixed points coincide (Section 3.2)
# ----------------------------------------------------------------------------------------
def _lloyd_step(W, C):
    lab = np.argmin(((W[:, None] - C[None]) ** 2).sum(-1), 1)
    out = C.copy()
    for j in range(C.shape[0]):
        if np.any(lab == j):
            out[j] = W[lab == j].mean(0)
    return out


@pytest.mark.parametrize("d,k", [(1, 3), (2, 4), (4, 4)])
def test_lloyd_limit(d, k):
    rng = np.random.default_rng(100 + d)
    centers = rng.standard_normal((k, d))
    W = np.concatenate([c + 0.05 * rng.standard_normal((12, d)) for c in centers])
    C = centers + 0.1 * rng.standard_normal((k, d))
    tau = 1e-5
    for _ in range(6):
        soft, _, _ = R.step(W, C, tau)
        hard = _lloyd_step(W, C)
        np.testing.assert_allclose(soft, hard, rtol=1e-9, atol=1e-12)
        C = hard
    np.testing.assert_allclose(_lloyd_step(W, C), C, atol=1e-15)       # Lloyd fixed point
    Cs, _, _, _ = R.forward(W, C, tau, 0.0, 5)
    np.testing.assert_allclose(Cs, C, rtol=1e-9, atol=1e-12)


# ----------------------------------------------------------------------------------------
# Algorithm 1: returned C is a fixed point to tol; stop rule; max_iter = 0
# ----------------------------------------------------------------------------------------
def test_forward_returns_fixed_point_and_obeys_stop_rule():
    W, C0, _ = rand_problem(300, 2, 4, seed=21)
    tau = 0.02
    Ct, it, res, _ = R.forward(W, C0, tau, 1e-10, 5000)
    assert it < 5000 and res < 1e-10
    Cn, _, _ = R.step(W, Ct, tau)
    assert np.linalg.norm(Cn - Ct) / np.linalg.norm(Cn) < 1e-10
    # tol = 0 runs exactly max_iter steps and equals manual repetition of the map
    Cf, it2, _, _ = R.forward(W, C0, tau, 0.0, 7)
    assert it2 == 7
    Cm = C0.copy()
    for _ in range(7):
        Cm, _, _ = R.step(W, Cm, tau)
    np.testing.assert_array_equal(Cf, Cm)
    # the stop test is made on the relative change of the step just taken, strict <
    Cm, prev = C0.copy(), None
    for t in range(1, it + 1):
        nxt, _, _ = R.step(W, Cm, tau)
        r = np.linalg.norm(nxt - Cm) / np.linalg.norm(nxt)
        assert (r < 1e-10) == (t == it)
        Cm = nxt
    C_same, it0, _, _ = R.forward(W, C0, tau, 1e-6, 0)
    assert it0 == 0
    np.testing.assert_array_equal(C_same, C0)


# ----------------------------------------------------------------------------------------
# equivariances of F
# ----------------------------------------------------------------------------------------
def test_equivariances():
    W, C, G = rand_problem(120, 2, 5, seed=31)
    tau = 0.03
    base, S, _ = R.step(W, C, tau)
    perm = np.array([3, 0, 4, 1, 2])
    pc, pS, _ = R.step(W, C[perm], tau)
    np.testing.assert_allclose(pc, base[perm], rtol=1e-13)
    np.testing.assert_allclose(pS, S[perm], rtol=1e-13)
    rows = np.random.default_rng(0).permutation(120)
    np.testing.assert_allclose(R.step(W[rows], C, tau)[0], base, rtol=1e-12)
    t = np.array([0.3, -0.2])
    np.testing.assert_allclose(R.step(W + t, C + t, tau)[0], base + t, rtol=1e-12)
    np.testing.assert_allclose(R.step(3 * W, 3 * C, 3 * tau)[0], 3 * base, rtol=1e-12)
    np.testing.assert_allclose(R.step(np.tile(W, (3, 1)), C, tau)[0], base, rtol=1e-12)
    # gradients follow the centroid permutation too
    Ct, _, _, _ = R.forward(W, C, tau, 0.0, 20)
    _, _, Sf, F = R.final(W, Ct, tau)
    dW, dC, _, _ = R.backward(W, G, Ct, tau, Sf, F, adj_max_iter=15)
    _, _, Sp, Fp = R.final(W, Ct[perm], tau)
    dWp, dCp, _, _ = R.backward(W, G, Ct[perm], tau, Sp, Fp, adj_max_iter=15)
    np.testing.assert_allclose(dWp, dW, rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(dCp, dC[perm], rtol=1e-10, atol=1e-14)


# ----------------------------------------------------------------------------------------
# implicit gradient = central finite differences of L(W) = <G, Wq(W, C*(W))>  (m <= 64)
# ----------------------------------------------------------------------------------------
def _converged(W, C0, tau):
    Ct, it, res, _ = R.forward(W, C0, tau, 1e-15, 20000)
    assert res < 1e-13, (it, res)
    return Ct


@pytest.mark.parametrize("m,d,k,tau", [(40, 1, 4, 0.02), (48, 2, 4, 0.03), (64, 4, 8, 0.015), (33, 1, 2, 0.02)])
def test_implicit_gradient_matches_finite_differences(m, d, k, tau):
    W, C0, G = rand_problem(m, d, k, seed=m + d + k)
    Ct = _converged(W, C0, tau)
    _, _, S, F = R.final(W, Ct, tau)
    dW, dC, it, res = R.backward(W, G, Ct, tau, S, F, mode="implicit", adj_tol=1e-15, adj_max_iter=20000)
    assert res < 1e-13

    def loss(Wp):
        Cp = _converged(Wp, Ct, tau)
        return float((G * R.final(Wp, Cp, tau)[0]).sum())

    h = 1e-6
    rng = np.random.default_rng(5)
    coords = [(int(i), int(a)) for i, a in zip(rng.choice(m, 12, replace=False), rng.integers(0, d, 12))]
    for (i, a) in coords:
        Wp, Wm = W.copy(), W.copy()
        Wp[i, a] += h
        Wm[i, a] -= h
        fd = (loss(Wp) - loss(Wm)) / (2 * h)
        assert abs(fd - dW[i, a]) <= 2e-6 * max(1.0, np.abs(dW).max()), (i, a, fd, dW[i, a])
    # translation equivariance of Wq at the fixed point: sum_i dW_i = sum_i G_i (exact for implicit)
    np.testing.assert_allclose(dW.sum(0), G.sum(0), rtol=1e-9, atol=1e-10)
    # ... and it must fail for JFB, which drops the (I - J)^-1 factor
    dWj, _, _, _ = R.backward(W, G, Ct, tau, S, F, mode="jfb")
    assert np.abs(dWj.sum(0) - G.sum(0)).max() > 1e-3


# ----------------------------------------------------------------------------------------
# JFB gradient = exact derivative of the one-step function with the linearisation point held:
#   H(W) = <G, Wq(W, Cbar + F(Cbar, W) - F(Cbar, W0))>   =>   dH/dW at W0 = (dWq/dW)^T G + (dF/dW)^T g
# for ANY Cbar (converged or not).  (Section 4.3: M* = I.)
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,d,k,tau", [(30, 1, 4, 0.02), (24, 2, 3, 0.05), (20, 4, 4, 0.05)])
def test_jfb_gradient_is_one_step_derivative(m, d, k, tau):
    W, Cbar, G = rand_problem(m, d, k, seed=77 + d)
    _, _, S, F = R.final(W, Cbar, tau)
    dW, dC, _, _ = R.backward(W, G, Cbar, tau, S, F, mode="jfb")
    F0 = R.step(W, Cbar, tau)[0]

    def H(Wp):
        Cp = Cbar + R.step(Wp, Cbar, tau)[0] - F0
        return float((G * R.final(Wp, Cp, tau)[0]).sum())

    h = 1e-6
    for i in range(0, m, 3):
        for a in range(d):
            Wp, Wm = W.copy(), W.copy()
            Wp[i, a] += h
            Wm[i, a] -= h
            fd = (H(Wp) - H(Wm)) / (2 * h)
            assert abs(fd - dW[i, a]) <= 1e-6 * max(1.0, np.abs(dW).max()), (i, a, fd, dW[i, a])
    # dC in JFB mode is the direct codebook gradient: derivative of <G, Wq(W, C)> in C
    for j in range(k):
        for a in range(d):
            Cp, Cm = Cbar.copy(), Cbar.copy()
            Cp[j, a] += h
            Cm[j, a] -= h
            fd = float((G * (R.final(W, Cp, tau)[0] - R.final(W, Cm, tau)[0])).sum()) / (2 * h)
            assert abs(fd - dC[j, a]) <= 1e-6 * max(1.0, np.abs(dC).max())


# ----------------------------------------------------------------------------------------
# adjoint_apply is the transpose of the finite-difference Jacobian of F in C
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("d,k", [(1, 4), (2, 4), (4, 3)])
def test_adjoint_apply_is_transposed_fd_jacobian(d, k):
    W, C, _ = rand_problem(40, d, k, seed=55 + d)
    tau = 0.04
    _, _, S, F = R.final(W, C, tau)
    h = 1e-6
    J = np.zeros((k * d, k * d))
    for l in range(k):
        for b in range(d):
            Cp, Cm = C.copy(), C.copy()
            Cp[l, b] += h
            Cm[l, b] -= h
            J[:, l * d + b] = ((R.step(W, Cp, tau)[0] - R.step(W, Cm, tau)[0]) / (2 * h)).reshape(-1)
    rng = np.random.default_rng(1)
    for _ in range(3):
        u = rng.standard_normal((k, d))
        got = R.adjoint_apply(W, C, tau, S, F, u).reshape(-1)
        np.testing.assert_allclose(got, J.T @ u.reshape(-1), rtol=2e-7, atol=2e-7 * np.abs(J).max())
    # the dense analytic Jacobian agrees with the same finite differences
    Jd = dense.jacobians(W, C, tau)[0]
    np.testing.assert_allclose(Jd, J, rtol=2e-7, atol=2e-7 * np.abs(J).max())


# ----------------------------------------------------------------------------------------
# dense route (explicit Jacobians + LU) vs the iteration, plain and averaged (alpha = 0.25)
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,d,k,tau", [(40, 1, 4, 0.02), (36, 2, 4, 0.03), (32, 4, 8, 0.015)])
def test_dense_solve_matches_iteration(m, d, k, tau):
    W, C0, G = rand_problem(m, d, k, seed=3 * m + d)
    Ct = _converged(W, C0, tau)
    _, _, S, F = R.final(W, Ct, tau)
    dW_d, u_d, g_d = dense.gradients(W, G, Ct, tau, "implicit")
    np.testing.assert_allclose(R.codebook_grad(W, G, Ct, tau), g_d, rtol=1e-10, atol=1e-13)
    for alpha in (1.0, 0.25):
        dW, u, it, res = R.backward(W, G, Ct, tau, S, F, mode="implicit", alpha=alpha, adj_tol=1e-15,
                                    adj_max_iter=50000)
        assert res < 1e-13
        np.testing.assert_allclose(u, u_d, rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dW, dW_d, rtol=1e-9, atol=1e-12)
    dWj_d, uj_d, _ = dense.gradients(W, G, Ct, tau, "jfb")
    dWj, uj, it, _ = R.backward(W, G, Ct, tau, S, F, mode="jfb")
    assert it == 0
    np.testing.assert_allclose(uj, uj_d, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dWj, dWj_d, rtol=1e-10, atol=1e-13)
    # T adjoint iterations from u = g are the Neumann series to order T (Section 4.3)
    J = dense.jacobians(W, Ct, tau)[0]
    series, term = g_d.reshape(-1).copy(), g_d.reshape(-1).copy()
    for _ in range(4):
        term = J.T @ term
        series += term
    u4, it4, _ = R.adjoint_solve(W, Ct, tau, S, F, g_d, 1.0, 0.0, 4)
    assert it4 == 4
    np.testing.assert_allclose(u4.reshape(-1), series, rtol=1e-10, atol=1e-13)
    # J_C 1 + sum_i dF/dw_i = I_d per centroid (translation equivariance of F)
    _, dF_dW, _, _, _, _ = dense.jacobians(W, Ct, tau)
    tot = J.reshape(k, d, k, d).sum(2) + dF_dW.reshape(k, d, m, d).sum(2)
    np.testing.assert_allclose(tot, np.tile(np.eye(d), (k, 1, 1)), atol=1e-10)


# ----------------------------------------------------------------------------------------
# collapse criterion: at c_j = mean(W) (d = 1), J_C = (I - 11^T/k) MAD(W)/tau
# ----------------------------------------------------------------------------------------
def test_collapsed_point_jacobian_spectrum():
    rng = np.random.default_rng(9)
    W = rng.standard_normal((60, 1)) * 0.05
    k, tau = 4, 0.05
    mu = W.mean()
    C = np.full((k, 1), mu)
    _, _, S, F = R.final(W, C, tau)
    J = np.stack([R.adjoint_apply(W, C, tau, S, F, np.eye(k)[j].reshape(k, 1)).reshape(-1) for j in range(k)], 0)
    mad = np.abs(W - mu).mean()
    expect = (np.eye(k) - np.ones((k, k)) / k) * mad / tau
    np.testing.assert_allclose(J, expect, atol=1e-12)


# ----------------------------------------------------------------------------------------
# degenerate inputs: weight equal to a centroid (kink of the norm), dead cluster
# ----------------------------------------------------------------------------------------
def test_weight_on_centroid_uses_zero_subgradient():
    W = np.array([[0.0, 0.0], [1.0, 0.0], [0.0, 2.0]])
    C = np.array([[0.0, 0.0], [1.0, 1.0]])
    G = np.ones((3, 2))
    _, _, S, F = R.final(W, C, 0.5)
    dW, dC, _, _ = R.backward(W, G, C, 0.5, S, F, mode="jfb")
    assert np.all(np.isfinite(dW)) and np.all(np.isfinite(dC))
    dW_d, u_d, _ = dense.gradients(W, G, C, 0.5, "jfb")
    np.testing.assert_allclose(dW, dW_d, rtol=1e-12)
    np.testing.assert_allclose(dC, u_d, rtol=1e-12)


def test_dead_cluster_keeps_centroid():
    W = np.array([[0.0], [0.01], [0.02]])
    C = np.array([[0.01], [1e6]])
    Cp, S, dead = R.step(W, C, 1e-3)
    assert dead == 1 and S[1] < R.S_MIN
    assert Cp[1, 0] == 1e6
    np.testing.assert_allclose(Cp[0, 0], 0.01, rtol=1e-12)
    _, _, Sf, F = R.final(W, C, 1e-3)
    dW, dC, _, _ = R.backward(W, np.ones((3, 1)), C, 1e-3, Sf, F, mode="implicit", adj_max_iter=3)
    assert np.all(np.isfinite(dW)) and np.all(np.isfinite(dC))
