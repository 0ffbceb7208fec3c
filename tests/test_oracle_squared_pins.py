"""Pins of the oracle's squared-distance variant (softmax of -||w - c||^2 / tau, the distance the clustering
objectives of Sections 3.1 and 3.2 are written in) against closed forms, brute force, finite differences of the
forward map and the dense linear-algebra route.  The battery of tests/pin_battery.py runs in this setting too
(tests/test_oracle_mutations.py); the checks here are the ones particular to the variant."""
import numpy as np
import pytest

from oracle import dense
from oracle import idkm_ref as R


@pytest.fixture(autouse=True)
def squared_setting():
    with R.squared_distance():
        yield
    assert R.get_squared() is False


def rand_problem(m, d, k, scale=0.05, seed=0):
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((m, d)) * scale
    C = W[rng.choice(m, k, replace=False)] + rng.standard_normal((k, d)) * scale * 0.05
    G = rng.standard_normal((m, d))
    return W, C, G


@pytest.mark.parametrize("d,k", [(1, 2), (1, 4), (2, 4), (4, 8)])
def test_attention_is_the_softmax_of_minus_squared_distance(d, k):
    W, C, _ = rand_problem(40, d, k, seed=d + 3 * k)
    tau = 0.002
    A = R.attention(W, C, tau)
    np.testing.assert_allclose(A.sum(1), 1.0, atol=1e-14)
    for i in range(W.shape[0]):
        e = np.array([np.exp(-np.dot(W[i] - C[j], W[i] - C[j]) / tau) for j in range(k)])
        np.testing.assert_allclose(A[i], e / e.sum(), rtol=1e-12)
    # and it is NOT the published attention at the same temperature
    with R.squared_distance(False):
        assert np.abs(R.attention(W, C, tau) - A).max() > 1e-3


def test_attention_is_a_gaussian_mixture_posterior():
    """exp(-||w - c_j||^2 / tau) / sum is the posterior of an equal-weight mixture of isotropic Gaussians with
    variance tau / 2: checked against scipy's normal density."""
    from scipy.stats import multivariate_normal
    W, C, _ = rand_problem(25, 2, 3, seed=9)
    tau = 0.003
    dens = np.stack([multivariate_normal(mean=C[j], cov=(tau / 2) * np.eye(2)).pdf(W) for j in range(3)], 1)
    np.testing.assert_allclose(R.attention(W, C, tau), dens / dens.sum(1, keepdims=True), rtol=1e-10)


def test_scaling_equivariance_uses_the_square_of_the_scale():
    """F(sC, sW; s^2 tau) = s F(C, W; tau) for the squared distance (s tau for the published one)."""
    W, C, _ = rand_problem(80, 2, 4, seed=4)
    tau, s = 0.002, 3.7
    np.testing.assert_allclose(R.step(s * W, s * C, s * s * tau)[0], s * R.step(W, C, tau)[0], rtol=1e-12)
    t = np.array([0.3, -0.2])
    np.testing.assert_allclose(R.step(W + t, C + t, tau)[0], R.step(W, C, tau)[0] + t, rtol=1e-11, atol=1e-14)


@pytest.mark.parametrize("d,k,m", [(1, 3, 24), (2, 3, 30), (4, 4, 40)])
def test_iteration_matches_the_dense_solve(d, k, m):
    """Vector-Jacobian iteration of the oracle against explicit Jacobians and an LU solve (oracle/dense.py), both in
    the squared setting, at a converged fixed point."""
    W, C0, G = rand_problem(m, d, k, seed=10 * d + k)
    tau = 0.004
    Ct = R.forward(W, C0, tau, 1e-15, 20000)[0]
    np.testing.assert_allclose(dense.fixed_point_map(W, Ct, tau, squared=True)[0], Ct, rtol=1e-10, atol=1e-13)
    _, _, S, F = R.final(W, Ct, tau)
    J = dense.jacobians(W, Ct, tau, squared=True)[0]
    rho = np.abs(np.linalg.eigvals(J)).max()
    assert rho < 1.0
    dW_d, u_d, g_d = dense.gradients(W, G, Ct, tau, "implicit", squared=True)
    np.testing.assert_allclose(R.codebook_grad(W, G, Ct, tau), g_d, rtol=1e-9, atol=1e-12)
    u = rng_u = np.random.default_rng(1).standard_normal((k, d))
    np.testing.assert_allclose(R.adjoint_apply(W, Ct, tau, S, F, u).reshape(-1), J.T @ rng_u.reshape(-1), rtol=1e-9,
                               atol=1e-12)
    dW, dC, _, _ = R.backward(W, G, Ct, tau, S, F, mode="implicit", adj_tol=1e-15, adj_max_iter=200000)
    np.testing.assert_allclose(dC, u_d, rtol=1e-7, atol=1e-10)
    np.testing.assert_allclose(dW, dW_d, rtol=1e-7, atol=1e-10)
    dWj, dCj, _, _ = R.backward(W, G, Ct, tau, S, F, mode="jfb")
    dW_dj, u_dj, _ = dense.gradients(W, G, Ct, tau, "jfb", squared=True)
    np.testing.assert_allclose(dWj, dW_dj, rtol=1e-9, atol=1e-12)
    # translation equivariance of Wq: the implicit gradient sums to the upstream gradient's sum, JFB's does not
    np.testing.assert_allclose(dW.sum(0), G.sum(0), rtol=1e-7, atol=1e-9)


def test_gradient_is_continuous_where_a_weight_sits_on_a_centroid():
    """The squared distance has no kink: moving a centroid across a weight changes the gradients smoothly (for the
    published distance, d = 1, the same move flips sign(w - c) and the gradient jumps)."""
    rng = np.random.default_rng(2)
    W = np.sort(rng.standard_normal((40, 1)) * 0.05, axis=0)
    G = rng.standard_normal((40, 1))
    tau, h = 0.003, 1e-9
    base = np.array([[-0.04], [0.0], [0.04]])
    out = []
    for sign in (-1, +1):
        C = base.copy()
        C[1, 0] = W[20, 0] + sign * h          # just left / just right of a weight
        _, _, S, F = R.final(W, C, tau)
        out.append(R.backward(W, G, C, tau, S, F, mode="jfb")[0])
    assert np.abs(out[0] - out[1]).max() < 1e-5 * np.abs(out[0]).max()
    with R.squared_distance(False):
        outp = []
        for sign in (-1, +1):
            C = base.copy()
            C[1, 0] = W[20, 0] + sign * h
            _, _, S, F = R.final(W, C, 0.05)
            outp.append(R.backward(W, G, C, 0.05, S, F, mode="jfb")[0])
        assert np.abs(outp[0] - outp[1]).max() > 1e-3 * np.abs(outp[0]).max()


def test_temperature_schedule_with_warm_starts_ends_at_a_fixed_point_of_the_last_temperature():
    """Annealing (the paper's closing remark: a higher temperature first, then lower): each stage starts from the
    previous stage's centroids; the end result is a fixed point of the map at the final temperature, and differs
    from the cold start's by no more than two local optima can."""
    W, C0, _ = rand_problem(300, 2, 4, seed=6)
    C = C0
    for tau in (0.02, 0.008, 0.003):
        C = R.forward(W, C, tau, 1e-14, 50000)[0]
    np.testing.assert_allclose(R.step(W, C, 0.003)[0], C, rtol=1e-9, atol=1e-12)
    assert np.all(C >= W.min(0)) and np.all(C <= W.max(0))
