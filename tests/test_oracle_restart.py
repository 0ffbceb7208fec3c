"""The adjoint iteration's divergence watch and the restart with half the averaging weight (Section 4.2): pinned on
a problem whose Jacobian dF/dC has a complex eigenvalue pair of modulus 1.17 (found by a random search over small
problems at not-yet-converged centroids; inputs below are that case, rounded to fp32), where the plain iteration and
alpha = 1/2 spiral outwards and alpha = 1/4 converges to the solution of the linear system.  CPU only."""
import numpy as np

from oracle import dense
from oracle import idkm_ref as R

# d = 1, k = 3, m = 7: weights, centroids (not a fixed point), temperature
W = np.array([0.02958017587661743, 0.03282581642270088, 0.028027299791574478, -0.07381249964237213,
              0.07810479402542114, 0.12613466382026672, 0.01651347242295742]).reshape(7, 1)
C = np.array([0.0856543630361557, 0.037273112684488297, 0.022411182522773743]).reshape(3, 1)
TAU = 0.007819400168955326


def _setup():
    rng = np.random.default_rng(3)
    G = rng.standard_normal(W.shape)
    _, _, S, F = R.final(W, C, TAU)
    g = R.codebook_grad(W, G, C, TAU)
    J = dense.jacobians(W, C, TAU)[0]
    return G, S, F, g, J


def test_the_case_has_a_complex_pair_outside_the_unit_circle_that_damping_brings_inside():
    _, _, _, _, J = _setup()
    ev = np.linalg.eigvals(J)
    assert np.abs(ev).max() > 1.1 and ev.real.max() < 1.0 and np.abs(ev.imag).max() > 0.5
    assert np.abs(0.5 * ev + 0.5).max() > 1.0          # alpha = 1/2 still diverges
    assert np.abs(0.25 * ev + 0.75).max() < 0.99       # alpha = 1/4 converges


def test_restart_halves_alpha_until_the_iteration_converges_to_the_dense_solution():
    G, S, F, g, J = _setup()
    u, diverged, alpha, attempts, iters, res = R.adjoint_solve_restart(W, C, TAU, S, F, g, 1.0, 4, 1e-12, 20000)
    assert not diverged and alpha == 0.25 and attempts == 3 and res < 1e-12
    exact = np.linalg.solve(np.eye(3) - J.T, g.reshape(-1))
    np.testing.assert_allclose(u.reshape(-1), exact, rtol=1e-9)
    # without enough halvings it gives up and says so
    _, diverged, alpha, attempts, _, _ = R.adjoint_solve_restart(W, C, TAU, S, F, g, 1.0, 1, 1e-12, 20000)
    assert diverged and alpha == 0.5 and attempts == 2


def test_watch_leaves_a_converging_iteration_alone():
    rng = np.random.default_rng(5)
    Wc = rng.standard_normal((60, 2)) * 0.05
    Cc = R.forward(Wc, Wc[:3].copy(), 0.02, 1e-14, 20000)[0]
    Gc = rng.standard_normal(Wc.shape)
    _, _, S, F = R.final(Wc, Cc, 0.02)
    g = R.codebook_grad(Wc, Gc, Cc, 0.02)
    u0, it0, res0 = R.adjoint_solve(Wc, Cc, 0.02, S, F, g, 1.0, 1e-13, 5000)
    u1, diverged, alpha, attempts, it1, res1 = R.adjoint_solve_restart(Wc, Cc, 0.02, S, F, g, 1.0, 3, 1e-13, 5000)
    assert not diverged and alpha == 1.0 and attempts == 1 and it1 == it0
    assert np.array_equal(u0, u1)


def test_no_alpha_rescues_a_real_eigenvalue_above_one():
    """At the collapsed point dF/dC = (I - 11^T/k) MAD/tau (real, symmetric): with tau below the weights' mean absolute
    deviation the eigenvalue exceeds 1 and alpha lambda + 1 - alpha stays above 1 for every alpha in (0, 1]."""
    rng = np.random.default_rng(7)
    Wc = rng.standard_normal((50, 1)) * 0.05
    mu = Wc.mean()
    Cc = np.array([[mu - 1e-7], [mu + 1e-7]])
    tau = 0.5 * np.abs(Wc - mu).mean()
    Gc = rng.standard_normal(Wc.shape)
    _, _, S, F = R.final(Wc, Cc, tau)
    g = R.codebook_grad(Wc, Gc, Cc, tau)
    assert np.linalg.eigvals(dense.jacobians(Wc, Cc, tau)[0]).real.max() > 1.5
    _, diverged, alpha, attempts, _, _ = R.adjoint_solve_restart(Wc, Cc, tau, S, F, g, 1.0, 5, 1e-12, 5000)
    assert diverged and attempts == 6 and alpha == 1.0 / 32
