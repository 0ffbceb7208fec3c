"""The oracle-side unrolled (DKM-style) gradient: pinned by finite differences of the T-step loop, tied to the
implicit gradient in the converged limit, and used to report how far the implicit and Jacobian-free gradients are
from the true derivative of the truncated loop on the first benchmark configuration.  CPU only."""
import numpy as np
import pytest

from oracle import idkm_ref as R
from oracle import unrolled as U
from paper_2312_07759_b200 import workloads as WL


def _loss(W, G, C0, tau, T):
    CT = U.forward_iterates(W, C0, tau, T)[-1]
    return float((G * R.final(W, CT, tau)[0]).sum())


@pytest.mark.parametrize("d,k,m,T", [(1, 3, 40, 1), (1, 3, 40, 4), (2, 4, 48, 3), (4, 3, 30, 6), (2, 2, 64, 12)])
def test_unrolled_gradient_matches_finite_differences_of_the_truncated_loop(d, k, m, T):
    rng = np.random.default_rng(100 * d + 10 * k + T)
    W = rng.standard_normal((m, d)) * 0.05
    C0 = W[rng.choice(m, k, replace=False)] + 0.004 * rng.standard_normal((k, d))
    G = rng.standard_normal((m, d))
    tau = 0.03
    dW, dC0, CT = U.gradients(W, G, C0, tau, T)
    h = 1e-6
    scale = max(1.0, np.abs(dW).max())
    for (i, a) in ((0, 0), (m // 3, d - 1), (m - 1, 0)):
        Wp, Wm = W.copy(), W.copy()
        Wp[i, a] += h
        Wm[i, a] -= h
        fd = (_loss(Wp, G, C0, tau, T) - _loss(Wm, G, C0, tau, T)) / (2 * h)
        assert abs(fd - dW[i, a]) <= 2e-6 * scale, (i, a, fd, dW[i, a])
    for (j, a) in ((0, 0), (k - 1, d - 1)):
        Cp, Cm = C0.copy(), C0.copy()
        Cp[j, a] += h
        Cm[j, a] -= h
        fd = (_loss(W, G, Cp, tau, T) - _loss(W, G, Cm, tau, T)) / (2 * h)
        assert abs(fd - dC0[j, a]) <= 2e-6 * max(1.0, np.abs(dC0).max()), (j, a, fd, dC0[j, a])


def test_zero_iterations_leave_only_the_direct_terms():
    rng = np.random.default_rng(3)
    W, G = rng.standard_normal((30, 2)) * 0.05, rng.standard_normal((30, 2))
    C0 = W[:3] + 0.003
    dW, dC0, CT = U.gradients(W, G, C0, 0.03, 0)
    assert np.array_equal(CT, C0)
    np.testing.assert_allclose(dC0, R.codebook_grad(W, G, C0, 0.03), rtol=1e-13)
    _, _, S, F = R.final(W, C0, 0.03)
    np.testing.assert_allclose(dW, R.scatter(W, G, C0, 0.03, S, F, np.zeros_like(C0)), rtol=1e-13)


def test_unrolled_gradient_tends_to_the_implicit_gradient_as_the_loop_converges():
    """At a contraction the sensitivity to C_0 dies out and the sum over iterations becomes the Neumann series of
    (I - dF/dC)^-1 (Section 4.3), i.e. the implicit gradient at the fixed point."""
    rng = np.random.default_rng(5)
    W = rng.standard_normal((60, 2)) * 0.05
    G = rng.standard_normal((60, 2))
    C0 = W[rng.choice(60, 3, replace=False)]
    tau = 0.02
    errs = []
    for T in (5, 20, 80, 320):
        dW, dC0, CT = U.gradients(W, G, C0, tau, T)
        _, _, S, F = R.final(W, CT, tau)
        dWi = R.backward(W, G, CT, tau, S, F, mode="implicit", adj_tol=1e-15, adj_max_iter=100000)[0]
        errs.append(np.linalg.norm(dW - dWi) / np.linalg.norm(dWi))
    assert errs[-1] < 1e-9 and errs[0] > errs[1] > errs[2] > errs[3], errs
    assert np.abs(dC0).max() < 1e-9 * np.abs(G).max() * 60


def _compare(wl, Ts):
    W, G, C0 = wl.W.astype(np.float64), wl.G.astype(np.float64), wl.C0.astype(np.float64)
    rows = []
    for T in Ts:
        dWu, _, CT = U.gradients(W, G, C0, wl.tau, T)
        _, _, S, F = R.final(W, CT, wl.tau)
        dWi = R.backward(W, G, CT, wl.tau, S, F, mode="implicit", adj_max_iter=T)[0]
        dWj = R.backward(W, G, CT, wl.tau, S, F, mode="jfb")[0]
        nu = np.linalg.norm(dWu)
        res = np.linalg.norm(R.step(W, CT, wl.tau)[0] - CT) / np.linalg.norm(CT)
        rows.append((T, res, np.linalg.norm(dWi - dWu) / nu, np.linalg.norm(dWj - dWu) / nu))
    return rows


def test_report_implicit_and_jfb_against_unrolled_on_configs_1_and_2(capsys):
    """How far the two IDKM gradients are from the true derivative of the truncated loop, as the iteration count T
    grows (implicit: T adjoint steps; both evaluated at C_T).  First configuration (m = 4096 scalars, k = 4,
    tau = 0.05 above the weights' mean absolute deviation): the centroids slide into the mean, every gradient tends to
    the same trivial one and the three agree ever better.  Second configuration (a 64x64x3x3 layer, k = 8, tau = 0.01:
    separated clusters, contraction rate about 0.92): the implicit gradient closes in on the unrolled one at that
    rate while the Jacobian-free one keeps the error of dropping (I - dF/dC)^-1.  Printed, and checked only for what
    must hold."""
    r1 = _compare(WL.config1(), (5, 15, 30, 60))
    r2 = _compare(WL.config2(), (5, 15, 30, 60, 120))
    with capsys.disabled():
        for name, rows in (("configuration 1", r1), ("configuration 2", r2)):
            print(f"\n{name}:  T   ||F(C_T) - C_T|| / ||C_T||   ||implicit - unrolled|| / ||unrolled||   "
                  "||jfb - unrolled|| / ||unrolled||")
            for T, res, ei, ej in rows:
                print(f"{T:20d}   {res:.3e}   {ei:.3e}   {ej:.3e}")
    assert all(np.isfinite(x) for rows in (r1, r2) for r in rows for x in r)
    # collapsing case: all three gradients merge
    assert r1[-1][2] < 1e-6 and r1[-1][3] < 1e-6
    # separated case: the implicit gradient converges to the unrolled one, the Jacobian-free one does not
    assert r2[-1][2] < 1e-2 * r2[-1][3] and r2[-1][2] < r2[0][2]
