"""A compact battery of oracle pins that takes the oracle module as an argument, so that the same checks can be
run against deliberately broken copies of the oracle (tests/test_oracle_mutations.py).  Each check uses only
closed forms, brute-force definitions or finite differences of the forward map.

The battery runs in two settings: the method as published (Euclidean distance in the softmax) and the
squared-distance variant (``SQ[0] = True`` while the oracle is switched with ``R.squared_distance()``).  Checks that
spell out a distance or a closed form read ``SQ[0]``; the others only call the oracle and hold in both settings."""
import numpy as np

SQ = [False]     # which setting the battery is running in


def _dist(x):
    """The distance of the setting, from a difference vector."""
    return float(np.dot(x, x)) if SQ[0] else float(np.linalg.norm(x))


def _theta(a, c, tau):
    """Half the logit gap between the two centroids +-c seen from the weight +a: D(a, -c) - D(a, c) = 2 tau theta."""
    return 2 * a * c / tau if SQ[0] else c / tau


def _fixed_point_tanh(a, tau):
    """Non-zero solution of c = a tanh(theta(a, c)) by bisection (exists when the slope at 0 exceeds 1)."""
    lo, hi = 1e-12, a
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if a * np.tanh(_theta(a, mid, tau)) - mid > 0:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def check_bruteforce_attention(R):
    rng = np.random.default_rng(1)
    W, C, tau = rng.standard_normal((30, 2)) * 0.05, rng.standard_normal((4, 2)) * 0.05, 0.03
    if SQ[0]:
        tau = 0.002
    A = R.attention(W, C, tau)
    for i in range(30):
        e = np.array([np.exp(-_dist(W[i] - C[j]) / tau) for j in range(4)])
        np.testing.assert_allclose(A[i], e / e.sum(), rtol=1e-12)


def check_matrix_m_step(R):
    rng = np.random.default_rng(2)
    W, C, tau = rng.standard_normal((64, 2)) * 0.05, rng.standard_normal((4, 2)) * 0.05, 0.04
    D = np.linalg.norm(W[:, None] - C[None], axis=-1)
    if SQ[0]:
        D, tau = D * D, 0.003
    E = np.exp(-D / tau)
    A = E / E.sum(1, keepdims=True)
    np.testing.assert_allclose(R.step(W, C, tau)[0], np.diag(1 / A.sum(0)) @ A.T @ W, rtol=1e-12)
    Wq, _, S, F = R.final(W, C, tau)
    np.testing.assert_allclose(Wq, A @ C, rtol=1e-12)
    np.testing.assert_allclose(S, A.sum(0), rtol=1e-12)
    np.testing.assert_allclose(F, (A.T @ W) / A.sum(0)[:, None], rtol=1e-12)


def check_two_point_closed_form(R):
    """Weights -a, +a (repeated), centroids -c, +c: the iterate stays symmetric and c+ = a tanh(theta), with
    theta = c / tau for the Euclidean distance and 2 a c / tau for the squared one; Wq(+a) = c tanh(theta).  Moving
    the weights apart (a -> a + eps, i.e. along G = (-1, +1)) gives d<G, Wq>/d eps in closed form: with
    T = tanh(theta) + theta sech^2(theta) (= dWq/dc at fixed a), dWq/da at fixed c = (dtheta/da) c sech^2(theta) and
    c' = dc*/da either from differentiating the fixed-point equation (implicit) or of one application (JFB)."""
    a, tau, reps = 0.05, 0.02, 8
    if SQ[0]:
        tau = 0.002          # slope of c -> a tanh(2 a c / tau) at 0 is 2 a^2 / tau = 2.5 > 1
    W = np.array([[-a], [a]] * reps)
    cs = _fixed_point_tanh(a, tau)
    Ct, _, _, _ = R.forward(W, np.array([[-0.03], [0.03]]), tau, 1e-15, 3000)
    np.testing.assert_allclose(Ct[:, 0], [-cs, cs], rtol=1e-10)
    Wq, _, S, F = R.final(W, Ct, tau)
    theta = _theta(a, cs, tau)
    th, sech2 = np.tanh(theta), 1 / np.cosh(theta) ** 2
    np.testing.assert_allclose(Wq[1, 0], cs * th, rtol=1e-10)
    G = np.array([[-1.0], [1.0]] * reps)
    T = th + theta * sech2
    dtheta_da, dtheta_dc = (2 * cs / tau, 2 * a / tau) if SQ[0] else (0.0, 1 / tau)
    direct = dtheta_da * cs * sech2                     # dWq/da at fixed c
    one_step = th + a * sech2 * dtheta_da               # d(a tanh theta)/da at fixed c
    for mode, cprime in (("implicit", one_step / (1 - a * sech2 * dtheta_dc)), ("jfb", one_step)):
        dW, _, _, _ = R.backward(W, G, Ct, tau, S, F, mode=mode, adj_tol=1e-15, adj_max_iter=5000)
        np.testing.assert_allclose(float((dW * G).sum()), 2 * reps * (direct + cprime * T), rtol=1e-8)


def check_single_centroid(R):
    rng = np.random.default_rng(3)
    W, G = rng.standard_normal((21, 2)), rng.standard_normal((21, 2))
    Ct, _, _, _ = R.forward(W, rng.standard_normal((1, 2)), 0.1, 0.0, 2)
    np.testing.assert_allclose(Ct[0], W.mean(0), rtol=1e-12)
    _, _, S, F = R.final(W, Ct, 0.1)
    for mode in ("implicit", "jfb"):
        dW, dC, _, _ = R.backward(W, G, Ct, 0.1, S, F, mode=mode, adj_max_iter=4)
        np.testing.assert_allclose(dW, np.tile(G.mean(0), (21, 1)), rtol=1e-11, atol=1e-14)
        np.testing.assert_allclose(dC[0], G.sum(0), rtol=1e-11)


def check_implicit_gradient_fd(R):
    rng = np.random.default_rng(4)
    m, d, k, tau = 36, 2, 3, 0.03
    if SQ[0]:
        tau = 0.004
    W = rng.standard_normal((m, d)) * 0.05
    C0 = W[:k] + 0.002
    G = rng.standard_normal((m, d))

    def conv(Wp, Cs):
        return R.forward(Wp, Cs, tau, 1e-15, 20000)[0]

    Ct = conv(W, C0)
    _, _, S, F = R.final(W, Ct, tau)
    dW, _, _, _ = R.backward(W, G, Ct, tau, S, F, mode="implicit", adj_tol=1e-15, adj_max_iter=20000)
    h = 1e-6
    for (i, a) in ((0, 0), (5, 1), (17, 0), (30, 1)):
        Wp, Wm = W.copy(), W.copy()
        Wp[i, a] += h
        Wm[i, a] -= h
        fd = (float((G * R.final(Wp, conv(Wp, Ct), tau)[0]).sum()) - float((G * R.final(Wm, conv(Wm, Ct), tau)[0]).sum())) / (2 * h)
        assert abs(fd - dW[i, a]) <= 2e-6 * max(1.0, np.abs(dW).max()), (i, a, fd, dW[i, a])
    np.testing.assert_allclose(dW.sum(0), G.sum(0), rtol=1e-8, atol=1e-9)


def check_jfb_one_step_derivative(R):
    rng = np.random.default_rng(5)
    m, d, k, tau = 20, 2, 3, 0.05
    if SQ[0]:
        tau = 0.005
    W = rng.standard_normal((m, d)) * 0.05
    Cb = W[:k] + 0.003
    G = rng.standard_normal((m, d))
    _, _, S, F = R.final(W, Cb, tau)
    dW, dC, _, _ = R.backward(W, G, Cb, tau, S, F, mode="jfb")
    F0 = R.step(W, Cb, tau)[0]
    h = 1e-6
    for (i, a) in ((0, 0), (7, 1), (13, 0)):
        Wp, Wm = W.copy(), W.copy()
        Wp[i, a] += h
        Wm[i, a] -= h
        Hp = float((G * R.final(Wp, Cb + R.step(Wp, Cb, tau)[0] - F0, tau)[0]).sum())
        Hm = float((G * R.final(Wm, Cb + R.step(Wm, Cb, tau)[0] - F0, tau)[0]).sum())
        assert abs((Hp - Hm) / (2 * h) - dW[i, a]) <= 1e-6 * max(1.0, np.abs(dW).max())
    for (j, a) in ((0, 0), (2, 1)):
        Cp, Cm = Cb.copy(), Cb.copy()
        Cp[j, a] += h
        Cm[j, a] -= h
        fd = float((G * (R.final(W, Cp, tau)[0] - R.final(W, Cm, tau)[0])).sum()) / (2 * h)
        assert abs(fd - dC[j, a]) <= 1e-6 * max(1.0, np.abs(dC).max())


def check_adjoint_is_transposed_fd_jacobian(R):
    rng = np.random.default_rng(6)
    d, k, tau = 2, 3, 0.04
    if SQ[0]:
        tau = 0.004
    W = rng.standard_normal((30, d)) * 0.05
    C = W[:k] + 0.004
    _, _, S, F = R.final(W, C, tau)
    h = 1e-6
    J = np.zeros((k * d, k * d))
    for l in range(k):
        for b in range(d):
            Cp, Cm = C.copy(), C.copy()
            Cp[l, b] += h
            Cm[l, b] -= h
            J[:, l * d + b] = ((R.step(W, Cp, tau)[0] - R.step(W, Cm, tau)[0]) / (2 * h)).reshape(-1)
    u = rng.standard_normal((k, d))
    np.testing.assert_allclose(R.adjoint_apply(W, C, tau, S, F, u).reshape(-1), J.T @ u.reshape(-1), rtol=2e-7,
                               atol=2e-7 * np.abs(J).max())
    # averaged iteration (alpha = 0.25) reaches the same limit as the dense solve with the FD Jacobian
    g = rng.standard_normal((k, d))
    if np.abs(np.linalg.eigvals(J)).max() < 0.95:
        uu, _, res = R.adjoint_solve(W, C, tau, S, F, g, 0.25, 1e-14, 20000)
        np.testing.assert_allclose(uu.reshape(-1), np.linalg.solve(np.eye(k * d) - J.T, g.reshape(-1)), rtol=1e-5)


def check_lloyd_limit(R):
    rng = np.random.default_rng(7)
    centers = rng.standard_normal((3, 2))
    W = np.concatenate([c + 0.05 * rng.standard_normal((10, 2)) for c in centers])
    C = centers + 0.02 * rng.standard_normal((3, 2))
    lab = np.argmin(((W[:, None] - C[None]) ** 2).sum(-1), 1)
    hard = np.stack([W[lab == j].mean(0) for j in range(3)])
    np.testing.assert_allclose(R.step(W, C, 1e-5)[0], hard, rtol=1e-9)


CHECKS = [check_bruteforce_attention, check_matrix_m_step, check_two_point_closed_form, check_single_centroid,
          check_implicit_gradient_fd, check_jfb_one_step_derivative, check_adjoint_is_transposed_fd_jacobian,
          check_lloyd_limit]


def run_battery(R, squared=False):
    """Names of the checks that fail for this oracle module, in the published setting or the squared-distance one."""
    failed = []
    SQ[0] = bool(squared)
    try:
        with R.squared_distance(bool(squared)):
            for chk in CHECKS:
                try:
                    chk(R)
                except Exception:   # an assertion, or a numerical blow-up caused by the planted mistake
                    failed.append(chk.__name__)
    finally:
        SQ[0] = False
    return failed
