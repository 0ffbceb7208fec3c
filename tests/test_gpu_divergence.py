"""Backward robustness on the GPU (B200 only): the divergence status of the adjoint iteration, the restart with half
the averaging weight (Section 4.2) and the exact solve of the linear system on the explicit Jacobian.  Nothing here
faults or hangs a GPU: a diverging iteration is an ordinary computation whose numbers grow."""
import numpy as np
import pytest

from paper_2312_07759_b200 import workloads as WL
from parity_util import TOL_GRAD, assert_close

pytestmark = pytest.mark.gpu

# d = 1, k = 3, m = 7, centroids that are not a fixed point: dF/dC has the eigenvalue pair 0.84 +- 0.82 i (modulus
# 1.17), so alpha = 1 and alpha = 1/2 spiral outwards and alpha = 1/4 converges (tests/test_oracle_restart.py)
W7 = np.array([0.02958017587661743, 0.03282581642270088, 0.028027299791574478, -0.07381249964237213,
               0.07810479402542114, 0.12613466382026672, 0.01651347242295742], np.float32).reshape(7, 1)
C7 = np.array([0.0856543630361557, 0.037273112684488297, 0.022411182522773743], np.float32).reshape(3, 1)
TAU7 = float(np.float32(0.007819400168955326))


def _collapsed_case(k):
    """Centroids a hair apart around the weights' mean with tau at half their mean absolute deviation: dF/dC has
    the real eigenvalue MAD / tau = 2 there."""
    rng = np.random.default_rng(7)
    W = (rng.standard_normal((3000, 1)) * 0.05).astype(np.float32)
    mu = float(W.astype(np.float64).mean())
    C = (mu + np.linspace(-1e-6, 1e-6, k)).astype(np.float32).reshape(k, 1)
    tau = float(np.float32(0.5 * np.abs(W.astype(np.float64) - mu).mean()))
    G = rng.standard_normal(W.shape).astype(np.float32)
    return W, C, G, tau


@pytest.mark.parametrize("k,method", [(2, 0), (4, 0), (4, 1), (16, 0), (16, 1)])
def test_diverging_adjoint_is_reported_and_the_context_stays_usable(k, method):
    import torch
    from oracle import dense
    from oracle import idkm_ref as R
    from paper_2312_07759_b200 import binding as B
    W, C, G, tau = _collapsed_case(k)
    assert np.linalg.eigvals(dense.jacobians(W[:200].astype(np.float64), C.astype(np.float64), tau)[0]).real.max() > 1.5
    ctx = B.Context()
    ctx.set_adjoint_method(method)
    # a healthy problem first, to compare with afterwards
    good = WL.single_layer(20000, 1, k, 0.01, std=0.03, seed=3, max_iter=6, adj_max_iter=20)
    gW, gC0, gG = (torch.from_numpy(x).cuda() for x in (good.W, good.C0, good.G))
    ctx.forward(gW, gC0, good.tau, 0.0, good.max_iter)
    before = [t.cpu().numpy() for t in ctx.backward(gG, B.IMPLICIT, 0.0, good.adj_max_iter, 1.0)]
    assert ctx.info()[0].status == 0
    # the diverging one: loop switched off, the given centroids are the "returned" ones
    Wd, Cd, Gd = (torch.from_numpy(x).cuda() for x in (W, C, G))
    ctx.forward(Wd, Cd, tau, 0.0, 0)
    dW, dC = ctx.backward(Gd, B.IMPLICIT, 0.0, 500, 1.0)
    info = ctx.info()[0]
    assert info.status == B.ERR_DIVERGED, info
    assert 5 <= info.adj_iters < 100, info            # ||u|| doubles per step: 1e6 ||g|| after about 20
    assert "diverged" in B.status_string(B.ERR_DIVERGED)
    # the oracle's watch fires at the same step (within the rounding of the norm test)
    W64, C64, G64 = W.astype(np.float64), C.astype(np.float64), G.astype(np.float64)
    _, _, S, F = R.final(W64, C64, tau)
    g = R.codebook_grad(W64, G64, C64, tau)
    _, div, _, _, it_ref, _ = R.adjoint_solve_restart(W64, C64, tau, S, F, g, 1.0, 0, 0.0, 500)
    assert div and abs(it_ref - info.adj_iters) <= 2
    # tolerance mode reports it as well (the device ends the loop, the host stops queueing)
    ctx.backward(Gd, B.IMPLICIT, 1e-6, 500, 1.0)
    assert ctx.info()[0].status == B.ERR_DIVERGED
    # the context is as good as new: the healthy problem gives bitwise what it gave before
    ctx.forward(gW, gC0, good.tau, 0.0, good.max_iter)
    after = [t.cpu().numpy() for t in ctx.backward(gG, B.IMPLICIT, 0.0, good.adj_max_iter, 1.0)]
    assert ctx.info()[0].status == 0
    assert np.array_equal(before[0], after[0]) and np.array_equal(before[1], after[1])


@pytest.mark.parametrize("method", [0, 1])
def test_restart_with_half_the_alpha_rescues_a_spiralling_iteration(method):
    import torch
    from oracle import dense
    from oracle import idkm_ref as R
    from paper_2312_07759_b200 import binding as B
    rng = np.random.default_rng(3)
    G = rng.standard_normal(W7.shape).astype(np.float32)
    W64, C64, G64 = W7.astype(np.float64), C7.astype(np.float64), G.astype(np.float64)
    dW_ref, u_ref, _ = dense.gradients(W64, G64, C64, TAU7, "implicit")
    Wd, Cd, Gd = (torch.from_numpy(x).cuda() for x in (W7, C7, G))
    ctx = B.Context()
    ctx.set_adjoint_method(method)
    ctx.forward(Wd, Cd, TAU7, 0.0, 0)
    # alpha = 1 alone diverges
    ctx.backward(Gd, B.IMPLICIT, 1e-6, 6000, 1.0)
    assert ctx.info()[0].status == B.ERR_DIVERGED
    dW, dC, alpha, attempts = ctx.backward_restart(Gd, 1e-7, 6000, 1.0, 4)
    info = ctx.info()[0]
    assert info.status == 0 and alpha == 0.25 and attempts == 3, (info, alpha, attempts)
    assert info.adj_residual < 1e-7
    assert_close(dC.cpu().numpy(), u_ref, TOL_GRAD, "dC after the restart vs the dense solve")
    assert_close(dW.cpu().numpy(), dW_ref, TOL_GRAD, "dW after the restart vs the dense solve")
    # the oracle's policy takes the same decisions
    _, _, S, F = R.final(W64, C64, TAU7)
    g = R.codebook_grad(W64, G64, C64, TAU7)
    u_o, div, alpha_o, attempts_o, _, _ = R.adjoint_solve_restart(W64, C64, TAU7, S, F, g, 1.0, 4, 1e-7, 6000)
    assert not div and alpha_o == alpha and attempts_o == attempts
    assert_close(dC.cpu().numpy(), u_o, TOL_GRAD, "dC vs the oracle's restarted iteration")
    # not enough halvings: gives up, says so, still writes outputs
    _, _, alpha, attempts = ctx.backward_restart(Gd, 1e-7, 6000, 1.0, 1)
    assert ctx.info()[0].status == B.ERR_DIVERGED and alpha == 0.5 and attempts == 2
    # a healthy problem is left alone: one attempt at alpha0
    good = WL.single_layer(20000, 1, 3, 0.01, std=0.03, seed=3, max_iter=8, adj_max_iter=50)
    gW, gC0, gG = (torch.from_numpy(x).cuda() for x in (good.W, good.C0, good.G))
    ctx.forward(gW, gC0, good.tau, 0.0, good.max_iter)
    a = ctx.backward(gG, B.IMPLICIT, 0.0, 50, 1.0)
    b = ctx.backward_restart(gG, 0.0, 50, 1.0, 3)
    assert b[2] == 1.0 and b[3] == 1 and np.array_equal(a[0].cpu().numpy(), b[0].cpu().numpy())
    assert B.lib.idkm_backward_restart(ctx._h, gG.data_ptr(), 0.0, 5, 1.0, -1, None, None, ctx._ws.data_ptr(),
                                       ctx._ws.numel(), None, None, None) == B.ERR_PARAM


@pytest.mark.parametrize("m,d,k", [(200, 1, 4), (300, 2, 4), (250, 1, 16), (300, 4, 8), (280, 2, 32), (260, 4, 16),
                                   (240, 1, 64), (7, 1, 3)])
def test_exact_solve_matches_the_dense_route_of_the_oracle(m, d, k):
    """idkm_set_adjoint_method(2): (I - J^T) u = g solved on the device against explicit Jacobians + LU in float64
    (oracle/dense.py), at common centroids; also where the iteration would not converge (the last case)."""
    import torch
    from oracle import dense
    from oracle import idkm_ref as R
    from paper_2312_07759_b200 import binding as B
    if m == 7:
        W, C, tau = W7, C7, TAU7
        G = np.random.default_rng(3).standard_normal(W.shape).astype(np.float32)
    else:
        wl = WL.single_layer(m, d, k, 0.012, std=0.03, seed=m + k, init="rows", g_std=0.5)
        W, G, tau = wl.W, wl.G, wl.tau
        C = R.forward(W.astype(np.float64), wl.C0.astype(np.float64), tau, 0.0, 25)[0].astype(np.float32)
    W64, C64, G64 = W.astype(np.float64), C.astype(np.float64), G.astype(np.float64)
    dW_ref, u_ref, _ = dense.gradients(W64, G64, C64, tau, "implicit")
    ctx = B.Context()
    ctx.set_adjoint_method(2)
    assert B.describe_path(d, k, 10, 2)["adjoint_route"] == "exact solve on the explicit Jacobian"
    ctx.forward(torch.from_numpy(W).cuda(), torch.from_numpy(C).cuda(), tau, 0.0, 0)
    n0 = ctx.launches
    dW, dC = ctx.backward(torch.from_numpy(G).cuda(), B.IMPLICIT, 0.0, 10, 1.0)
    info = ctx.info()[0]
    assert info.status == 0 and info.adj_iters == 0 and ctx.launches - n0 == 3      # g, the matrix + solve, dL/dW
    # (I - J^T)^-1 amplifies the fp32 rounding of J by the conditioning of the system
    cond = np.linalg.cond(np.eye(k * d) - dense.jacobians(W64, C64, tau)[0].T)
    tol = max(TOL_GRAD, 2e-6 * cond)
    assert tol < 5e-3, cond
    assert_close(dC.cpu().numpy(), u_ref, tol, f"dC, condition number {cond:.1f}")
    assert_close(dW.cpu().numpy(), dW_ref, tol, f"dW, condition number {cond:.1f}")


def test_exact_solve_on_larger_layers_equals_the_converged_iteration():
    """Where the iteration on the explicit matrix converges, the exact solve gives its limit; where it does not (the
    centroids after 40 steps need not be near a fixed point), the exact solve still returns a finite answer."""
    import torch
    from paper_2312_07759_b200 import binding as B
    compared = 0
    for (m, d, k) in [(60000, 1, 8), (50000, 2, 16), (40000, 4, 16), (30000, 1, 64), (80000, 1, 4), (70000, 2, 4)]:
        wl = WL.single_layer(m, d, k, 0.012, std=0.03, seed=m + k, max_iter=40, init="rows", g_std=0.5)
        W, C0, G = (torch.from_numpy(x).cuda() for x in (wl.W, wl.C0, wl.G))
        res, status = {}, {}
        for method in (0, 2):
            ctx = B.Context()
            ctx.set_adjoint_method(method)
            ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter)
            dW, dC = ctx.backward(G, B.IMPLICIT, 1e-10, 200000, 1.0)      # both run on the explicit matrix in fp64
            status[method] = ctx.info()[0].status
            res[method] = (dW.cpu().numpy(), dC.cpu().numpy())
        assert status[2] == 0 and np.all(np.isfinite(res[2][0])) and np.all(np.isfinite(res[2][1])), (m, d, k)
        assert status[0] in (0, B.ERR_DIVERGED), (m, d, k, status[0])
        if status[0] == 0:
            compared += 1
            assert_close(res[2][1], res[0][1], 2e-5, f"dC {m, d, k}")
            assert_close(res[2][0], res[0][0], 2e-5, f"dW {m, d, k}")
    assert compared >= 2
    # a codebook too large for the explicit matrix falls back to the fused iteration
    assert B.describe_path(4, 256, 10, 2)["adjoint_route"] == "fused passes"
