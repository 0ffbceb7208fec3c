"""Argument checking and host-buffer entry point of the C-ABI library (B200 only)."""
import numpy as np
import pytest

from paper_2312_07759_b200 import workloads as WL
from parity_util import TOL_C, TOL_GRAD, assert_close, at_centroids, oracle_backward_at, oracle_run

pytestmark = pytest.mark.gpu


def test_argument_errors():
    import torch
    from paper_2312_07759_b200 import binding as B
    ctx = B.Context()
    dev = torch.device("cuda:0")
    W = torch.zeros(1024, 1, device=dev)
    C0 = torch.zeros(4, 1, device=dev)
    Co = torch.zeros(4, 1, device=dev)
    nbytes = B.workspace_bytes(1024, 1, 4, 1)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    args = dict(W=W.data_ptr(), m=1024, d=1, C0=C0.data_ptr(), k=4, tau=0.1, tol=0.0, max_iter=2,
                C_out=Co.data_ptr(), A_out=None, Wq_out=None, ws=ws.data_ptr(), ws_bytes=nbytes)

    def fwd(**kw):
        a = dict(args)
        a.update(kw)
        return ctx.forward_raw(**a)

    # backward before any forward
    assert ctx.backward_raw(W.data_ptr(), B.IMPLICIT, 0.0, 1, 1.0, None, None, ws.data_ptr(), nbytes) == B.ERR_ORDER
    assert fwd(W=None) == B.ERR_NULL
    assert fwd(W=W.data_ptr() + 4) == B.ERR_ALIGN
    assert fwd(m=0) == B.ERR_SHAPE
    assert fwd(d=3) == B.ERR_UNSUPPORTED
    assert fwd(k=257) == B.ERR_UNSUPPORTED
    assert fwd(k=0) == B.ERR_UNSUPPORTED
    assert fwd(tau=0.0) == B.ERR_PARAM
    assert fwd(tau=float("nan")) == B.ERR_PARAM
    assert fwd(tol=-1.0) == B.ERR_PARAM
    assert fwd(max_iter=-1) == B.ERR_PARAM
    assert fwd(ws_bytes=nbytes - 1) == B.ERR_WORKSPACE
    assert fwd() == B.OK
    G = torch.zeros(1024, 1, device=dev)
    dW = torch.zeros(1024, 1, device=dev)
    bw = lambda **kw: ctx.backward_raw(**{**dict(dWq=G.data_ptr(), mode=B.IMPLICIT, adj_tol=0.0, adj_max_iter=1,
                                                 alpha=1.0, dW_out=dW.data_ptr(), dC_out=None, ws=ws.data_ptr(),
                                                 ws_bytes=nbytes), **kw})
    assert bw(alpha=0.0) == B.ERR_PARAM
    assert bw(alpha=1.5) == B.ERR_PARAM
    assert bw(mode=7) == B.ERR_PARAM
    assert bw(dW_out=G.data_ptr()) == B.ERR_PARAM
    assert bw(adj_max_iter=-2) == B.ERR_PARAM
    assert bw() == B.OK
    torch.cuda.synchronize()
    assert B.workspace_bytes(10, 3, 4, 1) == 0
    assert "workspace" in B.status_string(B.ERR_WORKSPACE)


def test_quantize_host_matches_oracle():
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(50000, 2, 16, 0.012, std=0.03, seed=3, max_iter=10, adj_max_iter=6, init="rows")
    ctx = B.Context()
    for _ in range(2):   # second call reuses the device buffers
        C, Wq, dW, dC, infos = ctx.quantize_host(wl.W, wl.C0, wl.G, wl.tau, 0.0, wl.max_iter, B.IMPLICIT, 0.0,
                                                 wl.adj_max_iter, 1.0)
        ref = oracle_run(wl)
        assert infos[0].status == 0 and infos[0].fwd_iters == 10 and infos[0].adj_iters == 6
        assert_close(C, ref["C"], TOL_C, "C")
        assert_close(Wq, ref["Wq"], TOL_C, "Wq")
        assert_close(dW, ref["dW"], TOL_GRAD, "dW")
        assert_close(dC, ref["dC"], TOL_GRAD, "dC")
    assert ctx.launches == 2 * (1 + 1 + 1 + 1 + 6 + 1)   # init, the single-launch forward loop, final, g, adjoint, dW


def test_quantize_host_with_both_gradients_from_one_forward():
    """idkm_quantize_host_ex: the implicit and the Jacobian-free gradients of one forward, copies overlapped with the
    kernels on the ctx's own two streams (pinned and pageable host buffers both work)."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(120000, 4, 64, 0.012, std=0.03, seed=9, max_iter=8, adj_max_iter=5, init="rows")
    ref_i, ref_j = oracle_run(wl, mode="implicit"), oracle_run(wl, mode="jfb")
    ctx = B.Context()
    for pinned in (False, True):
        W, C0, G = wl.W, wl.C0, wl.G
        if pinned:
            W, C0, G = (torch.from_numpy(x).pin_memory().numpy() for x in (wl.W, wl.C0, wl.G))
        C, Wq, dW, dC, infos, dWj, dCj = ctx.quantize_host(W, C0, G, wl.tau, 0.0, wl.max_iter, B.IMPLICIT, 0.0,
                                                           wl.adj_max_iter, 1.0, also_jfb=True)
        assert infos[0].status == 0 and infos[0].fwd_iters == 8 and infos[0].adj_iters == 5
        assert_close(C, ref_i["C"], TOL_C, "C")
        assert_close(Wq, ref_i["Wq"], TOL_C, "Wq")
        assert_close(dW, ref_i["dW"], TOL_GRAD, "dW implicit")
        assert_close(dC, ref_i["dC"], TOL_GRAD, "dC implicit")
        assert_close(dWj, ref_j["dW"], TOL_GRAD, "dW jfb")
        assert_close(dCj, ref_j["dC"], TOL_GRAD, "dC jfb")
    out = B.describe_path(4, 64, 5)
    assert out["adjoint_route"] == "fused passes" and out["adjoint_layout"][0] * out["adjoint_layout"][1] >= 64
    assert B.describe_path(1, 4, 30)["adjoint_route"] == "explicit Jacobian in registers"
    assert B.describe_path(1, 16, 30)["adjoint_route"] == "explicit Jacobian in tiles"
    assert B.describe_path(1, 16, 4)["adjoint_route"] == "fused passes"


def test_non_default_stream():
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(10000, 1, 8, 0.01, std=0.03, seed=4, max_iter=8, adj_max_iter=4)
    ref = oracle_run(wl)
    s = torch.cuda.Stream()
    ctx = B.Context()
    with torch.cuda.stream(s):
        W = torch.from_numpy(wl.W).cuda()
        C0 = torch.from_numpy(wl.C0).cuda()
        G = torch.from_numpy(wl.G).cuda()
        fr = ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter)
        dW, dC = ctx.backward(G, B.IMPLICIT, 0.0, wl.adj_max_iter, 1.0)
    s.synchronize()
    assert_close(fr.C.cpu().numpy(), ref["C"], TOL_C, "C")
    assert_close(dW.cpu().numpy(), ref["dW"], TOL_GRAD, "dW")


@pytest.mark.parametrize("m,d,k", [(30001, 1, 4), (20000, 1, 8), (10000, 2, 4), (9000, 4, 2), (5000, 2, 3),
                                   (40000, 1, 16), (33333, 2, 16), (50000, 4, 16), (20001, 1, 64), (25000, 2, 32),
                                   (12345, 4, 5), (300000, 1, 12), (7000, 2, 7), (31, 4, 3)])
def test_explicit_jacobian_adjoint_equals_fused_passes(m, d, k):
    """For k*d <= 64 the adjoint iteration runs on the explicitly formed k d x k d matrix (one pass over W; for
    k*d > 8 from 16 steps on); it must give the iterates of the one-pass-per-step path, with the tolerance rule and
    the counters behaving the same."""
    import torch
    from paper_2312_07759_b200 import binding as B
    adj_iters = 12 if k * d <= 8 else 20
    wl = WL.single_layer(m, d, k, 0.012, std=0.03, seed=m + k, max_iter=15, adj_max_iter=adj_iters, init="rows",
                         g_std=0.3)
    W, C0, G = (torch.from_numpy(x).cuda() for x in (wl.W, wl.C0, wl.G))
    res = {}
    for method in (0, 1):
        ctx = B.Context()
        ctx.set_adjoint_method(method)
        ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter)
        before = ctx.launches
        dW, dC = ctx.backward(G, B.IMPLICIT, 0.0, wl.adj_max_iter, 1.0)
        info = ctx.info()[0]
        assert info.status == 0 and info.adj_iters == wl.adj_max_iter
        res[method] = (dW.cpu().numpy(), dC.cpu().numpy(), info.adj_residual, ctx.launches - before)
        # tolerance mode: both stop at the same iteration (or one apart, by fp32 rounding of the residual)
        dW2, dC2 = ctx.backward(G, B.IMPLICIT, 1e-4, 500, 0.5)
        res[(method, "tol")] = (ctx.info()[0].adj_iters, dC2.cpu().numpy())
    assert res[0][3] == 3 and res[1][3] == 2 + wl.adj_max_iter          # g, J (or 12 passes), dW
    assert_close(res[0][1], res[1][1], 1e-5, "dC")
    assert_close(res[0][0], res[1][0], 1e-5, "dW")
    assert abs(res[0][2] - res[1][2]) <= 1e-3 * max(res[1][2], 1e-30) + 1e-9
    assert abs(res[(0, "tol")][0] - res[(1, "tol")][0]) <= 1
    assert_close(res[(0, "tol")][1], res[(1, "tol")][1], 1e-3, "dC at tolerance")
    # against the oracle at common centroids (the oracle's, handed over with the loop switched off): the gradient
    # tolerance for every d, scalar weights included -- no weight can lie between two identical centroid sets
    ref = oracle_run(wl)
    wc = at_centroids(wl, ref["C"])
    refc = oracle_backward_at(wc, wc.C0)
    for method in (0, 1):
        ctx = B.Context()
        ctx.set_adjoint_method(method)
        ctx.forward(torch.from_numpy(wc.W).cuda(), torch.from_numpy(wc.C0).cuda(), wc.tau, 0.0, 0)
        dWc, dCc = ctx.backward(G, B.IMPLICIT, 0.0, wl.adj_max_iter, 1.0)
        assert_close(dCc.cpu().numpy(), refc["dC"], TOL_GRAD, f"dC vs oracle at common C, adjoint method {method}")
        assert_close(dWc.cpu().numpy(), refc["dW"], TOL_GRAD, f"dW vs oracle at common C, adjoint method {method}")


def test_pipe_rate_microbenchmarks():
    """The measured fp32 and special-function issue rates are positive, stand in the ratio of the two pipes' widths
    (128 : 16 results per clock per SM) and, divided by the SM clock read (never set) through NVML around the
    measurement, land near those widths.  The clock of a shared GPU is whatever it is, so nothing here depends on
    the part's maximum clock."""
    import torch
    from paper_2312_07759_b200 import binding as B
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    clocks = []
    try:
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(torch.cuda.current_device())
        read_clock = lambda: float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
    except Exception:
        read_clock = None
    B.measure_pipe_rates()                      # brings the clock up before it is read
    fp32 = sfu = 0.0
    for _ in range(3):
        if read_clock:
            clocks.append(read_clock())
        a, b = B.measure_pipe_rates()
        fp32, sfu = max(fp32, a), max(sfu, b)
        if read_clock:
            clocks.append(read_clock())
    assert fp32 > 0 and sfu > 0
    assert 6.0 < fp32 / sfu < 10.0, (fp32, sfu)
    if clocks:
        # the highest clock seen bounds the rate from above, the lowest from below (the clock may move in between)
        hi, lo = max(clocks) * 1e6, min(clocks) * 1e6
        assert fp32 / (sms * 128 * hi) < 1.10 and fp32 / (sms * 128 * lo) > 0.50, (fp32, clocks)
        assert sfu / (sms * 16 * hi) < 1.10 and sfu / (sms * 16 * lo) > 0.50, (sfu, clocks)
    assert B.lib.idkm_measure_pipe_rates(None, None, None) == B.ERR_NULL


@pytest.mark.parametrize("d,k,m", [(1, 4, 4096), (1, 8, 36864), (2, 2, 50001), (4, 8, 100000), (1, 4, 1 << 20),
                                   (1, 16, 70000), (2, 16, 300001), (2, 5, 33), (1, 4, 4500000), (4, 3, 3000000)])
def test_one_launch_forward_loop_matches_launch_per_iteration(d, k, m):
    """The cooperative one-launch forward loop and the launch-per-iteration loop run the same iteration: both match
    the oracle, they agree with each other far inside the tolerance, the one-launch path really is one launch, and a
    tolerance-mode run stops at the same iteration count."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(m, d, k, 0.01, std=0.03, seed=11, max_iter=12, adj_max_iter=1)
    dev = torch.device("cuda:0")
    W, C0 = torch.from_numpy(wl.W).to(dev), torch.from_numpy(wl.C0).to(dev)
    ref = oracle_run(wl, want_dW=False)
    outs = {}
    for method in (0, 1):
        ctx = B.Context()
        ctx.set_forward_loop(method)
        n0 = ctx.launches
        fr = ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter, want_Wq=True)
        torch.cuda.synchronize()
        outs[method] = (fr.C.cpu().numpy().astype(np.float64), ctx.launches - n0, ctx.info()[0])
        assert_close(outs[method][0], ref["C"], TOL_C, f"C, loop method {method}")
        assert outs[method][2].fwd_iters == wl.max_iter and outs[method][2].status == 0
    assert outs[0][1] == 3                       # init, the loop, the final pass
    # init, the step(s) of every iteration, the final pass: the smallest layouts step fp32 and fp64 layers in one
    # launch, the others in two
    dual = (d == 1 and k <= 4) or (d == 2 and k <= 2)
    assert outs[1][1] == 2 + (1 if dual else 2) * wl.max_iter
    assert_close(outs[0][0], outs[1][0], 1e-6, "one-launch vs per-iteration centroids")
    # tolerance mode: same stopping iteration
    its = []
    for method in (0, 1):
        ctx = B.Context()
        ctx.set_forward_loop(method)
        ctx.forward(W, C0, wl.tau, 1e-4, 200)
        torch.cuda.synchronize()
        its.append(ctx.info()[0].fwd_iters)
    assert its[0] == its[1] and 1 <= its[0] <= 200


def test_tiled_explicit_jacobian_on_batched_layers():
    """Three layers of different sizes in one call, k = 16 (k d = 16): the adjoint on the explicitly formed matrices
    equals the fused passes layer by layer, including a layer that spans several blocks and one smaller than a tile."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.config3(shapes=[(64, 32, 3, 3), (16, 8, 3, 3), (5, 4, 3, 3)], k=16, tau=0.01, iters=20, seed=21)
    offs = [int(x) for x in wl.layer_offsets]
    W, C0, G = (torch.from_numpy(x).cuda() for x in (wl.W, wl.C0, wl.G))
    res = {}
    for method in (0, 1):
        ctx = B.Context()
        ctx.set_adjoint_method(method)
        ctx.forward(W, C0, wl.tau, 0.0, 12, layer_offsets=offs)
        n0 = ctx.launches
        dW, dC = ctx.backward(G, B.IMPLICIT, 0.0, 20, 1.0)
        torch.cuda.synchronize()
        infos = ctx.info()
        assert all(i.status == 0 and i.adj_iters == 20 for i in infos)
        res[method] = (dW.cpu().numpy(), dC.cpu().numpy(), ctx.launches - n0)
    assert res[0][2] == 3 and res[1][2] == 22
    for l in range(3):
        a, b = offs[l], offs[l + 1]
        assert_close(res[0][1][16 * l:16 * (l + 1)], res[1][1][16 * l:16 * (l + 1)], 1e-5, f"dC layer {l}")
        assert_close(res[0][0][a:b], res[1][0][a:b], 1e-5, f"dW layer {l}")


@pytest.mark.parametrize("m,d,k,loop,adj", [(3000, 1, 4, 0, 0), (3000, 1, 4, 1, 1), (40000, 2, 16, 0, 0),
                                            (40000, 2, 16, 1, 1), (60000, 4, 32, 1, 1)])
def test_residual_history_matches_the_oracle_iteration_by_iteration(m, d, k, loop, adj):
    """idkm_get_history returns the stop-rule quantity of every iteration: compared with residuals recomputed from the
    oracle's own iterates (forward: one application of F at a time; adjoint: one application of the adjoint map)."""
    import torch
    from oracle import idkm_ref as R
    from paper_2312_07759_b200 import binding as B
    T, Ta = 9, 20
    wl = WL.single_layer(m, d, k, 0.01, std=0.03, seed=3 + k, max_iter=T, adj_max_iter=Ta, g_std=0.5)
    W, C0, G = (torch.from_numpy(x).cuda() for x in (wl.W, wl.C0, wl.G))
    ctx = B.Context()
    ctx.set_forward_loop(loop)
    ctx.set_adjoint_method(adj)
    ctx.forward(W, C0, wl.tau, 0.0, T)
    ctx.backward(G, B.IMPLICIT, 0.0, Ta, 1.0)
    hf, ha = ctx.history(0), ctx.history(1)
    info = ctx.info()[0]
    assert hf.shape == (T,) and ha.shape == (Ta,)
    assert hf[-1] == np.float32(info.fwd_residual) and ha[-1] == np.float32(info.adj_residual)
    assert ctx.history(0, capacity=4).shape == (4,)
    # oracle, iteration by iteration
    Wd, Gd = wl.W.astype(np.float64), wl.G.astype(np.float64)
    Cc = wl.C0.astype(np.float64)
    rf = []
    for _ in range(T):
        Cn = R.step(Wd, Cc, wl.tau)[0]
        rf.append(np.linalg.norm(Cn - Cc) / max(np.linalg.norm(Cn), 1e-300))
        Cc = Cn
    assert np.allclose(hf, rf, rtol=2e-3, atol=1e-9)
    _, _, S, F = R.final(Wd, Cc, wl.tau, want_Wq=False)
    g = R.codebook_grad(Wd, Gd, Cc, wl.tau)
    u, ra = g.copy(), []
    for _ in range(Ta):
        un = R.adjoint_apply(Wd, Cc, wl.tau, S, F, u) + g
        ra.append(np.linalg.norm(un - u) / max(np.linalg.norm(un), 1e-300))
        u = un
    if d > 1:      # d = 1: the sign kinks make later adjoint residuals differ at the percent level
        assert np.allclose(ha, ra, rtol=5e-3, atol=1e-9)
    else:
        assert np.allclose(ha[:3], ra[:3], rtol=5e-2)


def test_dual_step_kernel_routes_collapsing_layers_like_two_launches():
    """Batched scalar layers of which some collapse in mid-loop (tau above the mean absolute deviation of their
    weights): the kernel that steps fp32 and fp64 layers side by side must route every layer exactly as two ordered
    launches do -- bitwise equal centroids over many repeats, every arrival counter back at rest, and the oracle's
    centroids per layer (which the collapsing layers only reach through the fp64 step)."""
    import torch
    from paper_2312_07759_b200 import binding as B
    shapes = [(16, 512, 3, 3), (64, 64, 3, 3), (24, 512, 3, 3), (32, 256, 3, 3), (8, 512, 3, 3), (40, 128, 3, 3),
              (12, 512, 3, 3)]
    wl = WL.config3(shapes=shapes, iters=40)
    offs = [int(x) for x in wl.layer_offsets]
    W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    ref = None
    for method in (2, 1):
        ctx = B.Context()
        ctx.set_forward_loop(method)
        for rep in range(1 if method == 2 else 25):
            C = ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter, layer_offsets=offs, want_Wq=False).C
            torch.cuda.synchronize()
            assert ctx.busy_tickets() == 0
            assert all(i.status == 0 and i.fwd_iters == wl.max_iter for i in ctx.info())
            if ref is None:
                ref = C.cpu().numpy()
            else:
                assert np.array_equal(C.cpu().numpy(), ref), f"repeat {rep}"
    # tolerance mode: layers leave the loop at different iterations
    its = []
    for method in (2, 1):
        ctx = B.Context()
        ctx.set_forward_loop(method)
        Ct = ctx.forward(W, C0, wl.tau, 1e-5, 300, layer_offsets=offs, want_Wq=False).C.cpu().numpy()
        assert ctx.busy_tickets() == 0
        its.append(([i.fwd_iters for i in ctx.info()], Ct))
    assert its[0][0] == its[1][0] and np.array_equal(its[0][1], its[1][1])
    k = wl.k
    for l, lw in enumerate(WL.split_layers(wl)):
        r = oracle_run(lw, want_dW=False)
        assert_close(ref[l * k:(l + 1) * k], r["C"], TOL_C, f"layer {l} C")


@pytest.mark.parametrize("d,k,m", [(1, 2, 50001), (1, 4, 1 << 20), (2, 2, 300001), (2, 4, 70000), (4, 2, 123457),
                                   (4, 4, 65536), (1, 8, 99999), (4, 16, 40000), (1, 16, 5), (2, 8, 1023)])
def test_bulk_copy_pipeline_gives_the_result_of_the_per_thread_loads(d, k, m):
    """Forward-loop method 3 streams the rows of small-codebook layers into shared memory by bulk asynchronous copies
    (one per trip, three trips ahead, completion on a barrier with a bounded wait); the arithmetic per row is that of
    method 2 -- ragged tails, sizes below one tile and a tolerance-mode run included."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(m, d, min(k, m), 0.01, std=0.03, seed=m + k, max_iter=7, adj_max_iter=1, init="rows" if m >= k else "quantile")
    W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    res = {}
    for method in (2, 3):
        ctx = B.Context()
        ctx.set_forward_loop(method)
        fr = ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter)
        torch.cuda.synchronize()
        info = ctx.info()[0]
        assert info.status == 0 and info.fwd_iters == wl.max_iter, info
        assert ctx.busy_tickets() == 0
        tol_C = ctx.forward(W, C0, wl.tau, 1e-4, 60, want_Wq=False).C.cpu().numpy()
        res[method] = (fr.C.cpu().numpy(), fr.Wq.cpu().numpy(), tol_C, ctx.info()[0].fwd_iters)
    # (the stages take shared memory, so fewer blocks may be resident and the cross-block sums may be grouped
    # differently: equal to a few units in the last place, not always bitwise)
    assert_close(res[3][0], res[2][0], 2e-6, "C")
    assert_close(res[3][1], res[2][1], 2e-6, "Wq")
    assert_close(res[3][2], res[2][2], 2e-6, "C, tolerance mode")
    assert abs(res[2][3] - res[3][3]) <= 1


def test_bulk_copy_pipeline_on_batched_layers_with_unaligned_offsets():
    """Layers whose first row is not 16-byte aligned keep the per-thread loads inside the same launch; aligned ones
    take the copies; collapsing layers leave for the other step kernel in mid-loop."""
    import torch
    from paper_2312_07759_b200 import binding as B
    rng = np.random.default_rng(4)
    sizes = [4096, 1001, 37, 20000, 3, 8192, 50000]
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    stds = [0.05, 0.05, 0.05, 0.008, 0.05, 0.05, 0.008]          # two layers collapse at tau = 0.02
    W = np.concatenate([(rng.standard_normal((n, 1)) * s) for n, s in zip(sizes, stds)]).astype(np.float32)
    k = 3
    C0 = np.concatenate([WL.quantile_centroids(W[offs[l]:offs[l + 1]], k) for l in range(len(sizes))])
    Wd, Cd = torch.from_numpy(W).cuda(), torch.from_numpy(C0).cuda()
    out = {}
    for method in (2, 3):
        ctx = B.Context()
        ctx.set_forward_loop(method)
        C = ctx.forward(Wd, Cd, float(np.float32(0.02)), 0.0, 25, layer_offsets=[int(x) for x in offs], want_Wq=False).C
        torch.cuda.synchronize()
        assert all(i.status == 0 and i.fwd_iters == 25 for i in ctx.info())
        assert ctx.busy_tickets() == 0
        out[method] = C.cpu().numpy()
    assert np.array_equal(out[2], out[3])          # batched calls launch the same grid in both methods


@pytest.mark.parametrize("m,d,k", [(5003, 1, 4), (4099, 2, 16), (30001, 4, 64), (7, 4, 3), (20000, 1, 256)])
def test_half_precision_wq_is_the_rounded_fp32_result(m, d, k):
    """idkm_set_wq_dtype: Wq written as bfloat16 / float16 equals the fp32 Wq of the same call rounded to nearest even,
    bit for bit (ragged sizes and both store paths), and stays within half a unit in the last place of the oracle."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(m, d, min(k, m), 0.012, std=0.03, seed=m + k, max_iter=6, adj_max_iter=2,
                         init="rows" if m >= k else "quantile")
    ref = oracle_run(wl)
    W, C0, G = (torch.from_numpy(x).cuda() for x in (wl.W, wl.C0, wl.G))
    ctx = B.Context()
    full = ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter).Wq
    for dtype, ttype, eps in ((1, torch.bfloat16, 2.0 ** -8), (2, torch.float16, 2.0 ** -11)):
        ctx.set_wq_dtype(dtype)
        fr = ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter)
        assert fr.Wq.dtype == ttype and fr.Wq.shape == W.shape
        assert torch.equal(fr.Wq, full.to(ttype))
        err = np.abs(fr.Wq.float().cpu().numpy() - ref["Wq"])
        assert np.all(err <= eps * np.abs(ref["Wq"]) + 1e-7)
        dW, dC = ctx.backward(G, B.JFB, 0.0, 0, 1.0)          # the backward is unaffected
        assert_close(dC.cpu().numpy(), oracle_run(wl, mode="jfb")["dC"], TOL_GRAD, "dC")
    ctx.set_wq_dtype(0)
    assert torch.equal(ctx.forward(W, C0, wl.tau, 0.0, wl.max_iter).Wq, full)
    assert B.lib.idkm_set_wq_dtype(ctx._h, 3) == B.ERR_PARAM
