"""The forward loop of a batch of layers in a single cooperative launch (every block works for one layer; one grid
barrier per iteration), against the launch-per-iteration path it replaces and against the oracle.  The two paths
group the rows and the cross-block sums differently: agreement to a few ulp, not bitwise."""
import numpy as np
import pytest

from paper_2312_07759_b200 import workloads as WL
from parity_util import TOL_C, assert_close, oracle_run

pytestmark = pytest.mark.gpu


def batched(ms, d, k, tau, stds, iters, seed=0):
    parts = [WL.single_layer(m, d, k, tau, std=s, seed=seed + 17 * i, max_iter=iters, adj_max_iter=2)
             for i, (m, s) in enumerate(zip(ms, stds))]
    offs = np.concatenate([[0], np.cumsum([p.m for p in parts])]).astype(np.int64)
    return WL.Workload("batched", np.concatenate([p.W for p in parts]), np.concatenate([p.C0 for p in parts]),
                       np.concatenate([p.G for p in parts]), d, k, parts[0].tau, 0.0, iters, 0.0, 2, offs, seed)


def run(wl, method, tol=0.0, hooks=None):
    import torch
    from paper_2312_07759_b200 import binding as B
    ctx = B.Context()
    ctx.set_forward_loop(method)
    W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    n0 = ctx.launches
    fr = ctx.forward(W, C0, wl.tau, tol, wl.max_iter, layer_offsets=[int(x) for x in wl.layer_offsets], want_Wq=False)
    torch.cuda.synchronize()
    return fr.C.cpu().numpy(), ctx.info(), ctx.launches - n0, ctx


# the third layer's spread is a fraction of tau: it collapses and is handed to the increment-form step on the way
@pytest.mark.parametrize("d,k", [(1, 2), (1, 4), (1, 8), (1, 16), (2, 2), (2, 4), (2, 8), (2, 16), (4, 2), (4, 4), (4, 8),
                                 (4, 16), (1, 3), (2, 11), (4, 5)])
def test_single_launch_batch_equals_launch_per_iteration_and_the_oracle(d, k):
    wl = batched([70001, 3000, 40000, 517, 131072], d, k, 0.004, [0.03, 0.02, 0.0006, 0.05, 0.02], iters=14, seed=d * 100 + k)
    C1, info1, n1, _ = run(wl, 1)
    C0, info0, n0, _ = run(wl, 0)
    assert n1 >= 2 + wl.max_iter
    assert n0 == (n1 if (d == 4 and k > 8) else 3)    # init + ONE loop launch + final pass (no such kernel at d = 4, k > 8)
    for a, b in zip(info0, info1):
        assert a.status == 0 and b.status == 0 and a.fwd_iters == b.fwd_iters == wl.max_iter
        # (the residual is a difference of nearly equal centroid sets: the two paths' rounding shows in its digits)
        assert abs(a.fwd_residual - b.fwd_residual) <= 0.05 * b.fwd_residual + 1e-7
    for l, lw in enumerate(WL.split_layers(wl)):
        sl = slice(l * k, (l + 1) * k)
        assert_close(C0[sl], C1[sl], 2e-6, f"layer {l}: single launch against launch per iteration")
        assert_close(C0[sl], oracle_run(lw, mode="jfb")["C"], TOL_C, f"layer {l} C against the oracle")


def test_tolerance_mode_leaves_at_the_same_iterations():
    wl = batched([60000, 2500, 33333, 900, 200000, 12345], 1, 4, 0.01, [0.03, 0.02, 0.001, 0.05, 0.02, 0.04], iters=400, seed=7)
    C1, info1, _, _ = run(wl, 1, tol=1e-5)
    C0, info0, n0, _ = run(wl, 0, tol=1e-5)
    assert n0 == 3
    its = [i.fwd_iters for i in info0]
    assert len(set(its)) > 1 and max(its) < 400          # layers leave at different iterations, none hits the cap
    for l, (a, b) in enumerate(zip(info0, info1)):
        assert a.status == 0 and b.status == 0
        assert abs(a.fwd_iters - b.fwd_iters) <= 1, (l, a.fwd_iters, b.fwd_iters)
        assert a.fwd_residual < 1e-5
    assert_close(C0, C1, 2e-5, "C, tolerance mode")
    for l, lw in enumerate(WL.split_layers(wl)):
        lw.tol, lw.max_iter = 1e-5, 400
        ref = oracle_run(lw, mode="jfb", fixed=False)
        assert abs(info0[l].fwd_iters - ref["iters"]) <= 1
        assert_close(C0[l * 4:(l + 1) * 4], ref["C"], 2e-5, f"layer {l} C against the oracle, tolerance mode")


def test_runs_are_reproducible_bit_for_bit():
    wl = batched([70001, 3000, 40000, 517, 131072], 2, 4, 0.004, [0.03, 0.02, 0.0006, 0.05, 0.02], iters=10, seed=3)
    ref, _, n, ctx = run(wl, 0)
    assert n == 3
    for _ in range(5):
        again, _, _, _ = run(wl, 0)
        assert np.array_equal(ref, again)
    assert ctx.busy_tickets() == 0


def test_barrier_timeout_is_reported_for_every_layer_and_the_context_survives():
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = batched([30000, 2000, 50000], 1, 4, 0.01, [0.03, 0.02, 0.04], iters=6, seed=5)
    W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    offs = [int(x) for x in wl.layer_offsets]
    ctx = B.Context()
    good = ctx.forward(W, C0, wl.tau, 0.0, 6, layer_offsets=offs).C.cpu().numpy()
    assert all(i.status == 0 for i in ctx.info())
    ctx.set_test_hooks(missing_arrivals=1, spin_limit_ticks=2000000)      # about a millisecond per wait
    try:
        ctx.forward(W, C0, wl.tau, 0.0, 6, layer_offsets=offs)
        torch.cuda.synchronize()
        for info in ctx.info():
            assert info.status == B.ERR_TIMEOUT and info.fwd_iters == 0
        assert ctx.busy_tickets() == 0
    finally:
        ctx.set_test_hooks(0, 0)
    again = ctx.forward(W, C0, wl.tau, 0.0, 6, layer_offsets=offs).C.cpu().numpy()
    assert all(i.status == 0 and i.fwd_iters == 6 for i in ctx.info())
    assert np.array_equal(again, good)


def test_routing_of_batches():
    """A batch within the size limits takes the single launch; more layers than blocks, d = 4 beyond the single-layer
    size and the fp64 collapse step keep the launch per iteration."""
    from paper_2312_07759_b200 import binding as B
    wl = batched([30000, 2000, 50000], 1, 8, 0.01, [0.03, 0.02, 0.04], iters=6, seed=5)
    assert run(wl, 0)[2] == 3
    wl4 = batched([3_000_000, 2_500_000], 4, 4, 0.01, [0.03, 0.02], iters=3, seed=6)
    C0, info, n, _ = run(wl4, 0)
    assert n >= 2 + 3 and all(i.status == 0 and i.fwd_iters == 3 for i in info)
    ctx = B.Context()
    ctx.set_collapse_step(1)
    import torch
    W, Cs = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    n0 = ctx.launches
    ctx.forward(W, Cs, wl.tau, 0.0, 6, layer_offsets=[int(x) for x in wl.layer_offsets], want_Wq=False)
    assert ctx.launches - n0 >= 2 + 6
    assert B.lib.idkm_set_forward_loop(ctx._h, 4) == B.ERR_PARAM


def test_more_layers_than_a_small_grid_and_tiny_layers():
    """64 layers (the library's maximum) of a few hundred rows each: every layer gets one block."""
    ms = [257 + 13 * i for i in range(64)]
    wl = batched(ms, 2, 4, 0.01, [0.02 + 0.001 * (i % 7) for i in range(64)], iters=9, seed=9)
    C0, info0, n0, _ = run(wl, 0)
    C1, info1, _, _ = run(wl, 1)
    assert n0 == 3
    assert all(i.status == 0 and i.fwd_iters == 9 for i in info0)
    assert_close(C0, C1, 2e-6, "C")
    for l, lw in enumerate(WL.split_layers(wl)):
        assert_close(C0[l * 4:(l + 1) * 4], oracle_run(lw, mode="jfb")["C"], TOL_C, f"layer {l} C against the oracle")
