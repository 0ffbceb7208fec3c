"""The forward loop of a batch of layers (or of one layer too large for the one-layer loop kernel) in a single
cooperative launch, against the launch-per-iteration path it replaces and against the oracle.  Both paths run the
same step bodies; they differ in how the tiles are spread over blocks (the single launch uses only as many blocks as
are resident at once), hence in the grouping of the cross-block sums: agreement to a few ulp, not bitwise."""
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
    C0, info0, n0, _ = run(wl, 4)
    assert n0 == 3 and n1 >= 2 + wl.max_iter          # init + ONE loop launch + final pass, against one per iteration
    for a, b in zip(info0, info1):
        assert a.status == 0 and b.status == 0 and a.fwd_iters == b.fwd_iters == wl.max_iter
        assert abs(a.fwd_residual - b.fwd_residual) <= 1e-5 * max(b.fwd_residual, 1e-3)
    for l, lw in enumerate(WL.split_layers(wl)):
        sl = slice(l * k, (l + 1) * k)
        assert_close(C0[sl], C1[sl], 2e-6, f"layer {l}: single launch against launch per iteration")
        assert_close(C0[sl], oracle_run(lw, mode="jfb")["C"], TOL_C, f"layer {l} C against the oracle")


def test_tolerance_mode_leaves_at_the_same_iterations():
    wl = batched([60000, 2500, 33333, 900, 200000, 12345], 1, 4, 0.01, [0.03, 0.02, 0.001, 0.05, 0.02, 0.04], iters=400, seed=7)
    C1, info1, _, _ = run(wl, 1, tol=1e-5)
    C0, info0, n0, _ = run(wl, 4, tol=1e-5)
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


def test_one_layer_beyond_the_one_layer_loop_takes_the_single_launch_too():
    wl = WL.single_layer(6_000_000, 1, 4, 0.003, std=0.03, seed=11, max_iter=8, adj_max_iter=2)
    C1, info1, n1, _ = run(wl, 1)
    C0, info0, n0, _ = run(wl, 4)
    assert n0 == 3 and info0[0].status == 0 and info0[0].fwd_iters == 8
    assert_close(C0, C1, 2e-6, "C")
    assert_close(C0, oracle_run(wl, mode="jfb")["C"], TOL_C, "C against the oracle")


def test_runs_are_reproducible_bit_for_bit():
    wl = batched([70001, 3000, 40000, 517, 131072], 2, 4, 0.004, [0.03, 0.02, 0.0006, 0.05, 0.02], iters=10, seed=3)
    ref, _, _, ctx = run(wl, 4)
    for _ in range(5):
        again, _, _, _ = run(wl, 4)
        assert np.array_equal(ref, again)
    assert ctx.busy_tickets() == 0


def test_barrier_timeout_is_reported_for_every_layer_and_the_context_survives():
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = batched([30000, 2000, 50000], 1, 4, 0.01, [0.03, 0.02, 0.04], iters=6, seed=5)
    W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    offs = [int(x) for x in wl.layer_offsets]
    ctx = B.Context()
    ctx.set_forward_loop(4)
    good = ctx.forward(W, C0, wl.tau, 0.0, 6, layer_offsets=offs).C.cpu().numpy()
    assert all(i.status == 0 for i in ctx.info())
    ctx.set_test_hooks(missing_arrivals=1, spin_limit_ticks=2000000)      # about a millisecond per wait
    try:
        ctx.forward(W, C0, wl.tau, 0.0, 6, layer_offsets=offs)
        torch.cuda.synchronize()
        for info in ctx.info():
            assert info.status == B.ERR_TIMEOUT and info.fwd_iters == 1   # the first iteration's step completed
        assert ctx.busy_tickets() == 0
    finally:
        ctx.set_test_hooks(0, 0)
    again = ctx.forward(W, C0, wl.tau, 0.0, 6, layer_offsets=offs).C.cpu().numpy()
    assert all(i.status == 0 and i.fwd_iters == 6 for i in ctx.info())
    assert np.array_equal(again, good)


def test_default_routing_takes_the_single_launch_where_it_was_measured_faster():
    """Method 0: a small batch with a codebook beyond the side-by-side step kernel takes the single launch; a small
    batch of the smallest codebook and a single large layer keep the launch per iteration."""
    wl = batched([30000, 2000, 50000], 1, 8, 0.01, [0.03, 0.02, 0.04], iters=6, seed=5)
    assert run(wl, 0)[2] == 3
    wl = batched([30000, 2000, 50000], 1, 4, 0.01, [0.03, 0.02, 0.04], iters=6, seed=5)
    assert run(wl, 0)[2] >= 2 + 6
    from paper_2312_07759_b200 import binding as B
    assert B.lib.idkm_set_forward_loop(B.Context()._h, 5) == B.ERR_PARAM
