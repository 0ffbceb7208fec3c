"""idkm_step_noalloc, the entry point for callers that cannot allocate device memory (allocator callbacks,
fixed-arena servers, plug-ins barred from their host's CUDA allocator).

Collected last on purpose: a run that stops at the first failure has then already run every other test.
The new entry point is checked through the C ABI against the regular one (idkm_forward with one iteration)
on two calls in a row, because all calls share one built-in scratch array that keeps the previous call's
contents."""
import numpy as np
import pytest

from paper_2312_07759_b200 import workloads as WL
from parity_util import TOL_C, assert_close

pytestmark = pytest.mark.gpu


def _regular_one_step(ctx, W, C0, tau):
    return ctx.forward(W, C0, tau, 0.0, 1, want_Wq=False).C


@pytest.mark.parametrize("m,d,k,tau", [(50001, 1, 4, 0.01), (30011, 4, 64, 0.012), (20000, 2, 256, 0.01),
                                       (30000, 4, 256, 0.012), (30000, 1, 256, 0.01)])
def test_noalloc_step_matches_regular_forward_twice(m, d, k, tau):
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(m, d, k, tau, std=0.03, seed=m + k, init="rows")
    W = torch.from_numpy(wl.W).cuda()
    C0 = torch.from_numpy(wl.C0).cuda()
    ctx = B.Context()
    ref1 = _regular_one_step(ctx, W, C0, wl.tau)
    ref2 = _regular_one_step(ctx, W, ref1, wl.tau)
    out1 = torch.empty_like(C0)     # outputs are the caller's; the library call allocates nothing
    out2 = torch.empty_like(C0)
    B.step_noalloc(W, C0, wl.tau, C_out=out1)
    B.step_noalloc(W, out1, wl.tau, C_out=out2)     # second call reuses the scratch the first one left behind
    torch.cuda.synchronize()
    assert_close(out1.cpu().numpy(), ref1.cpu().numpy(), TOL_C, "first call")
    assert_close(out2.cpu().numpy(), ref2.cpu().numpy(), TOL_C, "second call")
    # and against the oracle, so that agreement is not two wrongs
    from oracle import idkm_ref as R
    Cp, _, _ = R.step(wl.W.astype(np.float64), wl.C0.astype(np.float64), wl.tau)
    assert_close(out1.cpu().numpy(), Cp, TOL_C, "first call vs oracle")


def test_noalloc_collapsed_start_takes_the_fp64_step():
    """All starting centroids within a sliver of tau: the call must route the layer through the fp64 kernel."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(40000, 1, 4, 0.05, std=0.02, seed=8)
    C0 = (np.float32(wl.W.mean()) + np.array([[-1e-6], [-3e-7], [3e-7], [1e-6]], np.float32)).astype(np.float32)
    W = torch.from_numpy(wl.W).cuda()
    out = B.step_noalloc(W, torch.from_numpy(C0).cuda(), wl.tau)
    ref = _regular_one_step(B.Context(), W, torch.from_numpy(C0).cuda(), wl.tau)
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy(), ref.cpu().numpy(), TOL_C, "collapsed start")


def test_noalloc_every_supported_codebook_fits_the_builtin_scratch():
    """The size check passes for every (d, codebook layout) on a layer large enough to fill the grid, the largest
    codebook included; the result still matches the regular entry point."""
    import torch
    from paper_2312_07759_b200 import binding as B
    ctx = B.Context()
    for d in (1, 2, 4):
        for k in (2, 4, 8, 16, 32, 64, 128, 256):
            m = 400000
            wl = WL.single_layer(m, d, k, 0.012, std=0.03, seed=d * 1000 + k, init="rows")
            W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
            out = torch.empty_like(C0)
            rc = B.lib.idkm_step_noalloc(W.data_ptr(), m, d, C0.data_ptr(), k, wl.tau, out.data_ptr(), None)
            assert rc == B.OK, (d, k, rc)
            ref = _regular_one_step(ctx, W, C0, wl.tau)
            torch.cuda.synchronize()
            assert B.step_noalloc_status() == B.OK
            assert_close(out.cpu().numpy(), ref.cpu().numpy(), TOL_C, f"d={d} k={k}")


def test_noalloc_status_reports_a_nan_in_the_weights():
    """The step has no context to report through: a NaN in W must show in idkm_step_noalloc_status, and a clean call
    afterwards must read OK again."""
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(30000, 1, 4, 0.01, std=0.03, seed=2)
    Wbad = wl.W.copy()
    Wbad[1234, 0] = np.nan
    C0 = torch.from_numpy(wl.C0).cuda()
    B.step_noalloc(torch.from_numpy(Wbad).cuda(), C0, wl.tau)
    assert B.step_noalloc_status() == B.ERR_NONFINITE
    B.step_noalloc(torch.from_numpy(wl.W).cuda(), C0, wl.tau)
    assert B.step_noalloc_status() == B.OK
    assert B.lib.idkm_step_noalloc_status(None, None) == B.ERR_NULL


def test_noalloc_argument_errors():
    import torch
    from paper_2312_07759_b200 import binding as B
    W = torch.zeros(1000, 1, device="cuda")
    C = torch.zeros(4, 1, device="cuda")
    f = B.lib.idkm_step_noalloc
    assert f(None, 1000, 1, C.data_ptr(), 4, 0.1, C.data_ptr(), None) == B.ERR_NULL
    assert f(W.data_ptr(), 0, 1, C.data_ptr(), 4, 0.1, C.data_ptr(), None) == B.ERR_SHAPE
    assert f(W.data_ptr(), 1000, 3, C.data_ptr(), 4, 0.1, C.data_ptr(), None) == B.ERR_UNSUPPORTED
    assert f(W.data_ptr(), 1000, 1, C.data_ptr(), 300, 0.1, C.data_ptr(), None) == B.ERR_UNSUPPORTED
    assert f(W.data_ptr(), 1000, 1, C.data_ptr(), 4, 0.0, C.data_ptr(), None) == B.ERR_PARAM
    assert f(W.data_ptr() + 4, 1000, 1, C.data_ptr(), 4, 0.1, C.data_ptr(), None) == B.ERR_ALIGN
    assert "scratch" in B.status_string(-11)
