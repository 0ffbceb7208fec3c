"""Out-of-bounds and failure-path checks on the GPU that need no sanitizer (B200 only).

Guard words: every output and the workspace sit inside a larger buffer filled with a sentinel; after the calls the
sentinels before and after each of them must be intact.  Timeout path: the single-launch forward loop is told (host-side
fault injection) to wait for an arrival that never comes; its bounded waits must run out, the status must say so and
the context must stay usable."""
import numpy as np
import pytest

from paper_2312_07759_b200 import workloads as WL

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes of sentinel on each side
SENT = 0xA5


def _carve(torch, nbytes_list):
    """One uint8 buffer holding the regions back to back, each 256-byte aligned with GUARD bytes of sentinel around."""
    offs, total = [], GUARD
    for n in nbytes_list:
        total = (total + 255) // 256 * 256
        offs.append(total)
        total += n + GUARD
    buf = torch.full((total + 256,), SENT, dtype=torch.uint8, device="cuda")
    base = (buf.data_ptr() + 255) // 256 * 256 - buf.data_ptr()
    return buf, [base + o for o in offs]


def _check(torch, buf, offs, sizes):
    host = buf.cpu().numpy()
    inside = np.zeros(host.shape[0], dtype=bool)
    for o, n in zip(offs, sizes):
        inside[o:o + n] = True
    assert np.all(host[~inside] == SENT), "a sentinel byte outside the buffers was overwritten"


@pytest.mark.parametrize("m,d,k", [(1, 1, 2), (33, 2, 3), (4097, 1, 4), (100003, 4, 16), (70001, 4, 200), (5000, 2, 32)])
def test_guard_words_around_outputs_and_workspace(m, d, k):
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(m, d, k, 0.01, std=0.03, seed=7 + m % 13, init="rows" if m >= k else "quantile") if m >= k \
        else None
    if wl is None:      # fewer rows than centroids: centroids drawn separately
        rng = np.random.default_rng(1)
        W = rng.standard_normal((m, d)).astype(np.float32) * 0.03
        C0 = rng.standard_normal((k, d)).astype(np.float32) * 0.03
        G = rng.standard_normal((m, d)).astype(np.float32)
    else:
        W, C0, G = wl.W, wl.C0, wl.G
    ws_bytes = B.workspace_bytes(m, d, k, 1)
    sizes = [4 * k * d, 4 * m * d, 4 * m * k, 4 * m * d, 4 * k * d, ws_bytes, int(B.lib.idkm_codes_bytes(m, k)), 4 * m * d]
    buf, offs = _carve(torch, sizes)
    p = [buf.data_ptr() + o for o in offs]
    Wd, C0d, Gd = (torch.from_numpy(x).cuda() for x in (W, C0, G))
    for loop_method in (0, 1):
        ctx = B.Context()
        ctx.set_forward_loop(loop_method)
        assert ctx.forward_raw(Wd.data_ptr(), m, d, C0d.data_ptr(), k, 0.01, 0.0, 5, p[0], p[2], p[1], p[5], ws_bytes) == 0
        assert ctx.backward_raw(Gd.data_ptr(), B.JFB, 0.0, 0, 1.0, p[3], p[4], p[5], ws_bytes) == 0
        assert ctx.backward_raw(Gd.data_ptr(), B.IMPLICIT, 0.0, 20, 1.0, p[3], p[4], p[5], ws_bytes) == 0
        ctx.set_adjoint_method(1)
        assert ctx.backward_raw(Gd.data_ptr(), B.IMPLICIT, 0.0, 3, 0.5, p[3], p[4], p[5], ws_bytes) == 0
        assert B.lib.idkm_assign(Wd.data_ptr(), m, d, p[0], k, p[6], p[7], None) == 0
        torch.cuda.synchronize()
        _check(torch, buf, offs, sizes)


def test_barrier_timeout_is_reported_and_the_context_survives():
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(20000, 1, 4, 0.01, std=0.03, seed=5)
    W, C0 = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    ctx = B.Context()
    good = ctx.forward(W, C0, wl.tau, 0.0, 6).C.cpu().numpy()
    assert ctx.info()[0].status == 0
    ctx.set_test_hooks(missing_arrivals=1, spin_limit_ticks=2000000)      # about a millisecond per wait
    try:
        ctx.forward(W, C0, wl.tau, 0.0, 6)
        torch.cuda.synchronize()
        info = ctx.info()[0]
        assert info.status == B.ERR_TIMEOUT and info.fwd_iters == 0
        assert "wait" in B.status_string(B.ERR_TIMEOUT)
    finally:
        ctx.set_test_hooks(0, 0)
    again = ctx.forward(W, C0, wl.tau, 0.0, 6).C.cpu().numpy()
    assert ctx.info()[0].status == 0 and ctx.info()[0].fwd_iters == 6
    assert np.array_equal(again, good)


@pytest.mark.parametrize("d,k", [(1, 4), (2, 8), (4, 4), (4, 16)])
def test_guard_words_around_a_batched_call(d, k):
    """The same for a batch of five layers (ragged sizes, a layer of one block, unaligned layer starts), on the
    one-launch loop and on the launch-per-iteration path, forward and both backward modes."""
    import ctypes
    import torch
    from paper_2312_07759_b200 import binding as B
    ms = [70001, 3000, 40000, 517, 131072]
    parts = [WL.single_layer(m, d, k, 0.004, std=0.02 + 0.01 * i, seed=31 + i) for i, m in enumerate(ms)]
    W = np.concatenate([p_.W for p_ in parts])
    C0 = np.concatenate([p_.C0 for p_ in parts])
    G = np.concatenate([p_.G for p_ in parts])
    L, m = len(ms), int(sum(ms))
    offs_host = (ctypes.c_int64 * (L + 1))(*np.concatenate([[0], np.cumsum(ms)]).tolist())
    ws_bytes = B.workspace_bytes(m, d, k, L)
    sizes = [4 * L * k * d, 4 * m * d, 4 * m * d, 4 * L * k * d, ws_bytes]       # C, Wq, dW, dC, workspace
    buf, offs = _carve(torch, sizes)
    p = [buf.data_ptr() + o for o in offs]
    Wd, C0d, Gd = (torch.from_numpy(x).cuda() for x in (W, C0, G))
    results = []
    for loop_method in (0, 1):
        ctx = B.Context()
        ctx.set_forward_loop(loop_method)
        rc = B.lib.idkm_forward_batched(ctx._h, Wd.data_ptr(), offs_host, L, d, C0d.data_ptr(), k, 0.004, 0.0, 7,
                                        p[0], None, p[1], p[4], ws_bytes, None)
        assert rc == 0
        assert ctx.backward_raw(Gd.data_ptr(), B.JFB, 0.0, 0, 1.0, p[2], p[3], p[4], ws_bytes) == 0
        assert ctx.backward_raw(Gd.data_ptr(), B.IMPLICIT, 0.0, 20, 1.0, p[2], p[3], p[4], ws_bytes) == 0
        torch.cuda.synchronize()
        ctx.n_layers = L
        # (seven iterations do not reach a fixed point, where the adjoint iteration need not contract: that status is
        # legitimate here)
        infos = ctx.info()
        assert all(i.status in (0, B.ERR_DIVERGED) and i.fwd_iters == 7 for i in infos), infos
        _check(torch, buf, offs, sizes)
        results.append(buf[offs[0]:offs[0] + sizes[0]].clone().view(torch.float32).cpu().numpy())
    assert np.abs(results[0] - results[1]).max() <= 2e-6 * np.abs(results[1]).max()
