"""Hard assignment (idkm_assign) against the float64 oracle (B200 only).

The decision is taken on fp32 squared distances, the oracle's on float64 ones: where the two smallest distances of a
weight differ by more than the fp32 rounding of the computation the index must be the oracle's; elsewhere any
centroid within that rounding of the minimum is a valid answer.  The dequantised weights are the assigned
centroids bit for bit, and the bytes follow the oracle's code format."""
import numpy as np
import pytest

from oracle import hard_assign as H
from paper_2312_07759_b200 import workloads as WL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,d,k", [(1000, 1, 2), (4097, 1, 4), (50001, 2, 3), (100000, 4, 16), (200003, 4, 256),
                                   (33, 2, 7), (1 << 20, 1, 16), (7, 4, 1), (262147, 2, 200)])
def test_assign_matches_oracle(m, d, k):
    import torch
    from paper_2312_07759_b200 import binding as B
    wl = WL.single_layer(m, d, k, 0.01, std=0.05, seed=m % 1000 + k, init="rows" if d > 1 else "quantile")
    W, Cm = torch.from_numpy(wl.W).cuda(), torch.from_numpy(wl.C0).cuda()
    codes, Wq = B.assign(W, Cm)
    torch.cuda.synchronize()
    codes = codes.cpu().numpy()
    assert codes.shape[0] == (m * H.code_bits(k) + 7) // 8 == B.lib.idkm_codes_bytes(m, k)
    idx = H.unpack_codes(codes, m, k)
    assert idx.min() >= 0 and idx.max() < k
    ref = H.hard_assign(wl.W, wl.C0)
    scale = float(np.abs(wl.W).max() + np.abs(wl.C0).max())
    tol = 16 * d * np.finfo(np.float32).eps * scale * scale
    clear = H.margins(wl.W, wl.C0) > tol
    assert clear.mean() > 0.95
    assert np.array_equal(idx[clear], ref[clear])
    # the rest: a centroid whose float64 distance is within the rounding of the minimum
    amb = np.nonzero(~clear)[0]
    if amb.size:
        d2 = H.squared_distances(wl.W[amb], wl.C0)
        assert np.all(d2[np.arange(amb.size), idx[amb]] <= d2.min(axis=1) + tol)
    # dequantised weights: the assigned centroid, bit for bit; bytes: the oracle's format (unused bits zero)
    assert np.array_equal(Wq.cpu().numpy(), wl.C0[idx])
    assert np.array_equal(codes, H.pack_codes(idx, k)) if m <= 5000 else True
    # either output alone
    c2, none = B.assign(W, Cm, want_Wq=False)
    assert none is None and np.array_equal(c2.cpu().numpy(), codes)
    none, q2 = B.assign(W, Cm, want_codes=False)
    assert none is None and torch.equal(q2, Wq)


def test_assign_argument_errors():
    import torch
    from paper_2312_07759_b200 import binding as B
    W = torch.zeros(64, 2, device="cuda")
    Cm = torch.zeros(4, 2, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    f = B.lib.idkm_assign
    assert f(None, 64, 2, Cm.data_ptr(), 4, out.data_ptr(), None, None) == B.ERR_NULL
    assert f(W.data_ptr(), 64, 2, Cm.data_ptr(), 4, None, None, None) == B.ERR_NULL
    assert f(W.data_ptr(), 64, 3, Cm.data_ptr(), 4, out.data_ptr(), None, None) == B.ERR_UNSUPPORTED
    assert f(W.data_ptr(), 64, 2, Cm.data_ptr(), 257, out.data_ptr(), None, None) == B.ERR_UNSUPPORTED
    assert f(W.data_ptr(), 0, 2, Cm.data_ptr(), 4, out.data_ptr(), None, None) == B.ERR_SHAPE
    assert f(W.data_ptr(), 64, 2, Cm.data_ptr(), 4, None, W.data_ptr(), None) == B.ERR_PARAM
    assert B.lib.idkm_code_bits(0) == 0 and B.lib.idkm_code_bits(3) == 2 and B.lib.idkm_codes_bytes(9, 2) == 2
    torch.cuda.synchronize()
