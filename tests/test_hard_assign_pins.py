"""Pins of the hard-quantiser oracle (oracle/hard_assign.py) against what the definition and the paper fix:
brute force, the tie rule, the d = 1 midpoint rule, the tau -> 0 limit of the soft quantiser (Section 3.1), and the
code format on a hand-computed example."""
import numpy as np

from oracle import hard_assign as H
from oracle import idkm_ref as R


def test_brute_force_and_ties():
    rng = np.random.default_rng(0)
    W = rng.standard_normal((23, 3))
    C = rng.standard_normal((5, 3))
    idx = H.hard_assign(W, C)
    for i in range(23):
        best, bd = -1, np.inf
        for j in range(5):
            dd = sum((W[i, a] - C[j, a]) ** 2 for a in range(3))
            if dd < bd:
                best, bd = j, dd
        assert idx[i] == best
    # a weight exactly between two centroids goes to the lower index; duplicated centroids too
    assert H.hard_assign(np.array([[0.0]]), np.array([[1.0], [-1.0], [1.0]]))[0] == 0
    assert H.hard_assign(np.array([[2.0, 0.0]]), np.array([[5.0, 0.0], [2.0, 3.0], [2.0, -3.0]]))[0] == 0


def test_scalar_weights_follow_the_midpoint_rule():
    rng = np.random.default_rng(1)
    c = np.sort(rng.standard_normal(7))
    w = rng.standard_normal(500)
    mids = 0.5 * (c[1:] + c[:-1])
    assert np.array_equal(H.hard_assign(w[:, None], c[:, None]), np.searchsorted(mids, w))


def test_soft_quantiser_tends_to_the_hard_one():
    """r_tau(w) -> q(w) as tau -> 0: with tau far below the smallest distance gap the soft-quantised weights equal
    the assigned centroids to exp(-gap / tau)."""
    rng = np.random.default_rng(2)
    W = rng.standard_normal((200, 2)) * 0.1
    C = rng.standard_normal((6, 2)) * 0.1
    idx = H.hard_assign(W, C)
    d = np.sqrt(H.squared_distances(W, C))
    gap = np.min(np.partition(d, 1, axis=1)[:, 1] - np.partition(d, 1, axis=1)[:, 0])
    tau = gap / 60.0
    Wq, _, _, _ = R.final(W, C, tau)
    assert np.max(np.abs(Wq - H.dequantize(idx, C))) < 1e-20 + 10 * np.exp(-60.0)
    # and the attention's argmax is the assignment at any tau
    A = R.attention(W, C, 0.05)
    assert np.array_equal(np.argmax(A, axis=1), idx)


def test_code_format():
    assert [H.code_bits(k) for k in (1, 2, 3, 4, 5, 16, 17, 256)] == [1, 1, 2, 2, 4, 4, 8, 8]
    # k = 4 (2 bits): codes 1, 2, 3, 0, 2 -> byte 0 = 1 | 2 << 2 | 3 << 4 | 0 << 6 = 57, byte 1 = 2
    assert H.pack_codes([1, 2, 3, 0, 2], 4).tolist() == [57, 2]
    # k = 2 (1 bit): 1,0,1,1,0,0,0,1, 1 -> 0b10001101 = 141, 1
    assert H.pack_codes([1, 0, 1, 1, 0, 0, 0, 1, 1], 2).tolist() == [141, 1]
    # k = 16 (4 bits): 10, 3, 15 -> 0x3A, 0x0F
    assert H.pack_codes([10, 3, 15], 16).tolist() == [0x3A, 0x0F]
    rng = np.random.default_rng(3)
    for k in (2, 3, 4, 9, 16, 100, 256):
        idx = rng.integers(0, k, size=1001)
        codes = H.pack_codes(idx, k)
        assert codes.shape[0] == (1001 * H.code_bits(k) + 7) // 8
        assert np.array_equal(H.unpack_codes(codes, 1001, k), idx)


def test_margins():
    W = np.array([[0.0], [0.9]])
    C = np.array([[0.0], [1.0], [3.0]])
    assert np.allclose(H.margins(W, C), [1.0, 0.81 - 0.01])
