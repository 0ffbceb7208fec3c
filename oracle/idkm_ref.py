"""ctypes front-end of the float64 C oracle (``idkm_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU
baseline; never by the CUDA package.  All arrays are float64 numpy, W [m, d], C [k, d].
The shared object is compiled on first use with gcc (compiling the checker is not using it).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "idkm_ref.c")
_LIB = os.path.join(_HERE, "libidkm_ref.so")

S_MIN = 1e-20


def build(force: bool = False) -> str:
    """Compile idkm_ref.c -> libidkm_ref.so (gcc -O2 -fopenmp; no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None
_dp = C.POINTER(C.c_double)
_ip = C.POINTER(C.c_int)


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.idkm_ref_threads.restype = C.c_int
    return _lib


def threads() -> int:
    return int(_L().idkm_ref_threads())


def set_threads(n: int) -> None:
    _L().idkm_ref_set_threads(C.c_int(n))


def set_squared(on: bool) -> None:
    """Switches the softmax to the squared distance D_ij = ||w_i - c_j||^2 (the variant in which the objectives of
    Sections 3.1 / 3.2 are written); off is the method as published."""
    _L().idkm_ref_set_squared(C.c_int(1 if on else 0))


def get_squared() -> bool:
    lib = _L()
    lib.idkm_ref_get_squared.restype = C.c_int
    return bool(lib.idkm_ref_get_squared())


class squared_distance:
    """``with squared_distance():`` runs the enclosed oracle calls with the squared-distance softmax."""

    def __init__(self, on: bool = True):
        self.on = on

    def __enter__(self):
        self.prev = get_squared()
        set_squared(self.on)
        return self

    def __exit__(self, *exc):
        set_squared(self.prev)
        return False


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(x: Optional[np.ndarray]):
    return None if x is None else x.ctypes.data_as(_dp)


def _shape(W, Cm) -> Tuple[int, int, int]:
    W = np.asarray(W)
    Cm = np.asarray(Cm)
    assert W.ndim == 2 and Cm.ndim == 2 and W.shape[1] == Cm.shape[1], (W.shape, Cm.shape)
    return W.shape[0], W.shape[1], Cm.shape[0]


def attention(W, Cm, tau: float) -> np.ndarray:
    W, Cm = _f64(W), _f64(Cm)
    m, d, k = _shape(W, Cm)
    A = np.empty((m, k))
    _L().idkm_ref_attention(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(A))
    return A


def sums(W, Cm, tau: float):
    W, Cm = _f64(W), _f64(Cm)
    m, d, k = _shape(W, Cm)
    S, N = np.empty(k), np.empty((k, d))
    _L().idkm_ref_sums(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(S), _p(N))
    return S, N


def step(W, Cm, tau: float):
    """One application of F.  Returns (C_plus, S, dead)."""
    W, Cm = _f64(W), _f64(Cm)
    m, d, k = _shape(W, Cm)
    Cp, S = np.empty((k, d)), np.empty(k)
    lib = _L()
    lib.idkm_ref_step.restype = C.c_int
    dead = lib.idkm_ref_step(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(Cp), _p(S))
    return Cp, S, int(dead)


def forward(W, C0, tau: float, tol: float, max_iter: int):
    """Algorithm 1.  Returns (C_T, iterations, last relative change, dead clusters)."""
    W, C0 = _f64(W), _f64(C0)
    m, d, k = _shape(W, C0)
    Co = np.empty((k, d))
    it, dead, res = C.c_int(0), C.c_int(0), C.c_double(0.0)
    _L().idkm_ref_forward(_p(W), C.c_int64(m), C.c_int(d), _p(C0), C.c_int(k), C.c_double(tau), C.c_double(tol),
                          C.c_int(max_iter), _p(Co), C.byref(it), C.byref(res), C.byref(dead))
    return Co, it.value, res.value, dead.value


def final(W, Cm, tau: float, want_A: bool = False, want_Wq: bool = True):
    """Final pass at C.  Returns (Wq or None, A or None, S, F)."""
    W, Cm = _f64(W), _f64(Cm)
    m, d, k = _shape(W, Cm)
    Wq = np.empty((m, d)) if want_Wq else None
    A = np.empty((m, k)) if want_A else None
    S, F = np.empty(k), np.empty((k, d))
    _L().idkm_ref_final(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(Wq), _p(A),
                        _p(S), _p(F))
    return Wq, A, S, F


def codebook_grad(W, G, Cm, tau: float) -> np.ndarray:
    W, G, Cm = _f64(W), _f64(G), _f64(Cm)
    m, d, k = _shape(W, Cm)
    g = np.empty((k, d))
    _L().idkm_ref_codebook_grad(_p(W), _p(G), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(g))
    return g


def adjoint_apply(W, Cm, tau: float, S, F, u) -> np.ndarray:
    W, Cm, S, F, u = _f64(W), _f64(Cm), _f64(S), _f64(F), _f64(u)
    m, d, k = _shape(W, Cm)
    out = np.empty((k, d))
    _L().idkm_ref_adjoint_apply(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(S), _p(F),
                                _p(u), _p(out))
    return out


def adjoint_solve(W, Cm, tau: float, S, F, g, alpha: float, adj_tol: float, adj_max_iter: int):
    """Returns (u, iterations, last relative change)."""
    W, Cm, S, F, g = _f64(W), _f64(Cm), _f64(S), _f64(F), _f64(g)
    m, d, k = _shape(W, Cm)
    u = np.empty((k, d))
    it, res = C.c_int(0), C.c_double(0.0)
    _L().idkm_ref_adjoint_solve(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(S), _p(F),
                                _p(g), C.c_double(alpha), C.c_double(adj_tol), C.c_int(adj_max_iter), _p(u),
                                C.byref(it), C.byref(res))
    return u, it.value, res.value


def adjoint_solve_restart(W, Cm, tau: float, S, F, g, alpha0: float, max_halvings: int, adj_tol: float,
                          adj_max_iter: int):
    """Section 4.2's safeguard: the watched iteration, restarted with half the alpha each time it diverges.
    Returns (u, diverged, alpha of the last attempt, attempts, iterations of the last attempt, last relative change)."""
    W, Cm, S, F, g = _f64(W), _f64(Cm), _f64(S), _f64(F), _f64(g)
    m, d, k = _shape(W, Cm)
    u = np.empty((k, d))
    it, att, res, al = C.c_int(0), C.c_int(0), C.c_double(0.0), C.c_double(0.0)
    lib = _L()
    lib.idkm_ref_adjoint_solve_restart.restype = C.c_int
    div = lib.idkm_ref_adjoint_solve_restart(_p(W), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(S),
                                             _p(F), _p(g), C.c_double(alpha0), C.c_int(max_halvings), C.c_double(adj_tol),
                                             C.c_int(adj_max_iter), _p(u), C.byref(al), C.byref(att), C.byref(it),
                                             C.byref(res))
    return u, bool(div), al.value, att.value, it.value, res.value


def scatter(W, G, Cm, tau: float, S, F, u) -> np.ndarray:
    W, G, Cm, S, F, u = _f64(W), _f64(G), _f64(Cm), _f64(S), _f64(F), _f64(u)
    m, d, k = _shape(W, Cm)
    dW = np.empty((m, d))
    _L().idkm_ref_scatter(_p(W), _p(G), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(S), _p(F),
                          _p(u), _p(dW))
    return dW


def backward(W, G, Cm, tau: float, S, F, mode: str = "implicit", alpha: float = 1.0, adj_tol: float = 0.0,
             adj_max_iter: int = 30, want_dW: bool = True):
    """Returns (dW or None, dC = u, adjoint iterations, last relative change).  mode: "implicit" | "jfb"."""
    W, G, Cm, S, F = _f64(W), _f64(G), _f64(Cm), _f64(S), _f64(F)
    m, d, k = _shape(W, Cm)
    dW = np.empty((m, d)) if want_dW else None
    dC = np.empty((k, d))
    it, res = C.c_int(0), C.c_double(0.0)
    _L().idkm_ref_backward(_p(W), _p(G), C.c_int64(m), C.c_int(d), _p(Cm), C.c_int(k), C.c_double(tau), _p(S),
                           _p(F), C.c_int({"implicit": 0, "jfb": 1}[mode]), C.c_double(alpha), C.c_double(adj_tol),
                           C.c_int(adj_max_iter), _p(dW), _p(dC), C.byref(it), C.byref(res))
    return dW, dC, it.value, res.value
