"""Thin ctypes binding of the C-ABI library ``libidkm.so`` (see ``include/idkm.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch
supplies device memory (``tensor.data_ptr()``) and the current stream.  Importing this module
raises if the library has not been built; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libidkm.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2312_07759_b200.build` "
                      "(nvcc, sm_100a).  There is no fallback path.")
lib = C.CDLL(LIB_PATH)

IMPLICIT, JFB = 0, 1
OK, MAXITER = 0, 1
ERR_NULL, ERR_ALIGN, ERR_SHAPE, ERR_UNSUPPORTED, ERR_PARAM = -1, -2, -3, -4, -5
ERR_WORKSPACE, ERR_ORDER, ERR_CUDA, ERR_NONFINITE, ERR_DIVERGED = -6, -7, -8, -9, -10
ERR_NOALLOC_TOO_LARGE, ERR_TIMEOUT = -11, -12


class Info(C.Structure):
    _fields_ = [("status", C.c_int32), ("fwd_iters", C.c_int32), ("fwd_residual", C.c_float),
                ("dead_clusters", C.c_int32), ("adj_iters", C.c_int32), ("adj_residual", C.c_float)]

    def __repr__(self):
        return (f"Info(status={self.status}, fwd_iters={self.fwd_iters}, fwd_residual={self.fwd_residual:.3e}, "
                f"dead={self.dead_clusters}, adj_iters={self.adj_iters}, adj_residual={self.adj_residual:.3e})")


_vp, _i64p, _fp = C.c_void_p, C.POINTER(C.c_int64), C.c_void_p
lib.idkm_create.argtypes = [C.POINTER(_vp)]
lib.idkm_create.restype = C.c_int
lib.idkm_destroy.argtypes = [_vp]
lib.idkm_destroy.restype = None
lib.idkm_workspace_bytes.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int]
lib.idkm_workspace_bytes.restype = C.c_size_t
lib.idkm_forward.argtypes = [_vp, _fp, C.c_int64, C.c_int, _fp, C.c_int, C.c_float, C.c_float, C.c_int, _fp, _fp, _fp,
                             _vp, C.c_size_t, _vp]
lib.idkm_forward.restype = C.c_int
lib.idkm_forward_batched.argtypes = [_vp, _fp, _i64p, C.c_int, C.c_int, _fp, C.c_int, C.c_float, C.c_float, C.c_int,
                                     _fp, _fp, _fp, _vp, C.c_size_t, _vp]
lib.idkm_forward_batched.restype = C.c_int
lib.idkm_backward.argtypes = [_vp, _fp, C.c_int, C.c_float, C.c_int, C.c_float, _fp, _fp, _vp, C.c_size_t, _vp]
lib.idkm_backward.restype = C.c_int
lib.idkm_backward_restart.argtypes = [_vp, _fp, C.c_float, C.c_int, C.c_float, C.c_int, _fp, _fp, _vp, C.c_size_t, _vp,
                                      C.POINTER(C.c_float), C.POINTER(C.c_int)]
lib.idkm_backward_restart.restype = C.c_int
lib.idkm_get_info.argtypes = [_vp, C.POINTER(Info)]
lib.idkm_get_info.restype = C.c_int
lib.idkm_quantize_host.argtypes = [_vp, _fp, _i64p, C.c_int, C.c_int, _fp, C.c_int, C.c_float, C.c_float, C.c_int,
                                   _fp, C.c_int, C.c_float, C.c_int, C.c_float, _fp, _fp, _fp, _fp, C.POINTER(Info)]
lib.idkm_quantize_host.restype = C.c_int
lib.idkm_quantize_host_ex.argtypes = [_vp, _fp, _i64p, C.c_int, C.c_int, _fp, C.c_int, C.c_float, C.c_float, C.c_int,
                                      _fp, C.c_int, C.c_float, C.c_int, C.c_float, _fp, _fp, _fp, _fp, _fp, _fp,
                                      C.POINTER(Info)]
lib.idkm_quantize_host_ex.restype = C.c_int
lib.idkm_set_timing.argtypes = [_vp, C.c_int]
lib.idkm_set_timing.restype = C.c_int
lib.idkm_get_phase_ms.argtypes = [_vp, C.POINTER(C.c_float)]
lib.idkm_get_phase_ms.restype = C.c_int
lib.idkm_step_noalloc.argtypes = [_fp, C.c_int64, C.c_int, _fp, C.c_int, C.c_float, _fp, _vp]
lib.idkm_step_noalloc.restype = C.c_int
lib.idkm_step_noalloc_status.argtypes = [C.POINTER(C.c_int), _vp]
lib.idkm_step_noalloc_status.restype = C.c_int
lib.idkm_set_test_hooks.argtypes = [_vp, C.c_int, C.c_int64]
lib.idkm_set_test_hooks.restype = C.c_int
lib.idkm_count_busy_tickets.argtypes = [_vp, C.POINTER(C.c_int)]
lib.idkm_count_busy_tickets.restype = C.c_int
lib.idkm_set_wq_dtype.argtypes = [_vp, C.c_int]
lib.idkm_set_wq_dtype.restype = C.c_int
lib.idkm_set_collapse_step.argtypes = [_vp, C.c_int]
lib.idkm_set_collapse_step.restype = C.c_int
lib.idkm_set_distance.argtypes = [_vp, C.c_int]
lib.idkm_set_distance.restype = C.c_int
lib.idkm_set_adjoint_method.argtypes = [_vp, C.c_int]
lib.idkm_set_adjoint_method.restype = C.c_int
lib.idkm_get_history.argtypes = [_vp, C.c_int, C.c_int, C.POINTER(C.c_float), C.c_int, C.POINTER(C.c_int)]
lib.idkm_get_history.restype = C.c_int
lib.idkm_set_forward_loop.argtypes = [_vp, C.c_int]
lib.idkm_set_forward_loop.restype = C.c_int
lib.idkm_describe_path.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int)]
lib.idkm_describe_path.restype = C.c_int
lib.idkm_launch_count.argtypes = [_vp]
lib.idkm_launch_count.restype = C.c_int64
lib.idkm_measure_pipe_rates.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), _vp]
lib.idkm_measure_pipe_rates.restype = C.c_int
lib.idkm_assign.argtypes = [_fp, C.c_int64, C.c_int, _fp, C.c_int, _vp, _fp, _vp]
lib.idkm_assign.restype = C.c_int
lib.idkm_code_bits.argtypes = [C.c_int]
lib.idkm_code_bits.restype = C.c_int
lib.idkm_codes_bytes.argtypes = [C.c_int64, C.c_int]
lib.idkm_codes_bytes.restype = C.c_size_t
lib.idkm_status_string.argtypes = [C.c_int]
lib.idkm_status_string.restype = C.c_char_p


class IdkmError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"idkm status {code}: {status_string(code)}")


def status_string(code: int) -> str:
    return lib.idkm_status_string(int(code)).decode()


def _check(rc: int) -> None:
    if rc != OK:
        raise IdkmError(rc)


def workspace_bytes(m_total: int, d: int, k: int, n_layers: int = 1) -> int:
    return int(lib.idkm_workspace_bytes(int(m_total), int(d), int(k), int(n_layers)))


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    h = int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)
    return h if h != 0 else None


@dataclass
class ForwardResult:
    C: "object"          # torch [L*k, d]
    Wq: "object"         # torch [m, d] or None
    A: "object"          # torch [m, k] or None


def step_noalloc(W, C_in, tau: float, C_out=None, stream=None):
    """``idkm_step_noalloc``: C_out = F(C_in, W) on CUDA tensors without any allocation inside the library.
    The caller passes C_out to keep the call itself allocation-free; if omitted it is created here, by torch."""
    import torch
    assert W.is_cuda and C_in.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and C_in.is_contiguous()
    if C_out is None:
        C_out = torch.empty_like(C_in)
    _check(lib.idkm_step_noalloc(_ptr(W), int(W.shape[0]), int(W.shape[1]), _ptr(C_in), int(C_in.shape[0]),
                                 float(tau), _ptr(C_out), _stream(stream)))
    return C_out


def step_noalloc_status(stream=None) -> int:
    """``idkm_step_noalloc_status``: the device-side status of the last ``step_noalloc`` on the current device."""
    st = C.c_int(0)
    _check(lib.idkm_step_noalloc_status(C.byref(st), _stream(stream)))
    return int(st.value)


def assign(W, Cm, want_codes: bool = True, want_Wq: bool = True, stream=None):
    """``idkm_assign``: packed nearest-centroid codes (uint8 CUDA tensor) and dequantised weights of CUDA fp32 W."""
    import torch
    assert W.is_cuda and Cm.is_cuda and W.dtype == torch.float32 and Cm.dtype == torch.float32
    assert W.is_contiguous() and Cm.is_contiguous() and W.shape[1] == Cm.shape[1]
    m, d, k = int(W.shape[0]), int(W.shape[1]), int(Cm.shape[0])
    codes = torch.empty(int(lib.idkm_codes_bytes(m, k)), dtype=torch.uint8, device=W.device) if want_codes else None
    Wq = torch.empty_like(W) if want_Wq else None
    _check(lib.idkm_assign(_ptr(W), m, d, _ptr(Cm), k, _ptr(codes) if codes is not None else None,
                           _ptr(Wq) if Wq is not None else None, _stream(stream)))
    return codes, Wq


def describe_path(d: int, k: int, adj_max_iter: int = 0, adjoint_method: int = 0) -> dict:
    """``idkm_describe_path``: the kernel layouts and the adjoint route the library picks for (d, k)."""
    out = (C.c_int * 5)()
    _check(lib.idkm_describe_path(int(d), int(k), int(adj_max_iter), int(adjoint_method), out))
    return {"step_layout": (out[0], out[1]), "adjoint_layout": (out[2], out[3]),
            "adjoint_route": ("fused passes", "explicit Jacobian in registers", "explicit Jacobian in tiles",
                              "exact solve on the explicit Jacobian")[out[4]]}


def measure_pipe_rates(stream=None):
    """``idkm_measure_pipe_rates``: (fp32 FMA lane-operations/s, special-function lane-operations/s) measured now."""
    a, b = C.c_double(0.0), C.c_double(0.0)
    _check(lib.idkm_measure_pipe_rates(C.byref(a), C.byref(b), _stream(stream)))
    return float(a.value), float(b.value)


class Context:
    """One ``idkm_ctx``: remembers the last forward so that ``backward`` can follow it."""

    def __init__(self):
        h = _vp()
        _check(lib.idkm_create(C.byref(h)))
        self._h = h
        self._ws = None
        self._keep = None
        self.n_layers = 0
        self._wq_dtype = 0

    def close(self):
        if getattr(self, "_h", None):
            lib.idkm_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- raw calls (pointers as ints; used by the error-path tests) ------------------------------
    def forward_raw(self, W, m, d, C0, k, tau, tol, max_iter, C_out, A_out, Wq_out, ws, ws_bytes, stream=None) -> int:
        return int(lib.idkm_forward(self._h, W, m, d, C0, k, tau, tol, max_iter, C_out, A_out, Wq_out, ws, ws_bytes,
                                    stream))

    def backward_raw(self, dWq, mode, adj_tol, adj_max_iter, alpha, dW_out, dC_out, ws, ws_bytes, stream=None) -> int:
        return int(lib.idkm_backward(self._h, dWq, mode, adj_tol, adj_max_iter, alpha, dW_out, dC_out, ws, ws_bytes,
                                     stream))

    # -- tensor-level calls ---------------------------------------------------------------------
    def forward(self, W, C0, tau: float, tol: float, max_iter: int, *, layer_offsets: Optional[Sequence[int]] = None,
                want_Wq: bool = True, want_A: bool = False, stream=None) -> ForwardResult:
        """``idkm_forward`` / ``idkm_forward_batched`` on CUDA tensors W [m, d], C0 [L*k, d] (float32, contiguous)."""
        import torch
        assert W.is_cuda and C0.is_cuda and W.dtype == torch.float32 and C0.dtype == torch.float32
        assert W.is_contiguous() and C0.is_contiguous()
        m, d = int(W.shape[0]), int(W.shape[1])
        if layer_offsets is None:
            layer_offsets = [0, m]
        L = len(layer_offsets) - 1
        k = int(C0.shape[0]) // L
        nbytes = workspace_bytes(m, d, k, L)
        if nbytes == 0:
            raise IdkmError(ERR_UNSUPPORTED)
        if self._ws is None or self._ws.numel() < nbytes or self._ws.device != W.device:
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
        Cout = torch.empty_like(C0)
        wq_type = (torch.float32, torch.bfloat16, torch.float16)[self._wq_dtype]
        Wq = torch.empty(W.shape, dtype=wq_type, device=W.device) if want_Wq else None
        A = torch.empty((m, k), dtype=torch.float32, device=W.device) if want_A else None
        offs = (C.c_int64 * (L + 1))(*[int(x) for x in layer_offsets])
        rc = lib.idkm_forward_batched(self._h, _ptr(W), offs, L, d, _ptr(C0), k, float(tau), float(tol), int(max_iter),
                                      _ptr(Cout), _ptr(A), _ptr(Wq), _ptr(self._ws), self._ws.numel(), _stream(stream))
        _check(rc)
        self._keep = (W, Cout)   # the backward reads them
        self.n_layers = L
        self._shape = (m, d, k, L)
        return ForwardResult(Cout, Wq, A)

    def backward(self, dWq, mode: int = IMPLICIT, adj_tol: float = 0.0, adj_max_iter: int = 30, alpha: float = 1.0,
                 *, want_dW: bool = True, want_dC: bool = True, stream=None):
        """``idkm_backward``; returns (dW [m, d] or None, dC [L*k, d] or None)."""
        import torch
        assert dWq.is_cuda and dWq.dtype == torch.float32 and dWq.is_contiguous()
        if self._keep is None:
            raise IdkmError(ERR_ORDER)
        m, d, k, L = self._shape
        assert tuple(dWq.shape) == (m, d)
        dW = torch.empty_like(dWq) if want_dW else None
        dC = torch.empty((L * k, d), dtype=torch.float32, device=dWq.device) if want_dC else None
        rc = lib.idkm_backward(self._h, _ptr(dWq), int(mode), float(adj_tol), int(adj_max_iter), float(alpha), _ptr(dW),
                               _ptr(dC), _ptr(self._ws), self._ws.numel(), _stream(stream))
        _check(rc)
        return dW, dC

    def backward_restart(self, dWq, adj_tol: float, adj_max_iter: int, alpha0: float = 1.0, max_halvings: int = 4, *,
                         want_dW: bool = True, want_dC: bool = True, stream=None):
        """``idkm_backward_restart``; returns (dW or None, dC or None, alpha of the last attempt, attempts)."""
        import torch
        assert dWq.is_cuda and dWq.dtype == torch.float32 and dWq.is_contiguous()
        if self._keep is None:
            raise IdkmError(ERR_ORDER)
        m, d, k, L = self._shape
        dW = torch.empty_like(dWq) if want_dW else None
        dC = torch.empty((L * k, d), dtype=torch.float32, device=dWq.device) if want_dC else None
        al, att = C.c_float(0.0), C.c_int(0)
        _check(lib.idkm_backward_restart(self._h, _ptr(dWq), float(adj_tol), int(adj_max_iter), float(alpha0),
                                         int(max_halvings), _ptr(dW), _ptr(dC), _ptr(self._ws), self._ws.numel(),
                                         _stream(stream), C.byref(al), C.byref(att)))
        return dW, dC, float(al.value), int(att.value)

    def info(self) -> List[Info]:
        arr = (Info * max(1, self.n_layers))()
        _check(lib.idkm_get_info(self._h, arr))
        return list(arr)

    def quantize_host(self, W, C0, G, tau, tol, max_iter, mode=IMPLICIT, adj_tol=0.0, adj_max_iter=30, alpha=1.0,
                      layer_offsets=None, want_Wq=True, want_dW=True, out=None, also_jfb=False):
        """``idkm_quantize_host`` on HOST arrays (numpy float32, C-contiguous; pinned memory is the caller's choice).

        ``out`` may carry preallocated host arrays {"C", "Wq", "dW", "dC", "dW_jfb", "dC_jfb"} to write into.  With
        ``also_jfb`` (``idkm_quantize_host_ex``) the Jacobian-free gradients are computed from the same forward and
        returned as two more arrays after the info list."""
        import numpy as np
        m, d = W.shape
        if layer_offsets is None:
            layer_offsets = [0, m]
        L = len(layer_offsets) - 1
        k = C0.shape[0] // L
        out = {} if out is None else out
        Cout = out.get("C") if out.get("C") is not None else np.empty_like(C0)
        Wq = (out.get("Wq") if out.get("Wq") is not None else np.empty_like(W)) if want_Wq else None
        dW = (out.get("dW") if out.get("dW") is not None else np.empty_like(W)) if want_dW else None
        dC = out.get("dC") if out.get("dC") is not None else np.empty_like(C0)
        offs = (C.c_int64 * (L + 1))(*[int(x) for x in layer_offsets])
        infos = (Info * L)()
        hp = lambda a: None if a is None else a.ctypes.data
        if also_jfb:
            dWj = out.get("dW_jfb") if out.get("dW_jfb") is not None else np.empty_like(W)
            dCj = out.get("dC_jfb") if out.get("dC_jfb") is not None else np.empty_like(C0)
            rc = lib.idkm_quantize_host_ex(self._h, hp(W), offs, L, d, hp(C0), k, float(tau), float(tol), int(max_iter),
                                           hp(G), int(mode), float(adj_tol), int(adj_max_iter), float(alpha), hp(Cout),
                                           hp(Wq), hp(dW), hp(dC), hp(dWj), hp(dCj), infos)
            _check(rc)
            self.n_layers = L
            return Cout, Wq, dW, dC, list(infos), dWj, dCj
        rc = lib.idkm_quantize_host(self._h, hp(W), offs, L, d, hp(C0), k, float(tau), float(tol), int(max_iter), hp(G),
                                    int(mode), float(adj_tol), int(adj_max_iter), float(alpha), hp(Cout), hp(Wq), hp(dW),
                                    hp(dC), infos)
        _check(rc)
        self.n_layers = L
        return Cout, Wq, dW, dC, list(infos)

    def set_wq_dtype(self, dtype: int) -> None:
        """``idkm_set_wq_dtype``: 0 = Wq in fp32 (default), 1 = bfloat16, 2 = float16; ``forward`` then returns Wq as a
        tensor of that type."""
        _check(lib.idkm_set_wq_dtype(self._h, int(dtype)))
        self._wq_dtype = int(dtype)

    def set_collapse_step(self, method: int) -> None:
        """``idkm_set_collapse_step``: 0 = collapsing layers step in the fp32 increment form (default), 1 = in fp64."""
        _check(lib.idkm_set_collapse_step(self._h, int(method)))

    def set_distance(self, squared: bool) -> None:
        """``idkm_set_distance``: False = Euclidean distance in the softmax (Algorithm 1), True = its square."""
        _check(lib.idkm_set_distance(self._h, 1 if squared else 0))
        self._keep = None if squared != getattr(self, "_squared", False) else self._keep
        self._squared = bool(squared)

    def set_adjoint_method(self, method: int) -> None:
        """0: explicit Jacobian where k*d <= 64 (default); 1: always one fused pass per adjoint step; 2: exact solve
        on the explicit Jacobian where k*d <= 64."""
        _check(lib.idkm_set_adjoint_method(self._h, int(method)))

    def history(self, which: int = 0, layer: int = 0, capacity: int = 1024):
        """``idkm_get_history``: residuals of the last forward (which=0) or implicit backward (which=1) loop of a layer,
        as a float32 numpy array, first iteration first."""
        import numpy as np
        buf = (C.c_float * capacity)()
        n = C.c_int(0)
        _check(lib.idkm_get_history(self._h, int(which), int(layer), buf, int(capacity), C.byref(n)))
        return np.frombuffer(buf, dtype=np.float32, count=n.value).copy()

    def set_forward_loop(self, method: int) -> None:
        """0: small layers and batches of them run the whole forward loop in one cooperative launch (default); 1: a launch per iteration;
        2: a launch per iteration and never the kernel that steps fp32 and fp64 layers side by side; 3: as 2 with the
        rows of small-codebook layers streamed by bulk asynchronous copies."""
        _check(lib.idkm_set_forward_loop(self._h, int(method)))

    def set_test_hooks(self, missing_arrivals: int = 0, spin_limit_ticks: int = 0) -> None:
        """``idkm_set_test_hooks``: host-side fault injection for the timeout path; (0, 0) switches it off."""
        _check(lib.idkm_set_test_hooks(self._h, int(missing_arrivals), int(spin_limit_ticks)))

    def busy_tickets(self) -> int:
        """``idkm_count_busy_tickets``: arrival counters of the last forward's workspace that are not at rest."""
        n = C.c_int(0)
        _check(lib.idkm_count_busy_tickets(self._h, C.byref(n)))
        return int(n.value)

    def set_timing(self, enable: bool = True) -> None:
        _check(lib.idkm_set_timing(self._h, 1 if enable else 0))

    def phase_ms(self) -> dict:
        """Elapsed milliseconds per phase of the last forward / backward (``idkm_get_phase_ms``)."""
        arr = (C.c_float * 6)()
        _check(lib.idkm_get_phase_ms(self._h, arr))
        return dict(zip(("init", "steps", "final", "grad", "adjoint", "scatter"), [float(x) for x in arr]))

    @property
    def launches(self) -> int:
        return int(lib.idkm_launch_count(self._h))
