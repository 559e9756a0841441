"""ctypes binding of libmuxq.so.  Function names and argument order follow include/muxq.h;
tensors are torch CUDA tensors whose data_ptr() is passed straight through."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmuxq.so")

MUXQ_OK, MUXQ_ERR_INVALID_ARG, MUXQ_ERR_UNSUPPORTED, MUXQ_ERR_WORKSPACE = 0, 1, 2, 3
MUXQ_ERR_CUDA, MUXQ_ERR_CAPACITY, MUXQ_ERR_TIMEOUT, MUXQ_ERR_STATIC_LIMIT = 4, 5, 6, 7
MUXQ_PER_TENSOR, MUXQ_PER_VECTOR = 0, 1
MUXQ_AUX_SHARED, MUXQ_AUX_OWN = 0, 1
MUXQ_OUT_F16, MUXQ_OUT_F32, MUXQ_OUT_ACC_I32 = 0, 1, 2

EXPORTS = (
    "muxq_default_params", "muxq_aux_cols", "muxq_workspace_bytes", "muxq_small_workspace_bytes",
    "muxq_host_workspace_bytes", "muxq_workspace_init", "muxq_workspace_view", "muxq_detect_outliers", "muxq_build_aux",
    "muxq_quantize", "muxq_gemm", "muxq_linear", "muxq_linear_bias", "muxq_linear_events", "muxq_linear_host",
    "muxq_linear_decode_noalloc", "muxq_int8_mma_peak", "muxq_test_hooks", "muxq_read_status",
    "muxq_chain_plan_bytes", "muxq_chain_device_bytes", "muxq_chain_build", "muxq_chain_run",
    "muxq_status_string",
)


class MuxqError(RuntimeError):
    def __init__(self, fn: str, status: int):
        super().__init__(f"{fn}: {muxq_status_string(status)} (status {status})")
        self.status = status


class _CParams(ctypes.Structure):
    _fields_ = [("threshold", ctypes.c_float), ("exp_factor", ctypes.c_int), ("act_bits", ctypes.c_int),
                ("w_bits", ctypes.c_int), ("gran", ctypes.c_int), ("aux_scale", ctypes.c_int),
                ("max_outliers", ctypes.c_int)]


class _CWsView(ctypes.Structure):
    _fields_ = [("col_absmax", ctypes.c_size_t), ("outlier_idx", ctypes.c_size_t),
                ("n_outliers", ctypes.c_size_t), ("s_x", ctypes.c_size_t), ("body_q", ctypes.c_size_t),
                ("aux_q", ctypes.c_size_t), ("w_aux", ctypes.c_size_t), ("s_a", ctypes.c_size_t),
                ("ld_body_q", ctypes.c_int), ("aux_cols", ctypes.c_int)]


@dataclass
class MuxqParams:
    threshold: float = 6.0
    exp_factor: int = 2
    act_bits: int = 8
    w_bits: int = 8
    gran: int = MUXQ_PER_TENSOR
    aux_scale: int = MUXQ_AUX_SHARED
    max_outliers: int = 64

    def c(self) -> _CParams:
        return _CParams(self.threshold, self.exp_factor, self.act_bits, self.w_bits, self.gran,
                        self.aux_scale, self.max_outliers)


_lib = None


def library_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """Loads libmuxq.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2604_04701_b200.build` "
                "(nvcc, sm_100a).  There is no CPU fallback.")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i, sz, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_float
        pp = ctypes.POINTER(_CParams)
        L.muxq_default_params.argtypes = [pp]; L.muxq_default_params.restype = None
        L.muxq_aux_cols.argtypes = [pp]; L.muxq_aux_cols.restype = i
        L.muxq_workspace_bytes.argtypes = [i, i, i, pp]; L.muxq_workspace_bytes.restype = sz
        L.muxq_small_workspace_bytes.argtypes = [i]; L.muxq_small_workspace_bytes.restype = sz
        L.muxq_host_workspace_bytes.argtypes = [i, i, i, pp, i]; L.muxq_host_workspace_bytes.restype = sz
        L.muxq_workspace_init.argtypes = [vp, sz, vp]; L.muxq_workspace_init.restype = i
        L.muxq_workspace_view.argtypes = [i, i, i, pp, ctypes.POINTER(_CWsView)]; L.muxq_workspace_view.restype = i
        L.muxq_detect_outliers.argtypes = [vp, i, i, i, f, vp, vp, vp, i, vp, sz, vp]; L.muxq_detect_outliers.restype = i
        L.muxq_build_aux.argtypes = [vp, i, i, i, vp, vp, i, i, vp, i, vp, i, vp]; L.muxq_build_aux.restype = i
        L.muxq_quantize.argtypes = [vp, i, i, i, pp, i, vp, vp, vp, vp, i, vp, i, vp, vp, sz, vp]; L.muxq_quantize.restype = i
        L.muxq_gemm.argtypes = [vp, i, vp, i, vp, i, vp, i, vp, i, i, i, pp, vp, vp, vp, i, i, vp, vp]; L.muxq_gemm.restype = i
        L.muxq_linear.argtypes = [vp, i, i, i, vp, i, vp, i, pp, vp, i, i, vp, sz, vp, vp]; L.muxq_linear.restype = i
        L.muxq_linear_bias.argtypes = [vp, i, i, i, vp, i, vp, vp, i, pp, vp, i, i, vp, sz, vp, vp]; L.muxq_linear_bias.restype = i
        L.muxq_linear_events.argtypes = [vp, i, i, i, vp, i, vp, i, pp, vp, i, i, vp, sz, vp, vp, vp]; L.muxq_linear_events.restype = i
        L.muxq_linear_host.argtypes = [vp, i, i, vp, i, vp, i, pp, vp, i, vp, sz, vp, vp]; L.muxq_linear_host.restype = i
        L.muxq_linear_decode_noalloc.argtypes = [vp, i, i, i, vp, i, vp, i, pp, vp, i, i, vp, vp]; L.muxq_linear_decode_noalloc.restype = i
        L.muxq_int8_mma_peak.argtypes = [i, i, i, vp, vp, vp]; L.muxq_int8_mma_peak.restype = i
        L.muxq_test_hooks.argtypes = [vp]; L.muxq_test_hooks.restype = i
        L.muxq_chain_plan_bytes.argtypes = [i]; L.muxq_chain_plan_bytes.restype = sz
        L.muxq_chain_device_bytes.argtypes = [vp, i, i]; L.muxq_chain_device_bytes.restype = sz
        L.muxq_chain_build.argtypes = [vp, i, i, pp, i, vp, sz, vp, sz, vp]; L.muxq_chain_build.restype = i
        L.muxq_chain_run.argtypes = [vp, vp, vp, vp, vp]; L.muxq_chain_run.restype = i
        L.muxq_read_status.argtypes = [vp, vp]; L.muxq_read_status.restype = i
        L.muxq_status_string.argtypes = [i]; L.muxq_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(fn: str, rc: int):
    if rc != MUXQ_OK:
        raise MuxqError(fn, rc)


def muxq_status_string(status: int) -> str:
    return lib().muxq_status_string(int(status)).decode()


def muxq_aux_cols(p: MuxqParams) -> int:
    return int(lib().muxq_aux_cols(ctypes.byref(p.c())))


def muxq_workspace_bytes(M: int, K: int, N: int, p: MuxqParams) -> int:
    return int(lib().muxq_workspace_bytes(M, K, N, ctypes.byref(p.c())))


def muxq_small_workspace_bytes(cols: int) -> int:
    return int(lib().muxq_small_workspace_bytes(cols))


def muxq_host_workspace_bytes(M: int, K: int, N: int, p: MuxqParams, out_kind: int) -> int:
    return int(lib().muxq_host_workspace_bytes(M, K, N, ctypes.byref(p.c()), out_kind))


def muxq_workspace_view(M: int, K: int, N: int, p: MuxqParams) -> _CWsView:
    v = _CWsView()
    _check("muxq_workspace_view", lib().muxq_workspace_view(M, K, N, ctypes.byref(p.c()), ctypes.byref(v)))
    return v


class Workspace:
    """Caller-owned device scratch (a torch uint8 tensor) plus the device status word."""

    def __init__(self, nbytes: int, device="cuda"):
        self.buf = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.init()

    def init(self) -> None:
        """muxq_workspace_init on the current stream (needed again after a time-out status or foreign writes);
        also zeroes the status word, which the library itself only ever raises."""
        with torch.cuda.device(self.buf.device):
            _check("muxq_workspace_init", lib().muxq_workspace_init(_ptr(self.buf), self.nbytes, _stream()))
            self.status.zero_()

    def clear_status(self) -> None:
        self.status.zero_()

    @property
    def nbytes(self) -> int:
        return self.buf.numel()


def muxq_detect_outliers(X: torch.Tensor, threshold: float, cap: int, ws: Workspace
                         ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Returns (col_absmax [K] f32, outlier_idx [cap] i32, n_outliers [1] i32), all on device."""
    assert X.is_cuda and X.dtype == torch.float16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    col_absmax = torch.empty(K, dtype=torch.float32, device=X.device)
    idx = torch.full((cap,), -1, dtype=torch.int32, device=X.device)
    n = torch.empty(1, dtype=torch.int32, device=X.device)
    _check("muxq_detect_outliers",
           lib().muxq_detect_outliers(_ptr(X), M, K, X.stride(0), float(threshold), _ptr(col_absmax), _ptr(idx),
                                      _ptr(n), cap, _ptr(ws.buf), ws.nbytes, _stream()))
    return col_absmax, idx, n


def muxq_build_aux(X: torch.Tensor, outlier_idx: torch.Tensor, n_outliers: torch.Tensor, exp_factor: int,
                   want_body: bool = True):
    """Real-domain Eq. 4-5: returns (Aux [M,cap] f32, Body [M,K] f32 or None)."""
    M, K = X.shape
    cap = outlier_idx.numel()
    aux = torch.empty(M, cap, dtype=torch.float32, device=X.device)
    body = torch.empty(M, K, dtype=torch.float32, device=X.device) if want_body else None
    _check("muxq_build_aux",
           lib().muxq_build_aux(_ptr(X), M, K, X.stride(0), _ptr(outlier_idx), _ptr(n_outliers), cap, exp_factor,
                                _ptr(aux), cap, _ptr(body), K, _stream()))
    return aux, body


def muxq_quantize(A: torch.Tensor, p: MuxqParams, is_weight: bool, ws: Workspace,
                  col_absmax: Optional[torch.Tensor] = None, outlier_idx: Optional[torch.Tensor] = None,
                  n_outliers: Optional[torch.Tensor] = None, want_aux: bool = True):
    """Weights: returns (W_q [N,K] i8, s_w).  Activations: returns (Body_q [M,K] i8, Aux_q [M,aux_cols] i8
    or None, s_x)."""
    assert A.is_cuda and A.dtype == torch.float16 and A.dim() == 2 and A.stride(1) == 1
    rows, cols = A.shape
    per_vec = p.gran == MUXQ_PER_VECTOR
    if is_weight:
        A_q = torch.empty(cols, rows, dtype=torch.int8, device=A.device)
        scales = torch.empty(cols if per_vec else 1, dtype=torch.float32, device=A.device)
        _check("muxq_quantize",
               lib().muxq_quantize(_ptr(A), rows, cols, A.stride(0), ctypes.byref(p.c()), 1, None, None, None,
                                   _ptr(A_q), rows, None, 0, _ptr(scales), _ptr(ws.buf), ws.nbytes, _stream()))
        return A_q, scales
    A_q = torch.empty(rows, cols, dtype=torch.int8, device=A.device)
    aux_cols = muxq_aux_cols(p)
    aux_q = torch.empty(rows, aux_cols, dtype=torch.int8, device=A.device) if want_aux else None
    scales = torch.empty(rows if per_vec else 1, dtype=torch.float32, device=A.device)
    _check("muxq_quantize",
           lib().muxq_quantize(_ptr(A), rows, cols, A.stride(0), ctypes.byref(p.c()), 0, _ptr(col_absmax),
                               _ptr(outlier_idx), _ptr(n_outliers), _ptr(A_q), cols, _ptr(aux_q), aux_cols,
                               _ptr(scales), _ptr(ws.buf), ws.nbytes, _stream()))
    return A_q, aux_q, scales


def _alloc_out(M: int, N: int, out_kind: int, device) -> torch.Tensor:
    dt = {MUXQ_OUT_F16: torch.float16, MUXQ_OUT_F32: torch.float32, MUXQ_OUT_ACC_I32: torch.int32}[out_kind]
    return torch.empty(M, N, dtype=dt, device=device)


def muxq_gemm(body_q: torch.Tensor, aux_q: Optional[torch.Tensor], w_q: torch.Tensor,
              w_aux: Optional[torch.Tensor], n_outliers: Optional[torch.Tensor], p: MuxqParams,
              s_x: Optional[torch.Tensor], s_w: Optional[torch.Tensor], out_kind: int, ws: Workspace,
              out: Optional[torch.Tensor] = None) -> torch.Tensor:
    M, K = body_q.shape
    N = w_q.shape[0]
    Y = out if out is not None else _alloc_out(M, N, out_kind, body_q.device)
    _check("muxq_gemm",
           lib().muxq_gemm(_ptr(body_q), body_q.stride(0), _ptr(aux_q), aux_q.stride(0) if aux_q is not None else 0,
                           _ptr(w_q), w_q.stride(0), _ptr(w_aux), w_aux.stride(0) if w_aux is not None else 0,
                           _ptr(n_outliers), M, K, N, ctypes.byref(p.c()), _ptr(s_x), _ptr(s_w), _ptr(Y),
                           Y.stride(0), out_kind, _ptr(ws.status), _stream()))
    return Y


def muxq_linear(X: torch.Tensor, w_q: torch.Tensor, s_w: torch.Tensor, p: MuxqParams, ws: Workspace,
                out_kind: int = MUXQ_OUT_F16, out: Optional[torch.Tensor] = None,
                bias: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Y = MUXQ-quantized X.W [+ bias]; w_q [N,K] int8 and s_w from muxq_quantize(is_weight=True); bias fp32 [N]."""
    assert X.is_cuda and X.dtype == torch.float16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    N = w_q.shape[0]
    Y = out if out is not None else _alloc_out(M, N, out_kind, X.device)
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float32 and bias.is_contiguous() and bias.numel() == N
        _check("muxq_linear_bias",
               lib().muxq_linear_bias(_ptr(X), M, K, X.stride(0), _ptr(w_q), w_q.stride(0), _ptr(s_w), _ptr(bias), N,
                                      ctypes.byref(p.c()), _ptr(Y), Y.stride(0), out_kind, _ptr(ws.buf), ws.nbytes,
                                      _ptr(ws.status), _stream()))
        return Y
    _check("muxq_linear",
           lib().muxq_linear(_ptr(X), M, K, X.stride(0), _ptr(w_q), w_q.stride(0), _ptr(s_w), N,
                             ctypes.byref(p.c()), _ptr(Y), Y.stride(0), out_kind, _ptr(ws.buf), ws.nbytes,
                             _ptr(ws.status), _stream()))
    return Y


def muxq_linear_events(X: torch.Tensor, w_q: torch.Tensor, s_w: torch.Tensor, p: MuxqParams, ws: Workspace,
                       events, out_kind: int = MUXQ_OUT_F16, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """muxq_linear recording four torch.cuda.Event objects (created with enable_timing=True and already
    recorded once, so that their CUDA handles exist) at the kernel boundaries."""
    M, K = X.shape
    N = w_q.shape[0]
    Y = out if out is not None else _alloc_out(M, N, out_kind, X.device)
    arr = (ctypes.c_void_p * 4)(*[ctypes.c_void_p(e.cuda_event) for e in events])
    _check("muxq_linear_events",
           lib().muxq_linear_events(_ptr(X), M, K, X.stride(0), _ptr(w_q), w_q.stride(0), _ptr(s_w), N,
                                    ctypes.byref(p.c()), _ptr(Y), Y.stride(0), out_kind, _ptr(ws.buf), ws.nbytes,
                                    _ptr(ws.status), _stream(), arr))
    return Y


def muxq_linear_host(X_host: torch.Tensor, w_q: torch.Tensor, s_w: torch.Tensor, p: MuxqParams, ws: Workspace,
                     Y_host: torch.Tensor, out_kind: int = MUXQ_OUT_F16) -> torch.Tensor:
    """X_host / Y_host are CPU tensors (pinned for asynchronous copies); everything else on device."""
    assert not X_host.is_cuda and not Y_host.is_cuda and X_host.is_contiguous() and Y_host.is_contiguous()
    M, K = X_host.shape
    N = w_q.shape[0]
    _check("muxq_linear_host",
           lib().muxq_linear_host(_ptr(X_host), M, K, _ptr(w_q), w_q.stride(0), _ptr(s_w), N, ctypes.byref(p.c()),
                                  _ptr(Y_host), out_kind, _ptr(ws.buf), ws.nbytes, _ptr(ws.status), _stream()))
    return Y_host


def muxq_linear_decode_noalloc(X: torch.Tensor, w_q: torch.Tensor, s_w: torch.Tensor, p: MuxqParams,
                               status: torch.Tensor, out_kind: int = MUXQ_OUT_F16,
                               out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """muxq_linear for M <= 16 rows and K <= 8192 channels with no workspace argument: the scratch is
    a fixed array inside the library, for callers that cannot allocate device memory at the call site.
    `out` should be given by such callers (otherwise torch allocates it); `status` is a device int32[1].
    Calls share the scratch, so keep them on one stream."""
    assert X.is_cuda and X.dtype == torch.float16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    N = w_q.shape[0]
    Y = out if out is not None else _alloc_out(M, N, out_kind, X.device)
    _check("muxq_linear_decode_noalloc",
           lib().muxq_linear_decode_noalloc(_ptr(X), M, K, X.stride(0), _ptr(w_q), w_q.stride(0), _ptr(s_w), N,
                                            ctypes.byref(p.c()), _ptr(Y), Y.stride(0), out_kind, _ptr(status),
                                            _stream()))
    return Y


def muxq_int8_mma_peak(mma_n: int, iters: int, ctas: int, ws: Workspace) -> torch.Tensor:
    """Enqueues the issue-bound INT8 MMA loop; returns the per-CTA cycle counts (device uint64 as int64)."""
    cycles = torch.zeros(ctas, dtype=torch.int64, device=ws.buf.device)
    _check("muxq_int8_mma_peak", lib().muxq_int8_mma_peak(mma_n, iters, ctas, _ptr(cycles), _ptr(ws.status), _stream()))
    return cycles


MUXQ_LAYER_WAIT_PREV = 1


class _CLayer(ctypes.Structure):
    _fields_ = [("X_f16", ctypes.c_void_p), ("W_q", ctypes.c_void_p), ("s_w", ctypes.c_void_p), ("Y", ctypes.c_void_p),
                ("ldx", ctypes.c_int), ("ldw", ctypes.c_int), ("ldy", ctypes.c_int), ("K", ctypes.c_int),
                ("N", ctypes.c_int), ("flags", ctypes.c_int), ("bias", ctypes.c_void_p)]


class Chain:
    """A list of decode-shaped layers run by one persistent launch (muxq_chain_build / muxq_chain_run).

    layers: sequence of (X [M,K] f16, w_q [N,K] i8, s_w, Y [M,N], flags[, bias f32 [N]]).  The tensors are kept alive by this
    object; results (one row of [r, status, s_x bits, 0] per layer, int32) and the status word live on the device."""

    def __init__(self, layers, p: MuxqParams, out_kind: int = MUXQ_OUT_F16):
        n = len(layers)
        self.layers = list(layers)
        self.M = int(layers[0][0].shape[0])
        dev = layers[0][0].device
        arr = (_CLayer * n)()
        for k, entry in enumerate(layers):
            X, w_q, s_w, Y, flags = entry[:5]
            bias = entry[5] if len(entry) > 5 else None
            assert X.is_cuda and X.dtype == torch.float16 and X.stride(1) == 1 and X.shape[0] == self.M
            assert bias is None or (bias.is_cuda and bias.dtype == torch.float32 and bias.numel() == w_q.shape[0])
            arr[k] = _CLayer(X.data_ptr(), w_q.data_ptr(), s_w.data_ptr(), Y.data_ptr(), X.stride(0), w_q.stride(0),
                             Y.stride(0), X.shape[1], w_q.shape[0], int(flags),
                             bias.data_ptr() if bias is not None else None)
        nbytes = int(lib().muxq_chain_plan_bytes(n))
        if nbytes == 0:
            raise MuxqError("muxq_chain_plan_bytes", MUXQ_ERR_INVALID_ARG)
        dbytes = int(lib().muxq_chain_device_bytes(arr, n, self.M))
        if dbytes == 0:
            raise MuxqError("muxq_chain_device_bytes", MUXQ_ERR_UNSUPPORTED)
        self.plan_host = (ctypes.c_uint8 * nbytes)()
        self.plan_dev = torch.empty(dbytes, dtype=torch.uint8, device=dev)
        self.results = torch.zeros(n, 4, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        with torch.cuda.device(dev):
            _check("muxq_chain_build",
                   lib().muxq_chain_build(arr, n, self.M, ctypes.byref(p.c()), out_kind, self.plan_host, nbytes,
                                          _ptr(self.plan_dev), dbytes, _stream()))
            torch.cuda.current_stream().synchronize()  # the copy has read plan_host

    def run(self) -> None:
        with torch.cuda.device(self.plan_dev.device):
            _check("muxq_chain_run", lib().muxq_chain_run(self.plan_host, _ptr(self.plan_dev), _ptr(self.results),
                                                          _ptr(self.status), _stream()))

    def read_status(self) -> int:
        return int(lib().muxq_read_status(_ptr(self.status), _stream()))


class _CTestHooks(ctypes.Structure):
    _fields_ = [("spin_limit", ctypes.c_uint32), ("prep_extra_arrivals", ctypes.c_uint32),
                ("gemm_skip_k_block", ctypes.c_int32)]


def muxq_test_hooks(spin_limit: int = 0, prep_extra_arrivals: int = 0, gemm_skip_k_block: int = 0) -> None:
    """Fault injection for tests (include/muxq_measure.h); all zero restores normal operation."""
    h = _CTestHooks(spin_limit, prep_extra_arrivals, gemm_skip_k_block)
    _check("muxq_test_hooks", lib().muxq_test_hooks(ctypes.byref(h)))


def muxq_read_status(ws: Workspace) -> int:
    return int(lib().muxq_read_status(_ptr(ws.status), _stream()))
