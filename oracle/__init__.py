"""MUXQ oracle -- TEST INFRASTRUCTURE ONLY (numpy/ctypes front end of muxq_oracle.c).

The product (the CUDA library and its Python binding) never imports this package.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg do.  All arithmetic lives in the C
file; this module only marshals numpy arrays.  fp16 tensors are numpy float16 arrays (their raw
bits are handed to C unchanged).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "muxq_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

OK, ERR_ARG, ERR_NONFINITE, ERR_CAPACITY = 0, 1, 2, 5


def build(force: bool = False) -> str:
    """Compile muxq_oracle.c with gcc (plain -O2, OpenMP, no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-Wall",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_f16_to_f32.restype = ctypes.c_float
        _lib.oracle_f16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.oracle_f32_to_f16.restype = ctypes.c_uint16
        _lib.oracle_f32_to_f16.argtypes = [ctypes.c_float]
    return _lib


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def f16_to_f32(bits: int) -> float:
    return float(lib().oracle_f16_to_f32(int(bits)))


def f32_to_f16(v: float) -> int:
    return int(lib().oracle_f32_to_f16(float(v)))


def colmax(x: np.ndarray) -> np.ndarray:
    """Step 1: per-channel abs-max of X [M,K] fp16."""
    assert x.dtype == np.float16 and x.ndim == 2
    x = np.ascontiguousarray(x)
    M, K = x.shape
    out = np.empty(K, np.float32)
    rc = lib().oracle_colmax(_p(x), M, K, K, _p(out))
    if rc:
        raise ValueError(f"oracle_colmax rc={rc}")
    return out


def detect(cm: np.ndarray, tau: float, cap: int):
    """Step 2: ascending outlier channel indices; returns (O[:min(r,cap)], r, rc)."""
    cm = np.ascontiguousarray(cm, np.float32)
    O = np.zeros(max(cap, 1), np.int32)
    r = ctypes.c_int32(0)
    rc = lib().oracle_detect(_p(cm), cm.size, ctypes.c_float(tau), _p(O), cap, ctypes.byref(r))
    return O[: min(r.value, cap)].copy(), r.value, rc


def decompose(x: np.ndarray, O: np.ndarray, e: int):
    """Steps 3-4: Body [M,K] and Aux [M,r] in fp32 (Eq. 4, Eq. 5)."""
    x = np.ascontiguousarray(x)
    M, K = x.shape
    O = np.ascontiguousarray(O, np.int32)
    r = O.size
    body = np.empty((M, K), np.float32)
    aux = np.empty((M, max(r, 1)), np.float32)
    rc = lib().oracle_decompose(_p(x), M, K, K, _p(O), r, e, _p(body), _p(aux))
    assert rc == 0
    return body, aux[:, :r]


def quantize_act(body: np.ndarray, aux: np.ndarray, bits: int, per_token: bool, aux_own: bool):
    """Steps 5-6: returns s_x, s_a, body_q, aux_q."""
    body = np.ascontiguousarray(body, np.float32)
    M, K = body.shape
    r = aux.shape[1]
    auxc = np.ascontiguousarray(aux, np.float32) if r else np.zeros((M, 1), np.float32)
    ns = M if per_token else 1
    s_x = np.empty(ns, np.float32)
    s_a = np.empty(ns, np.float32)
    bq = np.empty((M, K), np.int8)
    aq = np.empty((M, max(r, 1)), np.int8)
    rc = lib().oracle_quantize_act(_p(body), _p(auxc), M, K, r, bits, int(per_token),
                                   int(aux_own), _p(s_x), _p(s_a), _p(bq), _p(aq))
    assert rc == 0
    if r:
        aq = np.ascontiguousarray(aq.reshape(-1)[: M * r].reshape(M, r))
    else:
        aq = np.zeros((M, 0), np.int8)
    return s_x, s_a, bq, aq


def quantize_weight(w: np.ndarray, bits: int = 8, per_channel: bool = False):
    """Step 7 (Eq. 2): W [K,N] fp16 -> (w_q [K,N] int8, s_w [1] or [N])."""
    assert w.dtype == np.float16 and w.ndim == 2
    w = np.ascontiguousarray(w)
    K, N = w.shape
    wq = np.empty((K, N), np.int8)
    s_w = np.empty(N if per_channel else 1, np.float32)
    rc = lib().oracle_quantize_weight(_p(w), K, N, N, bits, int(per_channel), _p(wq), _p(s_w))
    if rc:
        raise ValueError(f"oracle_quantize_weight rc={rc}")
    return wq, s_w


@dataclass
class LinearResult:
    rc: int
    colmax: np.ndarray
    O: np.ndarray
    r: int
    s_x: np.ndarray
    s_a: np.ndarray
    body_q: Optional[np.ndarray]
    aux_q: Optional[np.ndarray]  # [M, r]
    acc_b: np.ndarray
    acc_a: np.ndarray
    acc: np.ndarray
    y32: np.ndarray
    y16: np.ndarray  # float16 view of the RNE-rounded output


def linear(x: np.ndarray, w_q: np.ndarray, s_w: np.ndarray, *, tau: float = 6.0, e: int = 2,
           act_bits: int = 8, per_vector: bool = False, aux_own: bool = False, cap: int = 64,
           rows: Optional[np.ndarray] = None, want_codes: bool = True,
           bias: Optional[np.ndarray] = None) -> LinearResult:
    """Steps 1-6 and 8-10 for one call; w_q [K,N] and s_w come from quantize_weight.

    bias: optional fp32 [N], the layer's additive term (the GPT-2 projections of Section IV-C carry one): added to
    the dequantized fp32 value of Eq. 3 with one fp32 addition, before the cast to fp16.

    rows: optional int32 row subset for the products and the output (outputs are [len(rows), N]).
    """
    assert x.dtype == np.float16 and w_q.dtype == np.int8
    x = np.ascontiguousarray(x)
    w_q = np.ascontiguousarray(w_q)
    s_w = np.ascontiguousarray(s_w, np.float32)
    M, K = x.shape
    K2, N = w_q.shape
    assert K2 == K and s_w.size == (N if per_vector else 1)
    if rows is not None:
        rows = np.ascontiguousarray(rows, np.int32)
        n_rows = rows.size
    else:
        n_rows = M
    ns = M if per_vector else 1
    cm = np.empty(K, np.float32)
    O = np.zeros(max(cap, 1), np.int32)
    r = ctypes.c_int32(0)
    s_x = np.empty(ns, np.float32)
    s_a = np.empty(ns, np.float32)
    bq = np.empty((M, K), np.int8) if want_codes else None
    aq = np.zeros((M, max(cap, 1)), np.int8) if want_codes else None
    acc_b = np.empty((n_rows, N), np.int32)
    acc_a = np.empty((n_rows, N), np.int32)
    acc = np.empty((n_rows, N), np.int32)
    y32 = np.empty((n_rows, N), np.float32)
    y16 = np.empty((n_rows, N), np.uint16)
    rc = lib().oracle_linear(_p(x), M, K, K, _p(w_q), _p(s_w), N, ctypes.c_float(tau), e,
                             act_bits, int(per_vector), int(aux_own), cap, _p(rows), n_rows,
                             _p(cm), _p(O), ctypes.byref(r), _p(s_x), _p(s_a), _p(bq), _p(aq),
                             _p(acc_b), _p(acc_a), _p(acc), _p(y32), _p(y16))
    if rc not in (OK, ERR_CAPACITY):
        raise ValueError(f"oracle_linear rc={rc}")
    if bias is not None:
        b32 = np.ascontiguousarray(bias, np.float32).reshape(1, N)
        y32 = y32 + b32                       # float32 + float32: one IEEE addition per element, round to nearest even
        assert y32.dtype == np.float32
        with np.errstate(over="ignore"):
            y16 = y32.astype(np.float16).view(np.uint16)   # round to nearest even, overflow to infinity
    rr = r.value
    return LinearResult(rc, cm, O[: min(rr, cap)].copy(), rr, s_x, s_a, bq,
                        None if aq is None else aq[:, : min(rr, cap)].copy(), acc_b, acc_a, acc,
                        y32, y16.view(np.float16))
