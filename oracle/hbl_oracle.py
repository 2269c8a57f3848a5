"""ctypes front end of the CPU oracle (hbl_oracle.cpp).

TEST INFRASTRUCTURE, not product.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module; the CUDA path never does
and shares no code with it.  Each function wraps the C function of the same
name; see the C++ source for the equation each one restates.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hbl_oracle.cpp")
_LIB = os.path.join(_HERE, "libhbl_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2 -fopenmp).  No CUDA involved."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-std=c++17", "-shared", "-fPIC",
                               "-ffp-contract=off", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def weight_quant(W: np.ndarray, eps: float = 1e-5, prec: int = 32):
    """Eq. 1-2.  Returns (wt int8 [N,K], alpha float32)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    wt = np.empty((N, K), dtype=np.int8)
    alpha = C.c_float(0)
    _check(lib().orc_weight_quant(_p(W, C.c_float), C.c_long(N), C.c_long(K), C.c_float(eps),
                                  C.c_int(prec), _p(wt, C.c_int8), C.byref(alpha)), "weight_quant")
    return wt, np.float32(alpha.value)


def rmsnorm_bf16(x: np.ndarray, g: np.ndarray, eps_ln: float):
    """The "LN" of Eq. 7 read as RMS normalisation with a gain vector; fp64, one rounding to bf16.
    Returns (out float32 [T,K] holding bf16 values, pre float64 [T,K] before that rounding)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    g = np.ascontiguousarray(g, dtype=np.float32)
    T, K = x.shape
    assert g.shape == (K,)
    out = np.empty((T, K), dtype=np.float32)
    pre = np.empty((T, K), dtype=np.float64)
    _check(lib().orc_rmsnorm_bf16(_p(x, C.c_float), _p(g, C.c_float), C.c_long(T), C.c_long(K), C.c_float(eps_ln),
                                  _p(out, C.c_float), _p(pre, C.c_double)), "rmsnorm_bf16")
    return out, pre


def swiglu_bf16(gate: np.ndarray, up: np.ndarray):
    """SiLU(gate) * up in fp64, one rounding to bf16.  Returns (out float32 holding bf16 values, pre float64)."""
    gate = np.ascontiguousarray(gate, dtype=np.float32)
    up = np.ascontiguousarray(up, dtype=np.float32)
    assert gate.shape == up.shape
    T, K = gate.shape
    out = np.empty((T, K), dtype=np.float32)
    pre = np.empty((T, K), dtype=np.float64)
    _check(lib().orc_swiglu_bf16(_p(gate, C.c_float), _p(up, C.c_float), C.c_long(T), C.c_long(K),
                                 _p(out, C.c_float), _p(pre, C.c_double)), "swiglu_bf16")
    return out, pre


def kv_quant(x: np.ndarray, bits: int, eps: float = 1e-5, prec: int = 32, bits_row: np.ndarray | None = None):
    """Section 3.1: absmax quantizer at `bits` bits, one statistic per row (= one head of one token), unsigned
    codes u = q + 2^(bits-1).  x fp32 [R, D].  bits_row int32 [R] overrides the width per row (the [BOS] rows at 8).
    Returns (u uint8 [R,D], v fp64 pre-rounding [R,D], s fp64 [R])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    R, D = x.shape
    u = np.empty((R, D), dtype=np.uint8)
    v = np.empty((R, D), dtype=np.float64)
    s = np.empty((R,), dtype=np.float64)
    br = None if bits_row is None else np.ascontiguousarray(bits_row, dtype=np.int32)
    _check(lib().orc_kv_quant(_p(x, C.c_float), C.c_long(R), C.c_long(D), C.c_int(bits), _p(br, C.c_int), C.c_float(eps),
                              C.c_int(prec), _p(u, C.c_uint8), _p(v, C.c_double), _p(s, C.c_double)), "kv_quant")
    return u, v, s


def hadamard(x: np.ndarray) -> np.ndarray:
    """Eq. 3-4.  fp32 [T,K] -> fp64 [T,K], orthonormal, natural order."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    T, K = x.shape
    xr = np.empty((T, K), dtype=np.float64)
    _check(lib().orc_hadamard(_p(x, C.c_float), C.c_long(T), C.c_long(K), _p(xr, C.c_double)), "hadamard")
    return xr


def act_quant(xr: np.ndarray, bits: int, eps: float = 1e-5, prec: int = 32):
    """Eq. 5 / Eq. 6.  fp64 [T,K] -> (codes int8, v fp64 pre-rounding, s fp64 [T], stat fp64 [T])."""
    xr = np.ascontiguousarray(xr, dtype=np.float64)
    T, K = xr.shape
    q = np.empty((T, K), dtype=np.int8)
    v = np.empty((T, K), dtype=np.float64)
    s = np.empty((T,), dtype=np.float64)
    st = np.empty((T,), dtype=np.float64)
    _check(lib().orc_act_quant(_p(xr, C.c_double), C.c_long(T), C.c_long(K), C.c_int(bits),
                               C.c_float(eps), C.c_int(prec), _p(q, C.c_int8), _p(v, C.c_double),
                               _p(s, C.c_double), _p(st, C.c_double)), "act_quant")
    return q, v, s, st


def gemm(q: np.ndarray, wt: np.ndarray) -> np.ndarray:
    """Eq. 7 contraction.  codes int8 [T,K] x wt int8 [N,K] -> int32 [T,N]."""
    q = np.ascontiguousarray(q, dtype=np.int8)
    wt = np.ascontiguousarray(wt, dtype=np.int8)
    T, K = q.shape
    N, K2 = wt.shape
    assert K == K2
    acc = np.empty((T, N), dtype=np.int32)
    _check(lib().orc_gemm(_p(q, C.c_int8), _p(wt, C.c_int8), C.c_long(T), C.c_long(K), C.c_long(N),
                          _p(acc, C.c_int32)), "gemm")
    return acc


def rescale(acc: np.ndarray, s: np.ndarray, alpha: float):
    """y = alpha * s_t * acc -> (bf16 bits uint16 [T,N], unrounded fp64 [T,N])."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    s = np.ascontiguousarray(s, dtype=np.float64)
    T, N = acc.shape
    yb = np.empty((T, N), dtype=np.uint16)
    y64 = np.empty((T, N), dtype=np.float64)
    _check(lib().orc_rescale(_p(acc, C.c_int32), _p(s, C.c_double), C.c_float(alpha), C.c_long(T),
                             C.c_long(N), _p(yb, C.c_uint16), _p(y64, C.c_double)), "rescale")
    return yb, y64


def forward(x: np.ndarray, wt: np.ndarray, alpha: float, bits: int, use_hadamard: bool,
            eps: float = 1e-5, prec: int = 32, want_stages: bool = False):
    """Eq. 3-7 chained for fp32 x [T,K] against ternary wt [N,K].

    Returns a dict with y_bits (uint16 bf16 patterns), y64, and, if asked,
    codes, acc and s."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    wt = np.ascontiguousarray(wt, dtype=np.int8)
    T, K = x.shape
    N = wt.shape[0]
    yb = np.empty((T, N), dtype=np.uint16)
    y64 = np.empty((T, N), dtype=np.float64)
    codes = np.empty((T, K), dtype=np.int8) if want_stages else None
    acc = np.empty((T, N), dtype=np.int32) if want_stages else None
    s = np.empty((T,), dtype=np.float64)
    _check(lib().orc_forward(_p(x, C.c_float), C.c_long(T), C.c_long(K), _p(wt, C.c_int8),
                             C.c_float(alpha), C.c_long(N), C.c_int(bits), C.c_int(int(use_hadamard)),
                             C.c_float(eps), C.c_int(prec), _p(yb, C.c_uint16), _p(y64, C.c_double),
                             _p(codes, C.c_int8), _p(acc, C.c_int32), _p(s, C.c_double)), "forward")
    return {"y_bits": yb, "y64": y64, "codes": codes, "acc": acc, "s": s}


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
