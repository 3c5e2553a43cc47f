"""ctypes/numpy front end of ``q8_oracle.c``.  TEST INFRASTRUCTURE ONLY.

The arithmetic lives in the C file; this module only builds it with gcc, marshals numpy
arrays into it and returns numpy arrays.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "q8_oracle.c")
_SO = os.path.join(_HERE, "libq8oracle.so")
_lib = None

GCC_FLAGS = ["-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc when the shared object is missing or older than the source."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        subprocess.check_call(["gcc", *GCC_FLAGS, _SRC, "-lm", "-o", _SO])
    return _SO


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        # Q8_ORACLE_SO lets the mutation test point the pins at a deliberately broken build of the oracle
        L = C.CDLL(os.environ.get("Q8_ORACLE_SO") or build())
        fp, i8p, i32p, dp = (C.POINTER(C.c_float), C.POINTER(C.c_int8), C.POINTER(C.c_int32),
                             C.POINTER(C.c_double))
        ip = C.POINTER(C.c_int)
        L.q8o_M.restype = C.c_int64
        L.q8o_M.argtypes = [C.c_int]
        L.q8o_absmax.restype = C.c_float
        L.q8o_absmax.argtypes = [fp, C.c_int64]
        L.q8o_scale_from_absmax.restype = C.c_float
        L.q8o_scale_from_absmax.argtypes = [C.c_float, ip]
        L.q8o_ema_update.restype = C.c_float
        L.q8o_ema_update.argtypes = [fp, i32p, C.c_float, C.c_float, ip]
        L.q8o_calibrate_batch.restype = C.c_float
        L.q8o_calibrate_batch.argtypes = [fp, i32p, fp, C.c_int64, C.c_float, ip]
        L.q8o_quantize.restype = None
        L.q8o_quantize.argtypes = [fp, C.c_int64, C.c_float, i8p]
        L.q8o_quantize_weight.restype = C.c_float
        L.q8o_quantize_weight.argtypes = [fp, C.c_int64, i8p, ip]
        L.q8o_gemm_s8.restype = C.c_int64
        L.q8o_gemm_s8.argtypes = [i8p, i8p, C.c_int64, C.c_int64, C.c_int64, i32p]
        L.q8o_quantize_bias.restype = None
        L.q8o_quantize_bias.argtypes = [fp, C.c_int64, C.c_float, C.c_float, i32p]
        L.q8o_add_bias.restype = C.c_int64
        L.q8o_add_bias.argtypes = [i32p, i32p, C.c_int64, C.c_int64]
        L.q8o_dequantize.restype = None
        L.q8o_dequantize.argtypes = [i32p, C.c_int64, C.c_float, C.c_float, dp]
        L.q8o_gelu.restype = None
        L.q8o_gelu.argtypes = [dp, C.c_int64]
        L.q8o_linear.restype = C.c_int
        L.q8o_linear.argtypes = [fp, i8p, C.c_float, C.c_float, fp, C.c_int, C.c_int64, C.c_int64,
                                 C.c_int64, i8p, i32p, dp, fp]
        L.q8o_linear_entry.restype = C.c_int32
        L.q8o_linear_entry.argtypes = [i8p, i8p, C.c_int64, C.c_int32]
        L.q8o_embedding.restype = C.c_int64
        L.q8o_embedding.argtypes = [i32p, C.c_int64, i8p, C.c_float, C.c_int64, C.c_int64, i8p, dp]
        L.q8o_add_layernorm.restype = None
        L.q8o_add_layernorm.argtypes = [fp, fp, fp, fp, fp, C.c_double, C.c_int64, C.c_int64, dp]
        L.q8o_attention.restype = None
        L.q8o_attention.argtypes = [fp, C.c_int64, C.c_int64, C.c_int64, C.c_int64, dp]
        L.q8o_fake_quantize.restype = None
        L.q8o_fake_quantize.argtypes = [fp, C.c_int64, C.c_float, dp]
        L.q8o_ste_backward.restype = None
        L.q8o_ste_backward.argtypes = [fp, C.c_int64, dp]
        _lib = L
    return _lib


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i8(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int8)


def M_of(b: int) -> int:
    return int(lib().q8o_M(int(b)))


def absmax(t) -> np.float32:
    t = _f32(t)
    return np.float32(lib().q8o_absmax(_p(t, C.c_float), t.size))


def scale_from_absmax(a):
    """Returns (S, flag)."""
    flag = C.c_int(0)
    s = lib().q8o_scale_from_absmax(C.c_float(float(np.float32(a))), C.byref(flag))
    return np.float32(s), int(flag.value)


class EmaState:
    """Eq. 4 running state: (ema, n_batches, S_x)."""

    def __init__(self):
        self.ema = np.zeros(1, np.float32)
        self.n = np.zeros(1, np.int32)
        self.S_x = np.float32(0)
        self.flag = 0

    def update(self, batch_absmax, decay) -> np.float32:
        flag = C.c_int(0)
        s = lib().q8o_ema_update(_p(self.ema, C.c_float), _p(self.n, C.c_int32),
                                 C.c_float(float(np.float32(batch_absmax))),
                                 C.c_float(float(np.float32(decay))), C.byref(flag))
        self.S_x = np.float32(s)
        self.flag |= int(flag.value)
        return self.S_x

    def update_batch(self, x, decay) -> np.float32:
        """Eq. 4 on one calibration batch given as a tensor (an empty batch changes nothing)."""
        x = _f32(x).ravel()
        flag = C.c_int(0)
        s = lib().q8o_calibrate_batch(_p(self.ema, C.c_float), _p(self.n, C.c_int32), _p(x, C.c_float), x.size,
                                      C.c_float(float(np.float32(decay))), C.byref(flag))
        self.S_x = np.float32(s)
        self.flag |= int(flag.value)
        return self.S_x


def quantize(x, S) -> np.ndarray:
    x = _f32(x)
    out = np.empty(x.shape, np.int8)
    lib().q8o_quantize(_p(x, C.c_float), x.size, C.c_float(float(np.float32(S))), _p(out, C.c_int8))
    return out


def quantize_weight(w):
    """Returns (W_q, S_w, flag)."""
    w = _f32(w)
    out = np.empty(w.shape, np.int8)
    flag = C.c_int(0)
    s = lib().q8o_quantize_weight(_p(w, C.c_float), w.size, _p(out, C.c_int8), C.byref(flag))
    return out, np.float32(s), int(flag.value)


def gemm_s8(xq, wq):
    """acc[m,n] = sum_k xq[m,k]*wq[n,k]; returns (acc int32 [M,N], n_overflow)."""
    xq, wq = _i8(xq), _i8(wq)
    M, K = xq.shape
    N, K2 = wq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    bad = lib().q8o_gemm_s8(_p(xq, C.c_int8), _p(wq, C.c_int8), M, N, K, _p(acc, C.c_int32))
    return acc, int(bad)


def quantize_bias(b, S_x, S_w) -> np.ndarray:
    b = _f32(b)
    out = np.empty(b.shape, np.int32)
    lib().q8o_quantize_bias(_p(b, C.c_float), b.size, C.c_float(float(np.float32(S_x))),
                            C.c_float(float(np.float32(S_w))), _p(out, C.c_int32))
    return out


def add_bias(acc, bq):
    acc = np.array(acc, dtype=np.int32, order="C", copy=True)
    bq = np.ascontiguousarray(bq, dtype=np.int32)
    M, N = acc.shape
    bad = lib().q8o_add_bias(_p(acc, C.c_int32), _p(bq, C.c_int32), M, N)
    return acc, int(bad)


def dequantize(acc, S_x, S_w) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    y = np.empty(acc.shape, np.float64)
    lib().q8o_dequantize(_p(acc, C.c_int32), acc.size, C.c_float(float(np.float32(S_x))),
                         C.c_float(float(np.float32(S_w))), _p(y, C.c_double))
    return y


def gelu(y) -> np.ndarray:
    y = np.array(y, dtype=np.float64, order="C", copy=True)
    lib().q8o_gelu(_p(y, C.c_double), y.size)
    return y


def linear(X, Wq, S_w, S_x=None, bias=None, act: int = 0):
    """Whole inference-mode quantised FC.  S_x None => dynamic scale (Sec. 4.1).

    Returns dict(xq, acc, y, S_x, flags)."""
    X, Wq = _f32(X), _i8(Wq)
    M, K = X.shape
    N, K2 = Wq.shape
    assert K == K2
    xq = np.empty((M, K), np.int8)
    acc = np.empty((M, N), np.int32)
    y = np.empty((M, N), np.float64)
    sx = np.zeros(1, np.float32)
    b = _f32(bias) if bias is not None else None
    r = lib().q8o_linear(_p(X, C.c_float), _p(Wq, C.c_int8), C.c_float(float(np.float32(S_w))),
                         C.c_float(-1.0 if S_x is None else float(np.float32(S_x))),
                         _p(b, C.c_float) if b is not None else None, int(act), M, N, K,
                         _p(xq, C.c_int8), _p(acc, C.c_int32), _p(y, C.c_double), _p(sx, C.c_float))
    return dict(xq=xq, acc=acc, y=y, S_x=np.float32(sx[0]), flags=int(r))


def linear_entry(xq_row, wq_row, bq: int) -> int:
    xq_row, wq_row = _i8(xq_row), _i8(wq_row)
    return int(lib().q8o_linear_entry(_p(xq_row, C.c_int8), _p(wq_row, C.c_int8), xq_row.size, int(bq)))


def embedding(ids, Eq, S_e):
    """Returns (rows_q int8 [T,H], out fp64 [T,H], n_bad_ids)."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    Eq = _i8(Eq)
    V, H = Eq.shape
    T = ids.size
    rows = np.empty((T, H), np.int8)
    out = np.empty((T, H), np.float64)
    bad = lib().q8o_embedding(_p(ids, C.c_int32), T, _p(Eq, C.c_int8), C.c_float(float(np.float32(S_e))),
                              V, H, _p(rows, C.c_int8), _p(out, C.c_double))
    return rows, out, int(bad)


def add_layernorm(x, r1=None, r2=None, gamma=None, beta=None, eps: float = 1e-12) -> np.ndarray:
    """fp64 LayerNorm(x + r1 + r2) * gamma + beta over the last dimension."""
    x = _f32(x)
    rows, H = x.shape
    opt = lambda a: _f32(a) if a is not None else None
    r1, r2, gamma, beta = opt(r1), opt(r2), opt(gamma), opt(beta)
    out = np.empty((rows, H), np.float64)
    pf = lambda a: _p(a, C.c_float) if a is not None else None
    lib().q8o_add_layernorm(_p(x, C.c_float), pf(r1), pf(r2), pf(gamma), pf(beta), float(eps), rows, H,
                            _p(out, C.c_double))
    return out


def attention(qkv, B: int, S: int, heads: int, d: int = 64) -> np.ndarray:
    """fp64 multi-head self-attention on the fused projection [B*S, 3*heads*d]; returns ctx [B*S, heads*d]."""
    qkv = _f32(qkv)
    assert qkv.shape == (B * S, 3 * heads * d)
    ctx = np.empty((B * S, heads * d), np.float64)
    lib().q8o_attention(_p(qkv, C.c_float), B, S, heads, d, _p(ctx, C.c_double))
    return ctx


def fake_quantize(x, S) -> np.ndarray:
    """Training-mode fake quantisation x_hat = Quantize(x | S) / S (fp64)."""
    x = _f32(x)
    out = np.empty(x.shape, np.float64)
    lib().q8o_fake_quantize(_p(x, C.c_float), x.size, C.c_float(float(np.float32(S))), _p(out, C.c_double))
    return out


def ste_backward(grad_out) -> np.ndarray:
    g = _f32(grad_out)
    out = np.empty(g.shape, np.float64)
    lib().q8o_ste_backward(_p(g, C.c_float), g.size, _p(out, C.c_double))
    return out
