"""ctypes binding of ``libq8.so``: same names as ``include/q8.h``, argument marshalling only.

Every function takes torch tensors that already live on the CUDA device (torch supplies device
memory and streams, nothing else), checks dtype / device / contiguity, passes raw pointers to
the C ABI and raises :class:`Q8Error` on a non-zero status.  There is no CPU fallback: if the
shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libq8.so")

Q8_OK, Q8_ERR_NULL, Q8_ERR_SHAPE, Q8_ERR_ALIGN, Q8_ERR_SCALE, Q8_ERR_INDEX = 0, 1, 2, 3, 4, 5
Q8_ERR_OVERFLOW, Q8_ERR_WORKSPACE, Q8_ERR_TIMEOUT, Q8_ERR_CUDA, Q8_ERR_ARG = 6, 7, 8, 9, 10
Q8_ACT_NONE, Q8_ACT_GELU = 0, 1
Q8_MAX_K = 133144

# name -> (restype, argtypes); mirrors include/q8.h and include/q8_tools.h one to one.
_vp, _i64, _sz, _int, _f = C.c_void_p, C.c_int64, C.c_size_t, C.c_int, C.c_float
SIGNATURES = {
    "q8_quantize_weight": (_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp]),
    "q8_quantize_activation": (_int, [_vp, _i64, _vp, _vp, _vp, _vp, _vp]),
    "q8_fake_quantize": (_int, [_vp, _i64, _vp, _vp, _vp]),
    "q8_ste_backward": (_int, [_vp, _i64, _vp, _vp]),
    "q8_calibrate": (_int, [_vp, _i64, _f, _vp, _vp]),
    "q8_calibrate_state_bytes": (_sz, []),
    "q8_linear": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _i64, _i64, _i64, _vp, _sz, _vp, _vp, _vp]),
    "q8_linear_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "q8_linear_q": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "q8_linear_generic": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _i64, _i64, _i64, _vp, _sz, _vp, _vp, _vp]),
    "q8_linear_noalloc": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _i64, _i64, _i64, _vp, _vp, C.POINTER(_vp), _vp]),
    "q8_embedding": (_int, [_vp, _i64, _vp, _vp, _i64, _i64, _vp, _vp, _vp, _vp]),
    "q8_add_layernorm": (_int, [_vp, _vp, _vp, _vp, _vp, _f, _i64, _i64, _vp, _vp]),
    "q8_attention": (_int, [_vp, _i64, _i64, _i64, _vp, _vp]),
    "q8_add_layernorm_absmax": (_int, [_vp, _vp, _vp, _vp, _vp, _f, _i64, _i64, _vp, _vp, _vp]),
    "q8_attention_absmax": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "q8_linear_dyn": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _vp, _i64, _i64, _i64, _vp, _sz, _vp, _vp, _vp]),
    "q8_quantize_weight_segments": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "q8_linear_wseg": (_int, [_vp, _vp, _vp, _i64, _vp, _vp, _int, _vp, _i64, _i64, _i64, _vp, _sz, _vp, _vp, _vp]),
    "q8_linear_q_wseg": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _int, _vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "q8_linear_requant": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _sz, _vp, _vp, _vp]),
    "q8_linear_q_requant": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "q8_add_layernorm_quant": (_int, [_vp, _vp, _vp, _vp, _vp, _f, _i64, _i64, _vp, _vp, _vp, _vp]),
    "q8_attention_quant": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "q8_poll_status": (_int, [_vp, C.POINTER(C.c_uint32), _vp]),
    "q8_status_string": (C.c_char_p, [_int]),
    "q8_last_launch_info": (None, [C.POINTER(_int)] * 5),
    "q8_tune_gemm_tile": (_int, [_int, _int]),
    "q8_tune_gemm_tail_split": (None, [_int]),
    "q8_tune_gemm_direct_store": (None, [_int]),
    "q8_tune_attention": (None, [_int]),
    "q8_selftest_wait_timeout": (_int, [C.c_uint64, _vp, _vp, _vp]),
    "q8_attention_status_word": (_int, [C.POINTER(C.c_void_p)]),
    "q8_tune_gemm_epilogue_warps": (_int, [_int]),
    "q8_last_launch_tail_split": (_int, []),
    "q8_last_launch_store_mode": (_int, []),
    "q8_measure_hbm_peak": (_int, [C.c_void_p, C.c_size_t, _int, _int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                   C.c_void_p]),
    "q8_measure_l2_operand_peak": (_int, [C.c_void_p, C.c_int64, C.c_int64, _int, _int, _int, C.POINTER(C.c_double),
                                          C.POINTER(C.c_double), C.c_void_p]),
    "q8_measure_int8_mma_peak": (_int, [_int, C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(_int),
                                        C.c_void_p, C.c_void_p]),
}

_lib: Optional[C.CDLL] = None


class Q8Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: q8_status {status} ({status_string(status)})")


def load() -> C.CDLL:
    """Loads libq8.so (built by ``python -m paper_1910_06188_b200.build``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build the CUDA library first "
                "(python -m paper_1910_06188_b200.build); there is no CPU fallback")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().q8_status_string(int(status)).decode()


# ---------------------------------------------------------------- marshalling helpers
def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous")
    return t.data_ptr()


def _any_ptr(t: Optional[torch.Tensor], name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA tensor")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _check(status: int, where: str) -> None:
    if status != Q8_OK:
        raise Q8Error(status, where)


# ---------------------------------------------------------------- the calls
def q8_quantize_weight(W: torch.Tensor, Wq: Optional[torch.Tensor] = None, S_w: Optional[torch.Tensor] = None,
                       dev_status: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Eq. 3 + Eq. 1 on a weight (or embedding table) [N, K]; returns (W_q int8, S_w fp32[1])."""
    N, K = W.shape
    if Wq is None:
        Wq = torch.empty((N, K), dtype=torch.int8, device=W.device)
    if S_w is None:
        S_w = torch.empty(1, dtype=torch.float32, device=W.device)
    st = load().q8_quantize_weight(_ptr(W, torch.float32, "W"), N, K, _ptr(Wq, torch.int8, "Wq"),
                                   _ptr(S_w, torch.float32, "S_w"), _ptr(dev_status, torch.int32, "dev_status"),
                                   _stream(stream))
    _check(st, "q8_quantize_weight")
    return Wq, S_w


def q8_quantize_activation(X: torch.Tensor, S_x: Optional[torch.Tensor] = None, Xq: Optional[torch.Tensor] = None,
                           S_x_used: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                           stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Eq. 1 on an activation; S_x None selects the dynamic scale.  Returns (X_q, scale used)."""
    if Xq is None:
        Xq = torch.empty(X.shape, dtype=torch.int8, device=X.device)
    if S_x is None and S_x_used is None:
        S_x_used = torch.empty(1, dtype=torch.float32, device=X.device)
    st = load().q8_quantize_activation(_ptr(X, torch.float32, "X"), X.numel(), _ptr(S_x, torch.float32, "S_x"),
                                       _ptr(Xq, torch.int8, "Xq"), _ptr(S_x_used, torch.float32, "S_x_used"),
                                       _ptr(dev_status, torch.int32, "dev_status"), _stream(stream))
    _check(st, "q8_quantize_activation")
    return Xq, (S_x_used if S_x_used is not None else S_x)


def q8_fake_quantize(X, S, Xhat=None, stream=None):
    """Training-mode fake quantisation: Xhat = Quantize(X | S) / S."""
    if Xhat is None:
        Xhat = torch.empty_like(X)
    st = load().q8_fake_quantize(_ptr(X, torch.float32, "X"), X.numel(), _ptr(S, torch.float32, "S"),
                                 _ptr(Xhat, torch.float32, "Xhat"), _stream(stream))
    _check(st, "q8_fake_quantize")
    return Xhat


def q8_ste_backward(grad_out, grad_in=None, stream=None):
    """Straight-through estimator (Eq. 5): the gradient of fake quantisation is the incoming gradient."""
    if grad_in is None:
        grad_in = torch.empty_like(grad_out)
    st = load().q8_ste_backward(_ptr(grad_out, torch.float32, "grad_out"), grad_out.numel(),
                                _ptr(grad_in, torch.float32, "grad_in"), _stream(stream))
    _check(st, "q8_ste_backward")
    return grad_in


def q8_calibrate_state_bytes() -> int:
    return int(load().q8_calibrate_state_bytes())


def new_calibrate_state(device="cuda") -> torch.Tensor:
    """Zero-initialised Eq. 4 state block, viewed as int32 words: [ema, S_x, n_batches, scratch, status, ...]."""
    return torch.zeros(q8_calibrate_state_bytes() // 4, dtype=torch.int32, device=device)


def calibrate_S_x(state: torch.Tensor) -> torch.Tensor:
    """fp32[1] view of the S_x word inside a calibrate state (usable as q8_linear's S_x)."""
    return state.view(torch.float32)[1:2]


def q8_calibrate(X: torch.Tensor, decay: float, state: torch.Tensor, stream=None) -> None:
    st = load().q8_calibrate(_ptr(X, torch.float32, "X"), X.numel(), float(decay), _any_ptr(state, "state"),
                             _stream(stream))
    _check(st, "q8_calibrate")


def q8_linear_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(load().q8_linear_workspace_bytes(M, N, K))


def new_workspace(M: int, N: int, K: int, device="cuda") -> torch.Tensor:
    return torch.empty(q8_linear_workspace_bytes(M, N, K), dtype=torch.uint8, device=device)


def _linear(fn_name: str, X, Wq, S_w, S_x, bias, act, Y, workspace, dbg_Xq, dbg_acc, stream):
    M, K = X.shape
    N, K2 = Wq.shape
    if K != K2:
        raise ValueError(f"X is [M,{K}] but Wq is [N,{K2}]")
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=X.device)
    if workspace is None:
        workspace = new_workspace(M, N, K, X.device)
    fn = getattr(load(), fn_name)
    st = fn(_ptr(X, torch.float32, "X"), _ptr(Wq, torch.int8, "Wq"), _ptr(S_w, torch.float32, "S_w"),
            _ptr(S_x, torch.float32, "S_x"), _ptr(bias, torch.float32, "bias"), int(act),
            _ptr(Y, torch.float32, "Y"), M, N, K, _any_ptr(workspace, "workspace"),
            workspace.numel() * workspace.element_size(), _ptr(dbg_Xq, torch.int8, "dbg_Xq"),
            _ptr(dbg_acc, torch.int32, "dbg_acc"), _stream(stream))
    _check(st, fn_name)
    return Y


def q8_linear(X, Wq, S_w, S_x=None, bias=None, act: int = Q8_ACT_NONE, Y=None, workspace=None, dbg_Xq=None,
              dbg_acc=None, stream=None) -> torch.Tensor:
    """Inference-mode quantised FC (Sec. 3): quantise X, Int8 GEMM, Int32 bias, dequantise, act."""
    return _linear("q8_linear", X, Wq, S_w, S_x, bias, act, Y, workspace, dbg_Xq, dbg_acc, stream)


def q8_linear_generic(X, Wq, S_w, S_x=None, bias=None, act: int = Q8_ACT_NONE, Y=None, workspace=None, dbg_Xq=None,
                      dbg_acc=None, stream=None) -> torch.Tensor:
    return _linear("q8_linear_generic", X, Wq, S_w, S_x, bias, act, Y, workspace, dbg_Xq, dbg_acc, stream)


def q8_linear_q(Xq, S_x, Wq, S_w, bias=None, act: int = Q8_ACT_NONE, Y=None, dbg_acc=None, dev_status=None,
                stream=None) -> torch.Tensor:
    M, K = Xq.shape
    N, K2 = Wq.shape
    if K != K2:
        raise ValueError(f"Xq is [M,{K}] but Wq is [N,{K2}]")
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=Xq.device)
    st = load().q8_linear_q(_ptr(Xq, torch.int8, "Xq"), _ptr(S_x, torch.float32, "S_x"), _ptr(Wq, torch.int8, "Wq"),
                            _ptr(S_w, torch.float32, "S_w"), _ptr(bias, torch.float32, "bias"), int(act),
                            _ptr(Y, torch.float32, "Y"), M, N, K, _ptr(dbg_acc, torch.int32, "dbg_acc"),
                            _ptr(dev_status, torch.int32, "dev_status"), _stream(stream))
    _check(st, "q8_linear_q")
    return Y


Q8_NOALLOC_MAX_MK = 16 * 1024 * 1024


def q8_linear_noalloc(X, Wq, S_w, S_x=None, bias=None, act: int = Q8_ACT_NONE, Y=None, dbg_Xq=None, dbg_acc=None,
                      stream=None):
    """q8_linear without a caller workspace: for callers that may not allocate device memory (the scratch
    is a fixed array inside the library, M*K <= Q8_NOALLOC_MAX_MK).  Y must be supplied by such callers;
    when it is None this binding allocates it with torch for convenience.  Returns (Y, status_word_address)."""
    M, K = X.shape
    N, K2 = Wq.shape
    if K != K2:
        raise ValueError(f"X is [M,{K}] but Wq is [N,{K2}]")
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=X.device)
    word = C.c_void_p(0)
    st = load().q8_linear_noalloc(_ptr(X, torch.float32, "X"), _ptr(Wq, torch.int8, "Wq"),
                                  _ptr(S_w, torch.float32, "S_w"), _ptr(S_x, torch.float32, "S_x"),
                                  _ptr(bias, torch.float32, "bias"), int(act), _ptr(Y, torch.float32, "Y"), M, N, K,
                                  _ptr(dbg_Xq, torch.int8, "dbg_Xq"), _ptr(dbg_acc, torch.int32, "dbg_acc"),
                                  C.byref(word), _stream(stream))
    _check(st, "q8_linear_noalloc")
    return Y, word.value


def q8_poll_status_at(address: int, stream=None) -> Tuple[int, int]:
    """q8_poll_status on a raw device address (e.g. the status word returned by q8_linear_noalloc)."""
    raw = C.c_uint32(0)
    st = load().q8_poll_status(C.c_void_p(address), C.byref(raw), _stream(stream))
    return int(st), int(raw.value)


def q8_embedding(ids, Eq, S_e, out=None, rows_q=None, dev_status=None, stream=None) -> torch.Tensor:
    T = ids.numel()
    V, H = Eq.shape
    if out is None:
        out = torch.empty((T, H), dtype=torch.float32, device=Eq.device)
    st = load().q8_embedding(_ptr(ids, torch.int32, "ids"), T, _ptr(Eq, torch.int8, "Eq"),
                             _ptr(S_e, torch.float32, "S_e"), V, H, _ptr(out, torch.float32, "out"),
                             _ptr(rows_q, torch.int8, "rows_q"), _ptr(dev_status, torch.int32, "dev_status"),
                             _stream(stream))
    _check(st, "q8_embedding")
    return out


def q8_add_layernorm(x, r1=None, r2=None, gamma=None, beta=None, eps: float = 1e-12, out=None, stream=None):
    """out = LayerNorm(x + r1 + r2) * gamma + beta over the last dimension (fp32, Sec. 3)."""
    rows, H = x.shape
    if out is None:
        out = torch.empty_like(x)
    st = load().q8_add_layernorm(_ptr(x, torch.float32, "x"), _ptr(r1, torch.float32, "r1"),
                                 _ptr(r2, torch.float32, "r2"), _ptr(gamma, torch.float32, "gamma"),
                                 _ptr(beta, torch.float32, "beta"), float(eps), rows, H,
                                 _ptr(out, torch.float32, "out"), _stream(stream))
    _check(st, "q8_add_layernorm")
    return out


def q8_attention(qkv, B: int, S: int, heads: int, ctx=None, stream=None):
    """fp32 multi-head self-attention (head dimension 64, no mask) on the fused projection [B*S, 3*heads*64]."""
    H = heads * 64
    if tuple(qkv.shape) != (B * S, 3 * H):
        raise ValueError(f"qkv must be [{B * S}, {3 * H}], got {tuple(qkv.shape)}")
    if ctx is None:
        ctx = torch.empty((B * S, H), dtype=torch.float32, device=qkv.device)
    st = load().q8_attention(_ptr(qkv, torch.float32, "qkv"), B, S, heads, _ptr(ctx, torch.float32, "ctx"),
                             _stream(stream))
    _check(st, "q8_attention")
    return ctx


def q8_add_layernorm_absmax(x, absmax_bits, r1=None, r2=None, gamma=None, beta=None, eps: float = 1e-12, out=None,
                            stream=None):
    """q8_add_layernorm that also folds max|out| into the int32 device word `absmax_bits` (fp32 bits; Sec. 4.1)."""
    rows, H = x.shape
    if out is None:
        out = torch.empty_like(x)
    st = load().q8_add_layernorm_absmax(_ptr(x, torch.float32, "x"), _ptr(r1, torch.float32, "r1"),
                                        _ptr(r2, torch.float32, "r2"), _ptr(gamma, torch.float32, "gamma"),
                                        _ptr(beta, torch.float32, "beta"), float(eps), rows, H,
                                        _ptr(out, torch.float32, "out"), _ptr(absmax_bits, torch.int32, "absmax_bits"),
                                        _stream(stream))
    _check(st, "q8_add_layernorm_absmax")
    return out


def q8_attention_absmax(qkv, B: int, S: int, heads: int, absmax_bits, ctx=None, stream=None):
    """q8_attention that also folds max|ctx| into the int32 device word `absmax_bits` (fp32 bits; Sec. 4.1)."""
    H = heads * 64
    if tuple(qkv.shape) != (B * S, 3 * H):
        raise ValueError(f"qkv must be [{B * S}, {3 * H}], got {tuple(qkv.shape)}")
    if ctx is None:
        ctx = torch.empty((B * S, H), dtype=torch.float32, device=qkv.device)
    st = load().q8_attention_absmax(_ptr(qkv, torch.float32, "qkv"), B, S, heads, _ptr(ctx, torch.float32, "ctx"),
                                    _ptr(absmax_bits, torch.int32, "absmax_bits"), _stream(stream))
    _check(st, "q8_attention_absmax")
    return ctx


def q8_linear_dyn(X, x_absmax, Wq, S_w, bias=None, act: int = Q8_ACT_NONE, Y=None, y_absmax=None, workspace=None,
                  dbg_Xq=None, dbg_acc=None, stream=None) -> torch.Tensor:
    """q8_linear with the dynamic scale 127 / max|X| taken from the device word `x_absmax` (written by the kernel
    that produced X); `y_absmax` optionally receives max|Y| for the next dynamically quantised layer."""
    M, K = X.shape
    N, K2 = Wq.shape
    if K != K2:
        raise ValueError(f"X is [M,{K}] but Wq is [N,{K2}]")
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=X.device)
    if workspace is None:
        workspace = new_workspace(M, N, K, X.device)
    st = load().q8_linear_dyn(_ptr(X, torch.float32, "X"), _ptr(x_absmax, torch.int32, "x_absmax"),
                              _ptr(Wq, torch.int8, "Wq"), _ptr(S_w, torch.float32, "S_w"),
                              _ptr(bias, torch.float32, "bias"), int(act), _ptr(Y, torch.float32, "Y"),
                              _ptr(y_absmax, torch.int32, "y_absmax"), M, N, K, _any_ptr(workspace, "workspace"),
                              workspace.numel() * workspace.element_size(), _ptr(dbg_Xq, torch.int8, "dbg_Xq"),
                              _ptr(dbg_acc, torch.int32, "dbg_acc"), _stream(stream))
    _check(st, "q8_linear_dyn")
    return Y


def q8_quantize_weight_segments(W, seg_rows: int, dev_status=None, stream=None):
    """Eq. 3 + Eq. 1 with one scale per block of `seg_rows` output rows; returns (W_q, S_w[ceil(N/seg_rows)])."""
    N, K = W.shape
    Wq = torch.empty((N, K), dtype=torch.int8, device=W.device)
    S_w = torch.empty((N + seg_rows - 1) // seg_rows, dtype=torch.float32, device=W.device)
    st = load().q8_quantize_weight_segments(_ptr(W, torch.float32, "W"), N, K, int(seg_rows), _ptr(Wq, torch.int8, "Wq"),
                                            _ptr(S_w, torch.float32, "S_w"), _ptr(dev_status, torch.int32, "dev_status"),
                                            _stream(stream))
    _check(st, "q8_quantize_weight_segments")
    return Wq, S_w


def q8_linear_wseg(X, Wq, S_w, seg_rows: int, S_x=None, bias=None, act: int = Q8_ACT_NONE, Y=None, workspace=None,
                   dbg_Xq=None, dbg_acc=None, stream=None):
    """q8_linear with one weight scale per block of `seg_rows` output features."""
    M, K = X.shape
    N = Wq.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=X.device)
    if workspace is None:
        workspace = new_workspace(M, N, K, X.device)
    st = load().q8_linear_wseg(_ptr(X, torch.float32, "X"), _ptr(Wq, torch.int8, "Wq"), _ptr(S_w, torch.float32, "S_w"),
                               int(seg_rows), _ptr(S_x, torch.float32, "S_x"), _ptr(bias, torch.float32, "bias"),
                               int(act), _ptr(Y, torch.float32, "Y"), M, N, K, _any_ptr(workspace, "workspace"),
                               workspace.numel() * workspace.element_size(), _ptr(dbg_Xq, torch.int8, "dbg_Xq"),
                               _ptr(dbg_acc, torch.int32, "dbg_acc"), _stream(stream))
    _check(st, "q8_linear_wseg")
    return Y


def q8_linear_q_wseg(Xq, S_x, Wq, S_w, seg_rows: int, bias=None, act: int = Q8_ACT_NONE, Y=None, dbg_acc=None,
                     dev_status=None, stream=None):
    M, K = Xq.shape
    N = Wq.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float32, device=Xq.device)
    st = load().q8_linear_q_wseg(_ptr(Xq, torch.int8, "Xq"), _ptr(S_x, torch.float32, "S_x"), _ptr(Wq, torch.int8, "Wq"),
                                 _ptr(S_w, torch.float32, "S_w"), int(seg_rows), _ptr(bias, torch.float32, "bias"),
                                 int(act), _ptr(Y, torch.float32, "Y"), M, N, K, _ptr(dbg_acc, torch.int32, "dbg_acc"),
                                 _ptr(dev_status, torch.int32, "dev_status"), _stream(stream))
    _check(st, "q8_linear_q_wseg")
    return Y


def q8_linear_requant(X, Wq, S_w, S_x, bias, act, S_y, Yq=None, Y=None, workspace=None, dbg_Xq=None, dbg_acc=None,
                      stream=None):
    """q8_linear whose output is (also) emitted as Int8 at the next layer's scale S_y.  Returns Yq."""
    M, K = X.shape
    N = Wq.shape[0]
    if Yq is None:
        Yq = torch.empty((M, N), dtype=torch.int8, device=X.device)
    if workspace is None:
        workspace = new_workspace(M, N, K, X.device)
    st = load().q8_linear_requant(_ptr(X, torch.float32, "X"), _ptr(Wq, torch.int8, "Wq"),
                                  _ptr(S_w, torch.float32, "S_w"), _ptr(S_x, torch.float32, "S_x"),
                                  _ptr(bias, torch.float32, "bias"), int(act), _ptr(S_y, torch.float32, "S_y"),
                                  _ptr(Yq, torch.int8, "Yq"), _ptr(Y, torch.float32, "Y"), M, N, K,
                                  _any_ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                                  _ptr(dbg_Xq, torch.int8, "dbg_Xq"), _ptr(dbg_acc, torch.int32, "dbg_acc"),
                                  _stream(stream))
    _check(st, "q8_linear_requant")
    return Yq


def q8_linear_q_requant(Xq, S_x, Wq, S_w, bias, act, S_y, Yq=None, Y=None, dbg_acc=None, dev_status=None, stream=None):
    """q8_linear_q whose output is (also) emitted as Int8 at the next layer's scale S_y.  Returns Yq."""
    M, K = Xq.shape
    N = Wq.shape[0]
    if Yq is None:
        Yq = torch.empty((M, N), dtype=torch.int8, device=Xq.device)
    st = load().q8_linear_q_requant(_ptr(Xq, torch.int8, "Xq"), _ptr(S_x, torch.float32, "S_x"),
                                    _ptr(Wq, torch.int8, "Wq"), _ptr(S_w, torch.float32, "S_w"),
                                    _ptr(bias, torch.float32, "bias"), int(act), _ptr(S_y, torch.float32, "S_y"),
                                    _ptr(Yq, torch.int8, "Yq"), _ptr(Y, torch.float32, "Y"), M, N, K,
                                    _ptr(dbg_acc, torch.int32, "dbg_acc"), _ptr(dev_status, torch.int32, "dev_status"),
                                    _stream(stream))
    _check(st, "q8_linear_q_requant")
    return Yq


def q8_add_layernorm_quant(x, r1, r2, S_q, out_q=None, out=None, gamma=None, beta=None, eps: float = 1e-12, stream=None):
    """LayerNorm(x + r1 + r2) written as fp32 (`out`, optional) and as Int8 at scale S_q (`out_q`)."""
    rows, H = x.shape
    if out_q is None:
        out_q = torch.empty((rows, H), dtype=torch.int8, device=x.device)
    st = load().q8_add_layernorm_quant(_ptr(x, torch.float32, "x"), _ptr(r1, torch.float32, "r1"),
                                       _ptr(r2, torch.float32, "r2"), _ptr(gamma, torch.float32, "gamma"),
                                       _ptr(beta, torch.float32, "beta"), float(eps), rows, H,
                                       _ptr(out, torch.float32, "out"), _ptr(S_q, torch.float32, "S_q"),
                                       _ptr(out_q, torch.int8, "out_q"), _stream(stream))
    _check(st, "q8_add_layernorm_quant")
    return out_q


def q8_attention_quant(qkv, B: int, S: int, heads: int, S_q, ctx_q=None, ctx=None, stream=None):
    """fp32 self-attention whose context is (also) emitted as Int8 at scale S_q."""
    H = heads * 64
    if ctx_q is None:
        ctx_q = torch.empty((B * S, H), dtype=torch.int8, device=qkv.device)
    st = load().q8_attention_quant(_ptr(qkv, torch.float32, "qkv"), B, S, heads, _ptr(ctx, torch.float32, "ctx"),
                                   _ptr(S_q, torch.float32, "S_q"), _ptr(ctx_q, torch.int8, "ctx_q"), _stream(stream))
    _check(st, "q8_attention_quant")
    return ctx_q


def q8_poll_status(dev_status: torch.Tensor, stream=None) -> Tuple[int, int]:
    """Synchronises, reads and clears a device status word; returns (first status code, raw bits)."""
    raw = C.c_uint32(0)
    st = load().q8_poll_status(_any_ptr(dev_status, "dev_status"), C.byref(raw), _stream(stream))
    return int(st), int(raw.value)


def q8_last_launch_info() -> dict:
    a, b, c, d, e = C.c_int(0), C.c_int(0), C.c_int(0), C.c_int(0), C.c_int(0)
    load().q8_last_launch_info(C.byref(a), C.byref(b), C.byref(c), C.byref(d), C.byref(e))
    return dict(gemm_kernel=a.value, launches=b.value, block_n=c.value, grid=d.value, ctas=e.value)


def q8_measure_int8_mma_peak(ctas: int = 2, seconds: float = 0.2, dev_status=None, stream=None) -> dict:
    """Issue-bound Int8 tensor-core rate of the current device (operands resident in shared memory)."""
    tops, ms, sms = C.c_double(0.0), C.c_double(0.0), C.c_int(0)
    st = load().q8_measure_int8_mma_peak(int(ctas), float(seconds), C.byref(tops), C.byref(ms), C.byref(sms),
                                         _ptr(dev_status, torch.int32, "dev_status"), _stream(stream))
    _check(st, "q8_measure_int8_mma_peak")
    return dict(tops=tops.value, elapsed_ms=ms.value, sms_used=sms.value, ctas=int(ctas))


def q8_measure_hbm_peak(buf: torch.Tensor, store: bool, repeats: int = 10, stream=None) -> dict:
    """Store-only (or load-only) HBM rate over the caller's device buffer `buf`, in GB/s."""
    gbs, ms = C.c_double(0.0), C.c_double(0.0)
    nbytes = buf.numel() * buf.element_size()
    st = load().q8_measure_hbm_peak(_any_ptr(buf, "buf"), nbytes, 1 if store else 0, int(repeats), C.byref(gbs),
                                    C.byref(ms), _stream(stream))
    _check(st, "q8_measure_hbm_peak")
    return {"gbs": gbs.value, "elapsed_ms": ms.value, "bytes": nbytes, "repeats": int(repeats), "store": bool(store)}


def q8_measure_l2_operand_peak(buf: torch.Tensor, rows: int, K: int, boxes_per_sm: int = 2048, sms_used: int = 0,
                               producers: int = 4, stream=None) -> dict:
    """Rate at which all SMs pull L2-resident 128 x 128-byte operand boxes of the Int8 matrix buf[rows, K] by TMA."""
    gbs, ms = C.c_double(0.0), C.c_double(0.0)
    if buf.numel() * buf.element_size() < rows * K:
        raise ValueError("buf is smaller than rows * K bytes")
    st = load().q8_measure_l2_operand_peak(_any_ptr(buf, "buf"), int(rows), int(K), int(boxes_per_sm), int(sms_used),
                                           int(producers), C.byref(gbs), C.byref(ms), _stream(stream))
    _check(st, "q8_measure_l2_operand_peak")
    return {"gbs": gbs.value, "elapsed_ms": ms.value, "rows": int(rows), "K": int(K), "boxes_per_sm": int(boxes_per_sm),
            "sms_used": int(sms_used), "producers": int(producers)}


def q8_selftest_wait_timeout(limit_ns: int, dev_status: torch.Tensor, dev_report: Optional[torch.Tensor] = None,
                             stream=None) -> None:
    """Launches the library's wait self-test: one CTA waits (bounded by limit_ns) on a barrier nobody arrives on."""
    st = load().q8_selftest_wait_timeout(int(limit_ns), _ptr(dev_status, torch.int32, "dev_status"),
                                         _ptr(dev_report, torch.int32, "dev_report"), _stream(stream))
    _check(st, "q8_selftest_wait_timeout")


def q8_tune_attention(use_tensor_cores: bool = True) -> None:
    """Chooses between the tensor-core (3 x TF32) and the CUDA-core fp32 attention kernel for later calls."""
    load().q8_tune_attention(1 if use_tensor_cores else 0)


def q8_attention_status_word() -> int:
    """Device address of the status word of the tensor-core attention kernel on the current device."""
    p = C.c_void_p(0)
    _check(load().q8_attention_status_word(C.byref(p)), "q8_attention_status_word")
    return int(p.value)


def q8_attention_status() -> Tuple[int, int]:
    """Synchronises, reads and clears the status word of the tensor-core attention kernel."""
    raw = C.c_uint32(0)
    st = load().q8_poll_status(C.c_void_p(q8_attention_status_word()), C.byref(raw), None)
    return int(st), int(raw.value)


def q8_tune_gemm_epilogue_warps(warps: int = 0) -> None:
    """Forces 8 or 16 epilogue warps in the CTA-pair GEMM kernel for later calls (0 = automatic)."""
    _check(load().q8_tune_gemm_epilogue_warps(int(warps)), "q8_tune_gemm_epilogue_warps")


def q8_tune_gemm_tail_split(enable: bool = True) -> None:
    """Switches the cutting of the last scheduling round's tiles into narrower ones on or off."""
    load().q8_tune_gemm_tail_split(1 if enable else 0)


def q8_tune_gemm_direct_store(mode: Optional[bool] = None) -> None:
    """fp32-only GEMM output stored straight from registers (True), staged and TMA-stored (False) or automatic (None)."""
    load().q8_tune_gemm_direct_store(-1 if mode is None else (1 if mode else 0))


def q8_last_launch_store_mode() -> int:
    """0 lanes stored their rows, 1 staged + TMA store, 2 stored straight from the accumulator fragments."""
    return int(load().q8_last_launch_store_mode())


def q8_last_launch_tail_split() -> int:
    """1, 2 or 4: how many narrower tiles each last-round tile of the latest tcgen05 GEMM was cut into."""
    return int(load().q8_last_launch_tail_split())


def q8_tune_gemm_tile(block_n: int = 0, ctas: int = 0) -> None:
    """Forces the tcgen05 GEMM tile shape for later calls ((0, 0) = automatic)."""
    _check(load().q8_tune_gemm_tile(int(block_n), int(ctas)), "q8_tune_gemm_tile")
