"""Oracle forward pass of an ASER-quantized linear layer (test infrastructure).

Thin ctypes front for `aser_oracle.c`; every step is one C function that
restates one definition.  The composition in `forward()` follows the inference
pass of Sec. 4.2 of the paper, "W_q X + L_A L_B X" on the smoothed activation
M^-1 X, with this build's operand names (L_A = down [r,K], L_B = up [N,r]).
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_P = C.c_void_p
_L = C.c_long
_lib.aser_oracle_set_threads.argtypes = [C.c_int]
_lib.aser_oracle_get_threads.restype = C.c_int
_lib.aser_oracle_max_threads.restype = C.c_int
_lib.aser_oracle_smooth_act.argtypes = [_P, _P, _L, _L, _P]
_lib.aser_oracle_quant_act.argtypes = [_P, _L, _L, _P, _P]
_lib.aser_oracle_quant_act_bits.argtypes = [_P, _L, _L, C.c_int, _P, _P]
_lib.aser_oracle_quant_w4.argtypes = [_P, _P, _L, _L, _P, _P, _P]
_lib.aser_oracle_pack_w4.argtypes = [_P, _L, _L, _P]
_lib.aser_oracle_unpack_w4.argtypes = [_P, _L, _L, _P]
_lib.aser_oracle_int_matmul.argtypes = [_P, _P, _L, _L, _L, _P, _L, _P]
_lib.aser_oracle_down_proj.argtypes = [_P, _P, _L, _L, _L, _P, _L, _P]
_lib.aser_oracle_dequant_add.argtypes = [_P, _P, _P, _P, _P, _L, _L, _L, _P, _L, _P]


def set_threads(n: int) -> None:
    _lib.aser_oracle_set_threads(int(n))


def get_threads() -> int:
    return int(_lib.aser_oracle_get_threads())


def max_threads() -> int:
    return int(_lib.aser_oracle_max_threads())


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.dtype(dtype):
        raise TypeError(f"expected {np.dtype(dtype)}, got {a.dtype}")
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f16_bits(a: np.ndarray) -> np.ndarray:
    return _c(a, np.float16).view(np.uint16)


def smooth_act(X: np.ndarray, s: np.ndarray | None) -> np.ndarray:
    """x~ = fp32(X) / s  (Eq. 10, the M^-1 X factor).  X fp16 [M,K], s fp32 [K] or None."""
    Xb = _f16_bits(X)
    M, K = Xb.shape
    sv = None if s is None else _c(s, np.float32)
    if sv is not None and sv.shape != (K,):
        raise ValueError("s must have shape [K]")
    xs = np.empty((M, K), np.float32)
    _lib.aser_oracle_smooth_act(_ptr(Xb), _ptr(sv), M, K, _ptr(xs))
    return xs


def quant_act(xs: np.ndarray, act_bits: int = 8) -> tuple[np.ndarray, np.ndarray]:
    """Per-token codes (act_bits wide, int8 container) and fp32 scales of the smoothed activation."""
    xs = _c(xs, np.float32)
    M, K = xs.shape
    Xq = np.empty((M, K), np.int8)
    a_scale = np.empty(M, np.float32)
    if act_bits == 8:
        _lib.aser_oracle_quant_act(_ptr(xs), M, K, _ptr(Xq), _ptr(a_scale))
    else:
        if not 2 <= act_bits <= 8:
            raise ValueError("act_bits must be 2..8")
        _lib.aser_oracle_quant_act_bits(_ptr(xs), M, K, int(act_bits), _ptr(Xq), _ptr(a_scale))
    return Xq, a_scale


def quant_w4(W: np.ndarray, s: np.ndarray | None, want_ws: bool = False):
    """Per-output-channel int4 codes [N,K] (int8 container), scales [N], optional ws fp32."""
    Wb = _f16_bits(W)
    N, K = Wb.shape
    sv = None if s is None else _c(s, np.float32)
    q = np.empty((N, K), np.int8)
    w_scale = np.empty(N, np.float32)
    ws = np.empty((N, K), np.float32) if want_ws else None
    _lib.aser_oracle_quant_w4(_ptr(Wb), _ptr(sv), N, K, _ptr(q), _ptr(w_scale), _ptr(ws))
    return (q, w_scale, ws) if want_ws else (q, w_scale)


def pack_w4(q: np.ndarray) -> np.ndarray:
    q = _c(q, np.int8)
    N, K = q.shape
    if K % 2:
        raise ValueError("K must be even")
    out = np.empty((N, K // 2), np.uint8)
    _lib.aser_oracle_pack_w4(_ptr(q), N, K, _ptr(out))
    return out


def unpack_w4(packed: np.ndarray) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N, K2 = packed.shape
    q = np.empty((N, 2 * K2), np.int8)
    _lib.aser_oracle_unpack_w4(_ptr(packed), N, 2 * K2, _ptr(q))
    return q


def _rows(rows, M):
    if rows is None:
        return None, 0
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    if r.ndim != 1 or (r.size and (r.min() < 0 or r.max() >= M)):
        raise ValueError("bad row subset")
    return r, r.size


def int_matmul(Xq: np.ndarray, q: np.ndarray, rows=None) -> np.ndarray:
    """acc = Xq q^T, exact int32, plain triple loop."""
    Xq = _c(Xq, np.int8)
    q = _c(q, np.int8)
    M, K = Xq.shape
    N, K2 = q.shape
    if K != K2:
        raise ValueError("K mismatch")
    rr, nr = _rows(rows, M)
    acc = np.empty((nr if rr is not None else M, N), np.int32)
    _lib.aser_oracle_int_matmul(_ptr(Xq), _ptr(q), M, N, K, _ptr(rr), nr, _ptr(acc))
    return acc


def int_matmul_dgemm(Xq: np.ndarray, q: np.ndarray, rows=None) -> np.ndarray:
    """The same integer product through a library fp64 matmul.

    Every product |x q| <= 127*8 and every partial sum stays far below 2^53, so
    the fp64 result is the exact integer.  Used only where the triple loop would
    take minutes; pinned against the triple loop in the tests.
    """
    Xs = Xq if rows is None else Xq[np.asarray(rows)]
    acc = Xs.astype(np.float64) @ q.astype(np.float64).T
    out = np.rint(acc)
    assert np.array_equal(out, acc)
    return out.astype(np.int32)


def down_proj(xs: np.ndarray, L_A: np.ndarray, rows=None) -> np.ndarray:
    """T = x~ L_A^T in fp64, [rows, r]."""
    xs = _c(xs, np.float32)
    M, K = xs.shape
    LAb = _f16_bits(L_A)
    r, K2 = LAb.shape
    if K != K2:
        raise ValueError("K mismatch")
    rr, nr = _rows(rows, M)
    T = np.empty((nr if rr is not None else M, r), np.float64)
    _lib.aser_oracle_down_proj(_ptr(xs), _ptr(LAb), M, K, r, _ptr(rr), nr, _ptr(T))
    return T


def dequant_add(acc, a_scale, w_scale, T, L_B, rows=None) -> np.ndarray:
    """y = acc * a_scale[m] * w_scale[n] + T L_B^T in fp64."""
    acc = _c(acc, np.int32)
    a_scale = _c(a_scale, np.float32)
    w_scale = _c(w_scale, np.float32)
    R, N = acc.shape
    M = a_scale.shape[0]
    if L_B is None or T is None or T.shape[1] == 0:
        r, LBb, Tc = 0, None, None
    else:
        LBb = _f16_bits(L_B)
        Tc = _c(T, np.float64)
        r = LBb.shape[1]
        if LBb.shape[0] != N or Tc.shape != (R, r):
            raise ValueError("factor shape mismatch")
    rr, nr = _rows(rows, M)
    y = np.empty((R, N), np.float64)
    _lib.aser_oracle_dequant_add(_ptr(acc), _ptr(a_scale), _ptr(w_scale), _ptr(Tc), _ptr(LBb),
                                 M, N, r, _ptr(rr), nr, _ptr(y))
    return y


@dataclass
class ForwardResult:
    xs: np.ndarray        # [M,K] fp32 smoothed activation
    Xq: np.ndarray        # [M,K] int8 codes
    a_scale: np.ndarray   # [M] fp32
    acc: np.ndarray       # [R,N] int32
    T: np.ndarray | None  # [R,r] fp64
    y: np.ndarray         # [R,N] fp64
    rows: np.ndarray | None


def forward(X, s, Wq_packed, w_scale, L_A=None, L_B=None, rows=None,
            use_dgemm: bool = False, act_bits: int = 8) -> ForwardResult:
    """Inference pass of one ASER linear (Sec. 4.2): smooth, quantize per token,
    integer product with the int4 weights, dequantize, add L_B (L_A x~).

    `rows` restricts the expensive products to a subset of tokens (quantization
    still covers every token).  `use_dgemm` swaps the triple loop for the exact
    fp64 library product on large shapes.  `act_bits` = 6 is the W4A6 setting.
    """
    xs = smooth_act(X, s)
    Xq, a_scale = quant_act(xs, act_bits)
    q = unpack_w4(Wq_packed)
    acc = (int_matmul_dgemm if use_dgemm else int_matmul)(Xq, q, rows)
    T = None
    if L_A is not None and L_A.shape[0] > 0:
        T = down_proj(xs, L_A, rows)
    y = dequant_add(acc, a_scale, w_scale, T, L_B, rows)
    return ForwardResult(xs=xs, Xq=Xq, a_scale=a_scale, acc=acc, T=T, y=y,
                         rows=None if rows is None else np.asarray(rows))
