"""CPU oracle for the Hadamard Binary Matrix Multiply -- TEST INFRASTRUCTURE ONLY.

A plain double-precision restatement of what the HadaNets inference path
computes (Section 3, Eq. 1-4; Section 4.2, Eq. 7), kept apart from the CUDA
library: nothing here imports, links or shares code with it, and the product
path never imports this package.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg call it.

The arithmetic lives in ``hbmm_oracle.c`` (plain C loops, double accumulation,
k ascending); this module builds it with gcc and wraps it with ctypes/numpy.
Every function is pinned by the CPU-only tests to facts fixed by the paper or by
mathematics (closed forms, exact rational brute force, the printed bit-packing
example, the storage ratio, the beta = 1 and beta = K special cases).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hbmm_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, -O2, OpenMP over rows only; no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_num_segments.restype = _i64
        _lib.oracle_num_segments.argtypes = [_i64, _i64, _i64]
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_p)


def num_threads() -> int:
    return int(_L().oracle_num_threads())


def n_groups(K: int, beta: int) -> int:
    return (K + beta - 1) // beta


def ld_words_for(K: int) -> int:
    """Words per packed row: ceil(K/32) rounded up to a multiple of 4 (16-byte rows)."""
    return ((K + 31) // 32 + 3) // 4 * 4


def quantize(x: np.ndarray, beta: int) -> Tuple[np.ndarray, np.ndarray]:
    """Hadamard binarization of the rows of ``x`` (Eq. 1-4).

    Returns ``(delta, sign)``: ``delta`` float64 [rows, ceil(K/beta)] = mean |x| of each
    run of ``beta`` consecutive row elements (tail group: over its own length), ``sign``
    int8 [rows, K] in {-1,+1} with Sign(0) = +1.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, K = x.shape
    G = n_groups(K, beta)
    delta = np.empty((rows, G), dtype=np.float64)
    sign = np.empty((rows, K), dtype=np.int8)
    _L().oracle_quantize(_ptr(x), _i64(rows), _i64(K), _i64(K), _i64(beta), _ptr(delta), _ptr(sign))
    return delta, sign


def binarize_backward(x: np.ndarray, gy: np.ndarray, beta: int) -> np.ndarray:
    """dC/dX from dC/dX~ for X~ = delta (.) Sign(X) (Eq. 6 with the straight-through estimator of Eq. 5):
    float64 [rows, K]."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    gy = np.ascontiguousarray(gy, dtype=np.float32)
    assert x.shape == gy.shape
    rows, K = x.shape
    gx = np.empty((rows, K), dtype=np.float64)
    _L().oracle_binarize_backward(_ptr(x), _ptr(gy), _i64(rows), _i64(K), _i64(K), _i64(K), _i64(beta), _ptr(gx))
    return gx


def round_scales(delta: np.ndarray, scale_dtype: Optional[str]) -> np.ndarray:
    """Value of the scale tensor after storage: None = exact, 'f32', or 'bf16' (RNE of the fp32 value)."""
    out = np.array(delta, dtype=np.float64, order="C", copy=True)
    if scale_dtype is None:
        return out
    if scale_dtype == "f32":
        _L().oracle_round_f32(_ptr(out), _i64(out.size))
    elif scale_dtype == "bf16":
        _L().oracle_round_bf16(_ptr(out), _i64(out.size))
    else:
        raise ValueError(scale_dtype)
    return out


def pack(sign: np.ndarray, ld_words: Optional[int] = None) -> np.ndarray:
    """Bit-pack a +-1 tensor along its rows: +1 -> 1, -1 -> 0, LSB first in uint32 words."""
    sign = np.ascontiguousarray(sign, dtype=np.int8)
    rows, K = sign.shape
    if ld_words is None:
        ld_words = ld_words_for(K)
    bits = np.empty((rows, ld_words), dtype=np.uint32)
    _L().oracle_pack(_ptr(sign), _i64(rows), _i64(K), _i64(ld_words), _ptr(bits))
    return bits


def unpack(bits: np.ndarray, K: int) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint32)
    rows, ldw = bits.shape
    sign = np.empty((rows, K), dtype=np.int8)
    _L().oracle_unpack(_ptr(bits), _i64(rows), _i64(K), _i64(ldw), _ptr(sign))
    return sign


def dequant(delta: np.ndarray, sign: np.ndarray, beta: int) -> np.ndarray:
    """X~ = delta (.) Sign(X) as a dense float64 matrix (Eq. 2 / Eq. 4)."""
    delta = np.ascontiguousarray(delta, dtype=np.float64)
    sign = np.ascontiguousarray(sign, dtype=np.int8)
    rows, K = sign.shape
    assert delta.shape == (rows, n_groups(K, beta))
    xt = np.empty((rows, K), dtype=np.float64)
    _L().oracle_dequant(_ptr(delta), _ptr(sign), _i64(rows), _i64(K), _i64(beta), _ptr(xt))
    return xt


def widen(x: np.ndarray) -> np.ndarray:
    """beta = 1: the tensor stays at full precision (X~ = X)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    rows, K = x.shape
    xt = np.empty((rows, K), dtype=np.float64)
    _L().oracle_widen(_ptr(x), _i64(rows), _i64(K), _i64(K), _ptr(xt))
    return xt


def matmul_nt(at: np.ndarray, wt: np.ndarray) -> np.ndarray:
    """C[m,n] = sum_k at[m,k] * wt[n,k] in double, k ascending (plain triple loop)."""
    at = np.ascontiguousarray(at, dtype=np.float64)
    wt = np.ascontiguousarray(wt, dtype=np.float64)
    M, K = at.shape
    N, K2 = wt.shape
    assert K == K2
    c = np.empty((M, N), dtype=np.float64)
    _L().oracle_matmul_nt(_ptr(at), _ptr(wt), _i64(M), _i64(N), _i64(K), _ptr(c))
    return c


def num_segments(K: int, beta_a: int, beta_w: int) -> int:
    return int(_L().oracle_num_segments(K, beta_a, beta_w))


def partials(sign_a, sign_w, beta_a: int, beta_w: int, delta_a=None, delta_w=None,
             want_d: bool = True):
    """Signed +-1 dot product of every K-segment (Eq. 7's integer term), by multiply-add.

    Returns ``(D, absref)``: ``D`` int32 [M, N, T] (None if ``want_d`` is False) and, when
    both scale tensors are given, ``absref[m,n] = sum_t |deltaA * deltaW * D_t|`` (else None).
    """
    sa = np.ascontiguousarray(sign_a, dtype=np.int8)
    sw = np.ascontiguousarray(sign_w, dtype=np.int8)
    M, K = sa.shape
    N, K2 = sw.shape
    assert K == K2
    T = num_segments(K, beta_a, beta_w)
    d = np.empty((M, N, T), dtype=np.int32) if want_d else None
    absref = None
    da = dw = None
    if delta_a is not None and delta_w is not None:
        da = np.ascontiguousarray(delta_a, dtype=np.float64)
        dw = np.ascontiguousarray(delta_w, dtype=np.float64)
        assert da.shape == (M, n_groups(K, beta_a)) and dw.shape == (N, n_groups(K, beta_w))
        absref = np.empty((M, N), dtype=np.float64)
    _L().oracle_partials(_ptr(sa), _ptr(sw), _i64(M), _i64(N), _i64(K), _i64(beta_a), _i64(beta_w),
                         _ptr(da), _ptr(dw), _ptr(d), _ptr(absref))
    return d, absref


def hbmm_from_quantized(delta_a, sign_a, beta_a: int, delta_w, sign_w, beta_w: int):
    """Product of two Hadamard-binary operands given as (scales, signs): dense double matmul
    of the unpacked, scaled operands, plus the tolerance reference ``absref``."""
    at = dequant(delta_a, sign_a, beta_a)
    wt = dequant(delta_w, sign_w, beta_w)
    c = matmul_nt(at, wt)
    _, absref = partials(sign_a, sign_w, beta_a, beta_w, delta_a, delta_w, want_d=False)
    return c, absref


def hbmm(a: np.ndarray, w: np.ndarray, beta_a: int, beta_w: int, scale_dtype: Optional[str] = None):
    """HBMM from raw inputs: binarize both operands (Eq. 1-4), optionally round the scales to
    their storage type, and multiply the dense Hadamard-product operands in double.
    Returns ``(C, absref)``."""
    da, sa = quantize(a, beta_a)
    dw, sw = quantize(w, beta_w)
    da = round_scales(da, scale_dtype)
    dw = round_scales(dw, scale_dtype)
    return hbmm_from_quantized(da, sa, beta_a, dw, sw, beta_w)


def hbwn(a: np.ndarray, w: np.ndarray, beta_w: int, scale_dtype: Optional[str] = None):
    """HBWN (beta_a = 1): full-precision activations times Hadamard-binary weights.
    ``absref[m,n] = sum_k |a[m,k]| * deltaW[n, k/beta_w]`` bounds the magnitude of the summands."""
    dw, sw = quantize(w, beta_w)
    dw = round_scales(dw, scale_dtype)
    return hbwn_from_quantized(a, dw, sw, beta_w)


def hbwn_from_quantized(a: np.ndarray, delta_w, sign_w, beta_w: int):
    at = widen(a)
    wt = dequant(delta_w, sign_w, beta_w)
    c = matmul_nt(at, wt)
    absref = matmul_nt(np.abs(at), np.abs(wt))
    return c, absref


def im2col(x: np.ndarray, kh: int, kw: int, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Rows m = (b, yo, xo), columns k = (c, i, j), c slowest; zero outside the image."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    B, C, H, W = x.shape
    Ho = (H + 2 * pad[0] - kh) // stride[0] + 1
    Wo = (W + 2 * pad[1] - kw) // stride[1] + 1
    out = np.empty((B * Ho * Wo, C * kh * kw), dtype=np.float32)
    _L().oracle_im2col(_ptr(x), _i64(B), _i64(C), _i64(H), _i64(W), _i64(kh), _i64(kw),
                       _i64(stride[0]), _i64(stride[1]), _i64(pad[0]), _i64(pad[1]), _ptr(out))
    return out


def conv_im2col(x, w2d, kh, kw, stride, pad, beta_a: int, beta_w: int,
                scale_dtype: Optional[str] = None):
    """Convolution as HBMM: explicit im2col, then ``hbmm`` (or ``hbwn`` when beta_a = 1) against
    the weight matrix ``w2d`` = Reshape(W, (filters, -1)).  Output [B*Ho*Wo, filters]."""
    a = im2col(x, kh, kw, stride, pad)
    if beta_a == 1:
        return hbwn(a, w2d, beta_w, scale_dtype)
    return hbmm(a, w2d, beta_a, beta_w, scale_dtype)


def binarize_map(x: np.ndarray, beta_a: int) -> np.ndarray:
    """Eq. 3-4 as printed: an NCHW activation map binarized in runs of ``beta_a`` neighbours along each row of the
    map (the width axis; the paper asks beta_a <= width, a larger value is taken as the width; a tail run has its
    own length).  Returns A~ = delta (.) Sign(A) as float64 NCHW."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    B, C, H, W = x.shape
    b = min(int(beta_a), W)
    if b == 1:
        return widen(x.reshape(B * C * H, W)).reshape(B, C, H, W)
    delta, sign = quantize(x.reshape(B * C * H, W), b)
    return dequant(delta, sign, b).reshape(B, C, H, W)


def im2col_f64(xt: np.ndarray, kh: int, kw: int, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """The gather of ``im2col`` on a float64 map: rows m = (b, yo, xo), columns k = (c, i, j), c slowest; zero outside
    the image."""
    xt = np.asarray(xt, dtype=np.float64)
    B, C, H, W = xt.shape
    Ho = (H + 2 * pad[0] - kh) // stride[0] + 1
    Wo = (W + 2 * pad[1] - kw) // stride[1] + 1
    xp = np.zeros((B, C, H + 2 * pad[0], W + 2 * pad[1]), dtype=np.float64)
    xp[:, :, pad[0]:pad[0] + H, pad[1]:pad[1] + W] = xt
    cols = np.empty((B, Ho, Wo, C, kh, kw), dtype=np.float64)
    for i in range(kh):
        for j in range(kw):
            win = xp[:, :, i:i + stride[0] * (Ho - 1) + 1:stride[0], j:j + stride[1] * (Wo - 1) + 1:stride[1]]
            cols[:, :, :, :, i, j] = win.transpose(0, 2, 3, 1)
    return cols.reshape(B * Ho * Wo, C * kh * kw)


def conv_map_binarized(x: np.ndarray, w2d: np.ndarray, kh: int, kw: int, stride, pad, beta_a: int, beta_w: int):
    """Convolution of Eq. 3's A~ (``binarize_map``) with W~ (Eq. 1-2 on Reshape(W, (filters, -1))): the activation
    is binarized on the map, before the gather, so an im2col row mixes scales of several map groups.  Returns
    ``(C, absref)`` like ``hbmm``: float64 [B*Ho*Wo, filters] and the same sum over absolute values."""
    at = im2col_f64(binarize_map(x, beta_a), kh, kw, stride, pad)
    w2d = np.ascontiguousarray(w2d, dtype=np.float32)
    bw = min(int(beta_w), w2d.shape[1])
    dw, sw = quantize(w2d, bw)
    wt = dequant(dw, sw, bw)
    return matmul_nt(at, wt), matmul_nt(np.abs(at), np.abs(wt))
