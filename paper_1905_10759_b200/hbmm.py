"""Python binding of the HBMM C-ABI library (``include/hbmm.h``).

Argument marshalling only: every function here has the name of the C entry point it
calls and passes device pointers of torch tensors straight through; all arithmetic
runs in the CUDA kernels of ``libhbmm.so``.  Importing this module loads the library
and raises if it has not been built -- there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhbmm.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libhbmm.so is missing (%s); build it with `python -m paper_1905_10759_b200.build` "
        "or __graft_entry__.build()" % LIB_PATH)

_lib = ctypes.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)
F32, BF16 = 0, 1
PATH_AUTO, PATH_POPC, PATH_B1MMA, PATH_TENSOR, PATH_TENSOR_PREPARED, PATH_FOLDED, PATH_FOLDED_PREPARED = 0, 1, 2, 3, 4, 5, 6

EXPORTS = [
    "hbmm_operand_bytes", "hbmm_quantize", "hbmm_gemm_workspace_bytes", "hbmm_gemm", "hbmm_gemm_ex",
    "hbmm_gemm_partials", "hbmm_conv_workspace_bytes", "hbmm_conv_im2col", "hbmm_status_string",
    "hbmm_version", "hbmm_conv_im2col_static", "hbmm_last_device_error", "hbmm_conv_im2col_ex",
    "hbmm_binarize_backward", "hbmm_gemm_binarize_next", "hbmm_binarize_dense",
    "hbmm_clear_device_error", "hbmm_debug_set_wait_limit", "hbmm_debug_expire_wait", "hbmm_bench_alu_rate",
    "hbmm_gemm_fused", "hbmm_conv_im2col_fused",
]
STATIC_SCRATCH_BYTES = 32 << 20


class hbmm_operand(ctypes.Structure):
    _fields_ = [
        ("rows", ctypes.c_int64), ("K", ctypes.c_int64),
        ("beta", ctypes.c_int32), ("scale_dtype", ctypes.c_int32),
        ("bits", ctypes.c_void_p), ("ld_words", ctypes.c_int64),
        ("scales", ctypes.c_void_p), ("ld_scales", ctypes.c_int64),
        ("dense", ctypes.c_void_p), ("ld_dense", ctypes.c_int64),
        ("dense_dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


class hbmm_conv_geom(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "C", "H", "W", "kh", "kw", "stride_h", "stride_w", "pad_h", "pad_w")]


_i32, _i64, _vp, _sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t
_P = ctypes.POINTER
_lib.hbmm_operand_bytes.argtypes = [_i64, _i64, _i32, _i32, _P(_sz), _P(_sz), _P(_i64), _P(_i64)]
_lib.hbmm_quantize.argtypes = [_vp, _i32, _i64, _i64, _i64, _P(hbmm_operand), _vp]
_lib.hbmm_gemm_workspace_bytes.argtypes = [_P(hbmm_operand), _P(hbmm_operand), _P(_sz)]
_lib.hbmm_gemm.argtypes = [_P(hbmm_operand), _P(hbmm_operand), _vp, _i64, _vp, _sz, _vp]
_lib.hbmm_gemm_ex.argtypes = [_P(hbmm_operand), _P(hbmm_operand), _vp, _i64, _vp, _sz, _i32, _vp]
_lib.hbmm_gemm_partials.argtypes = [_P(hbmm_operand), _P(hbmm_operand), _vp, _i32, _vp]
_lib.hbmm_conv_workspace_bytes.argtypes = [_P(hbmm_conv_geom), _i32, _i32, _P(hbmm_operand), _P(_sz)]
_lib.hbmm_conv_im2col.argtypes = [_vp, _i32, _P(hbmm_conv_geom), _i32, _i32, _P(hbmm_operand), _vp, _i64,
                                  _vp, _sz, _vp]
_lib.hbmm_conv_im2col_ex.argtypes = [_vp, _i32, _P(hbmm_conv_geom), _i32, _i32, _P(hbmm_operand), _vp, _i64,
                                     _vp, _sz, ctypes.c_uint32, _vp]
_lib.hbmm_conv_im2col_ex.restype = _i32
_lib.hbmm_conv_im2col_static.argtypes = [_vp, _i32, _P(hbmm_conv_geom), _i32, _i32, _P(hbmm_operand), _vp, _i64, _vp]
_lib.hbmm_conv_im2col_static.restype = _i32
_lib.hbmm_last_device_error.argtypes = [_P(_i32)]
_lib.hbmm_last_device_error.restype = _i32
_lib.hbmm_status_string.argtypes = [_i32]
_lib.hbmm_status_string.restype = ctypes.c_char_p
_lib.hbmm_version.restype = _i32
for _n in EXPORTS[:8]:
    getattr(_lib, _n).restype = _i32


class HbmmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


def _check(status: int, where: str) -> None:
    if status != OK:
        raise HbmmError(status, where)


def status_string(status: int) -> str:
    return _lib.hbmm_status_string(status).decode()


def version() -> int:
    return int(_lib.hbmm_version())


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise TypeError("only float32 and bfloat16 tensors are accepted, got %s" % dt)


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _dev_ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensor expected")
    return t.data_ptr()


def operand_bytes(rows: int, K: int, beta: int, scale_dtype: int):
    """hbmm_operand_bytes -> (bits_bytes, scales_bytes, ld_words, ld_scales)."""
    bb, sb, lw, ls = _sz(), _sz(), _i64(), _i64()
    _check(_lib.hbmm_operand_bytes(rows, K, beta, scale_dtype, bb, sb, lw, ls), "hbmm_operand_bytes")
    return bb.value, sb.value, lw.value, ls.value


@dataclass
class Operand:
    """A descriptor plus the torch tensors that own its device buffers."""
    desc: hbmm_operand
    bits: Optional[torch.Tensor] = None     # int32 view of the uint32 words [rows, ld_words]
    scales: Optional[torch.Tensor] = None   # [rows, ld_scales] float32 / bfloat16
    dense: Optional[torch.Tensor] = None    # [rows, ld_dense] for beta == 1

    @property
    def rows(self) -> int:
        return self.desc.rows

    @property
    def K(self) -> int:
        return self.desc.K

    @property
    def beta(self) -> int:
        return self.desc.beta


def alloc_operand(rows: int, K: int, beta: int, scale_dtype: int = F32, device="cuda") -> Operand:
    """Allocate the buffers of a packed operand (sizes from hbmm_operand_bytes) and fill its descriptor."""
    _, _, lw, ls = operand_bytes(rows, K, beta, scale_dtype)
    bits = torch.empty((rows, lw), dtype=torch.int32, device=device)
    scales = torch.empty((rows, ls), dtype=torch.float32 if scale_dtype == F32 else torch.bfloat16, device=device)
    return wrap_packed(bits, scales, K, beta)


def wrap_packed(bits: torch.Tensor, scales: torch.Tensor, K: int, beta: int) -> Operand:
    """Descriptor over existing device buffers (bits int32/uint32-as-int32 [rows, ld_words])."""
    d = hbmm_operand()
    d.rows, d.K, d.beta = bits.shape[0], K, beta
    d.scale_dtype = _dtype_code(scales.dtype)
    d.bits, d.ld_words = bits.data_ptr(), bits.stride(0)
    d.scales, d.ld_scales = scales.data_ptr(), scales.stride(0)
    return Operand(d, bits=bits, scales=scales)


def wrap_dense(a: torch.Tensor) -> Operand:
    """beta = 1 operand over a row-major [rows, K] device tensor (fp32 or bf16)."""
    d = hbmm_operand()
    d.rows, d.K, d.beta = a.shape[0], a.shape[1], 1
    d.dense, d.ld_dense, d.dense_dtype = a.data_ptr(), a.stride(0), _dtype_code(a.dtype)
    return Operand(d, dense=a)


def quantize(x: torch.Tensor, out: Operand, stream=None) -> Operand:
    """hbmm_quantize: Hadamard-binarize and pack the rows of ``x`` [rows, K] into ``out``."""
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("x must be a row-major 2-D tensor")
    _check(_lib.hbmm_quantize(_dev_ptr(x), _dtype_code(x.dtype), x.shape[0], x.shape[1], x.stride(0),
                              ctypes.byref(out.desc), _stream(stream)), "hbmm_quantize")
    return out


def gemm_workspace_bytes(A: Operand, W: Operand) -> int:
    n = _sz()
    _check(_lib.hbmm_gemm_workspace_bytes(ctypes.byref(A.desc), ctypes.byref(W.desc), n), "hbmm_gemm_workspace_bytes")
    return n.value


def gemm(A: Operand, W: Operand, C: torch.Tensor, workspace: Optional[torch.Tensor] = None, stream=None):
    """hbmm_gemm: C[M, N] (fp32, row-major, caller-allocated) = A~ W~^T."""
    ws_ptr = _dev_ptr(workspace)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.hbmm_gemm(ctypes.byref(A.desc), ctypes.byref(W.desc), _dev_ptr(C), C.stride(0), ws_ptr, ws_bytes,
                          _stream(stream)), "hbmm_gemm")
    return C


def gemm_ex(A: Operand, W: Operand, C: torch.Tensor, path: int, workspace: Optional[torch.Tensor] = None,
            stream=None):
    ws_ptr = _dev_ptr(workspace)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.hbmm_gemm_ex(ctypes.byref(A.desc), ctypes.byref(W.desc), _dev_ptr(C), C.stride(0), ws_ptr, ws_bytes,
                             path, _stream(stream)), "hbmm_gemm_ex")
    return C


def gemm_partials(A: Operand, W: Operand, D: torch.Tensor, path: int = PATH_AUTO, stream=None):
    """hbmm_gemm_partials: D int32 [M, N, T] contiguous."""
    _check(_lib.hbmm_gemm_partials(ctypes.byref(A.desc), ctypes.byref(W.desc), _dev_ptr(D), path, _stream(stream)),
           "hbmm_gemm_partials")
    return D


def make_geom(B, C, H, W, kh, kw, stride=(1, 1), pad=(0, 0)) -> hbmm_conv_geom:
    return hbmm_conv_geom(B, C, H, W, kh, kw, stride[0], stride[1], pad[0], pad[1])


def conv_workspace_bytes(geom: hbmm_conv_geom, beta_a: int, a_scale_dtype: int, W: Operand) -> int:
    n = _sz()
    _check(_lib.hbmm_conv_workspace_bytes(ctypes.byref(geom), beta_a, a_scale_dtype, ctypes.byref(W.desc), n),
           "hbmm_conv_workspace_bytes")
    return n.value


CONV_WEIGHTS_PREPARED = 1
CONV_PACK_ONLY = 2
CONV_INPUT_NHWC = 4
ACT_NONE, ACT_RELU = 0, 1
OUT_DENSE, OUT_PACKED = 1, 2

_lib.hbmm_binarize_backward.argtypes = [_vp, _i64, _vp, _i64, _i64, _i64, _i32, _vp, _i64, _vp]
_lib.hbmm_binarize_backward.restype = _i32
_lib.hbmm_binarize_dense.argtypes = [_vp, _i64, _i64, _i64, _i32, _vp, _i32, _i64, _vp]
_lib.hbmm_binarize_dense.restype = _i32


_lib.hbmm_gemm_binarize_next.argtypes = [_P(hbmm_operand), _P(hbmm_operand), _vp, _vp, _P(hbmm_operand), _vp, _sz, _vp]
_lib.hbmm_gemm_binarize_next.restype = _i32


def gemm_binarize_next(A: "Operand", W: "Operand", nxt: "Operand", workspace: torch.Tensor, bn_scale: Optional[torch.Tensor] = None,
                       bn_shift: Optional[torch.Tensor] = None, stream=None) -> "Operand":
    """hbmm_gemm_binarize_next: the product's rows, after an optional per-column affine map, leave the kernel
    already binarized for the next layer (bits and scales of `nxt`); the fp32 product is never stored."""
    _check(_lib.hbmm_gemm_binarize_next(ctypes.byref(A.desc), ctypes.byref(W.desc),
                                        _dev_ptr(bn_scale) if bn_scale is not None else None,
                                        _dev_ptr(bn_shift) if bn_shift is not None else None, ctypes.byref(nxt.desc),
                                        _dev_ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "hbmm_gemm_binarize_next")
    return nxt


def binarize_backward(x: torch.Tensor, gy: torch.Tensor, beta: int, gx: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """hbmm_binarize_backward: x, gy fp32 [rows, K] (row stride >= K, unit column stride); returns gx = dC/dX."""
    if x.dtype != torch.float32 or gy.dtype != torch.float32 or x.shape != gy.shape or x.dim() != 2:
        raise ValueError("x and gy must be fp32 matrices of one shape")
    if x.stride(1) != 1 or gy.stride(1) != 1:
        raise ValueError("rows must be contiguous")
    if gx is None:
        gx = torch.empty(x.shape, dtype=torch.float32, device=x.device)
    _check(_lib.hbmm_binarize_backward(_dev_ptr(x), x.stride(0), _dev_ptr(gy), gy.stride(0), x.shape[0], x.shape[1], beta,
                                       _dev_ptr(gx), gx.stride(0), _stream(stream)), "hbmm_binarize_backward")
    return gx


def binarize_dense(x: torch.Tensor, beta: int, out_dtype: int = F32, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """hbmm_binarize_dense: x fp32 [rows, K] (row stride >= K, unit column stride); returns delta (.) Sign(x) as fp32 or bf16."""
    if x.dtype != torch.float32 or x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("x must be an fp32 matrix with contiguous rows")
    tdt = torch.bfloat16 if out_dtype == BF16 else torch.float32
    if out is None:
        out = torch.empty(x.shape, dtype=tdt, device=x.device)
    if out.dtype != tdt or out.shape != x.shape or out.stride(1) != 1:
        raise ValueError("out must match x's shape and the requested type")
    _check(_lib.hbmm_binarize_dense(_dev_ptr(x), x.stride(0), x.shape[0], x.shape[1], beta, _dev_ptr(out), out_dtype, out.stride(0),
                                    _stream(stream)), "hbmm_binarize_dense")
    return out


def binarize_map(x: torch.Tensor, beta_a: int, out_dtype: int = F32, stream=None) -> torch.Tensor:
    """Eq. 3-4 on a contiguous NCHW activation map: groups of beta_a neighbours along each map row.  Argument
    marshalling only: the map is passed to hbmm_binarize_dense as [batch*channels*height, width]."""
    if x.dim() != 4 or not x.is_contiguous():
        raise ValueError("x must be a contiguous NCHW tensor")
    B, C, H, W = x.shape
    return binarize_dense(x.view(B * C * H, W), beta_a, out_dtype, stream=stream).view(B, C, H, W)


def conv_im2col(x: torch.Tensor, geom: hbmm_conv_geom, beta_a: int, a_scale_dtype: int, W: Operand,
                C_out: torch.Tensor, workspace: torch.Tensor, stream=None, flags: int = 0):
    """hbmm_conv_im2col (flags == 0) / hbmm_conv_im2col_ex: x NCHW contiguous; C_out fp32 [B*Ho*Wo, N]."""
    if not x.is_contiguous():
        raise ValueError("x must be a contiguous NCHW tensor")
    if flags:
        _check(_lib.hbmm_conv_im2col_ex(_dev_ptr(x), _dtype_code(x.dtype), ctypes.byref(geom), beta_a, a_scale_dtype,
                                        ctypes.byref(W.desc), _dev_ptr(C_out), 0 if C_out is None else C_out.stride(0),
                                        _dev_ptr(workspace), workspace.numel() * workspace.element_size(), flags, _stream(stream)),
               "hbmm_conv_im2col_ex")
        return C_out
    _check(_lib.hbmm_conv_im2col(_dev_ptr(x), _dtype_code(x.dtype), ctypes.byref(geom), beta_a, a_scale_dtype,
                                 ctypes.byref(W.desc), _dev_ptr(C_out), C_out.stride(0), _dev_ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream)), "hbmm_conv_im2col")
    return C_out


def conv_im2col_static(x: torch.Tensor, geom: hbmm_conv_geom, beta_a: int, a_scale_dtype: int, W: Operand,
                       C_out: torch.Tensor, stream=None):
    """hbmm_conv_im2col_static: hbmm_conv_im2col without a caller workspace, for callers that cannot
    allocate device memory; the scratch is a fixed STATIC_SCRATCH_BYTES array inside the library.
    Calls that may overlap on the GPU share that array and must be serialised by the caller."""
    if not x.is_contiguous():
        raise ValueError("x must be a contiguous NCHW tensor")
    _check(_lib.hbmm_conv_im2col_static(_dev_ptr(x), _dtype_code(x.dtype), ctypes.byref(geom), beta_a, a_scale_dtype,
                                        ctypes.byref(W.desc), _dev_ptr(C_out), C_out.stride(0), _stream(stream)),
           "hbmm_conv_im2col_static")
    return C_out


def last_device_error() -> int:
    """hbmm_last_device_error: 0 when no bounded device-side wait has ever expired (synchronises)."""
    code = _i32(0)
    st = _lib.hbmm_last_device_error(ctypes.byref(code))
    if st not in (OK, ERR_TIMEOUT):
        raise HbmmError(st, "hbmm_last_device_error")
    return int(code.value)


_lib.hbmm_clear_device_error.argtypes = []
_lib.hbmm_clear_device_error.restype = _i32
_lib.hbmm_debug_set_wait_limit.argtypes = [ctypes.c_uint32]
_lib.hbmm_debug_set_wait_limit.restype = _i32
_lib.hbmm_debug_expire_wait.argtypes = [_vp]
_lib.hbmm_debug_expire_wait.restype = _i32
_lib.hbmm_bench_alu_rate.argtypes = [_i32, _i32, _i32, _vp, _P(_i64), _vp]
_lib.hbmm_bench_alu_rate.restype = _i32


def clear_device_error() -> None:
    """hbmm_clear_device_error: zero the device-side health words (synchronises)."""
    _check(_lib.hbmm_clear_device_error(), "hbmm_clear_device_error")


def debug_set_wait_limit(polls: int) -> None:
    """hbmm_debug_set_wait_limit: polls before a device-side wait gives up; 0 restores the default."""
    _check(_lib.hbmm_debug_set_wait_limit(polls), "hbmm_debug_set_wait_limit")


def debug_expire_wait(stream=None) -> None:
    """hbmm_debug_expire_wait: one thread waits on a barrier nobody arrives at until the limit runs out."""
    _check(_lib.hbmm_debug_expire_wait(_stream(stream)), "hbmm_debug_expire_wait")


ALU_POPC, ALU_FADD, ALU_FFMA = 0, 1, 2


def bench_alu_rate(kind: int, blocks: int, iters: int, sink: torch.Tensor, stream=None) -> int:
    """hbmm_bench_alu_rate: enqueue the register-only loop; returns the operations one launch performs."""
    if sink.numel() * sink.element_size() < blocks * 1024 * 4:
        raise ValueError("sink too small")
    ops = _i64(0)
    _check(_lib.hbmm_bench_alu_rate(kind, blocks, iters, _dev_ptr(sink), ctypes.byref(ops), _stream(stream)), "hbmm_bench_alu_rate")
    return int(ops.value)


class hbmm_epilogue(ctypes.Structure):
    _fields_ = [
        ("activation", ctypes.c_int32), ("out_kind", ctypes.c_int32),
        ("bn_scale", ctypes.c_void_p), ("bn_shift", ctypes.c_void_p),
        ("out", ctypes.c_void_p), ("ld_out", ctypes.c_int64),
        ("out_dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("next", ctypes.POINTER(hbmm_operand)),
    ]


_lib.hbmm_gemm_fused.argtypes = [_P(hbmm_operand), _P(hbmm_operand), _P(hbmm_epilogue), _vp, _sz, _vp]
_lib.hbmm_gemm_fused.restype = _i32
_lib.hbmm_conv_im2col_fused.argtypes = [_vp, _i32, _P(hbmm_conv_geom), _i32, _i32, _P(hbmm_operand), _P(hbmm_epilogue), _vp, _sz,
                                        ctypes.c_uint32, _vp]
_lib.hbmm_conv_im2col_fused.restype = _i32


def make_epilogue(activation: int = ACT_NONE, bn_scale: Optional[torch.Tensor] = None, bn_shift: Optional[torch.Tensor] = None,
                  out: Optional[torch.Tensor] = None, nxt: Optional[Operand] = None) -> hbmm_epilogue:
    """Fills an hbmm_epilogue: `out` (a dense [M, N] fp32 / bf16 device tensor with contiguous rows) selects
    HBMM_OUT_DENSE, `nxt` (a packed operand) HBMM_OUT_PACKED.  Marshalling only."""
    ep = hbmm_epilogue()
    ep.activation = activation
    ep.bn_scale = _dev_ptr(bn_scale) if bn_scale is not None else None
    ep.bn_shift = _dev_ptr(bn_shift) if bn_shift is not None else None
    if (out is None) == (nxt is None):
        raise ValueError("exactly one of out / nxt")
    if out is not None:
        ep.out_kind = OUT_DENSE
        ep.out, ep.ld_out, ep.out_dtype = out.data_ptr(), out.stride(0), _dtype_code(out.dtype)
    else:
        ep.out_kind = OUT_PACKED
        ep.next = ctypes.pointer(nxt.desc)
    ep._keep_alive = (bn_scale, bn_shift, out, nxt)      # the struct holds raw pointers: keep their owners alive with it
    return ep


def gemm_fused(A: Operand, W: Operand, ep: hbmm_epilogue, workspace: torch.Tensor, stream=None) -> None:
    """hbmm_gemm_fused: the product goes through activation, affine map and dense / binarized output in the epilogue."""
    _check(_lib.hbmm_gemm_fused(ctypes.byref(A.desc), ctypes.byref(W.desc), ctypes.byref(ep), _dev_ptr(workspace),
                                workspace.numel() * workspace.element_size(), _stream(stream)), "hbmm_gemm_fused")


def conv_im2col_fused(x: torch.Tensor, geom: hbmm_conv_geom, beta_a: int, a_scale_dtype: int, W: Operand, ep: hbmm_epilogue,
                      workspace: torch.Tensor, stream=None, flags: int = 0) -> None:
    """hbmm_conv_im2col_fused: x NCHW contiguous (or NHWC bf16 with CONV_INPUT_NHWC)."""
    if not x.is_contiguous():
        raise ValueError("x must be contiguous")
    _check(_lib.hbmm_conv_im2col_fused(_dev_ptr(x), _dtype_code(x.dtype), ctypes.byref(geom), beta_a, a_scale_dtype,
                                       ctypes.byref(W.desc), ctypes.byref(ep), _dev_ptr(workspace),
                                       workspace.numel() * workspace.element_size(), flags, _stream(stream)), "hbmm_conv_im2col_fused")
