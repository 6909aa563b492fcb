"""Helpers shared by the GPU parity tests: moving oracle-built operands to the device and the tolerances."""
import numpy as np
import torch

import oracle
from paper_1905_10759_b200 import hbmm

U = 2.0 ** -24  # unit roundoff of fp32


def dev_bits(bits_np: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits_np.view(np.int32).copy()).cuda()


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def scales_to_dev(delta_rounded: np.ndarray, scale_dtype: int, ld: int) -> torch.Tensor:
    """delta_rounded already holds values representable in the storage type."""
    rows, G = delta_rounded.shape
    buf = np.zeros((rows, ld), dtype=np.float32)
    buf[:, :G] = delta_rounded.astype(np.float32)
    t = torch.from_numpy(buf).cuda()
    return t if scale_dtype == hbmm.F32 else t.to(torch.bfloat16)


def oracle_operand(x: np.ndarray, beta: int, scale_dtype: int = hbmm.F32):
    """Quantize+pack on the CPU oracle and upload: returns (Operand, delta_rounded, sign)."""
    rows, K = x.shape
    delta, sign = oracle.quantize(x, beta)
    dr = oracle.round_scales(delta, "f32" if scale_dtype == hbmm.F32 else "bf16")
    _, _, lw, ls = hbmm.operand_bytes(rows, K, beta, scale_dtype)
    bits = oracle.pack(sign, lw)
    op = hbmm.wrap_packed(dev_bits(bits), scales_to_dev(dr, scale_dtype, ls), K, beta)
    return op, dr, sign


def eff_beta(beta: int, K: int) -> int:
    return K if beta >= K else beta


def elementwise_magnitude(da: np.ndarray, beta_a: int, dw: np.ndarray, beta_w: int, K: int) -> np.ndarray:
    """F[m,n] = sum_k |A~[m,k]| |W~[n,k]| = sum_k deltaA[m, k/beta_a] deltaW[n, k/beta_w]: the magnitude of the
    K individual products.  A kernel that accumulates those products in fp32 (instead of cancelling the
    +-1 terms of a group in integers first) cannot be closer than a few 2^-24 F where the group dots vanish."""
    ea = np.repeat(np.asarray(da, dtype=np.float64), beta_a, axis=1)[:, :K]
    ew = np.repeat(np.asarray(dw, dtype=np.float64), beta_w, axis=1)[:, :K]
    return ea @ ew.T


# Absolute floor of the folded-scale kernel's bound, in units of 2^-24 F (see elementwise_magnitude).
FOLDED_FLOOR_ULPS = 4.0


def assert_close_rel_absref(c_gpu: np.ndarray, c_ref: np.ndarray, absref: np.ndarray, rtol: float, what="", floor=None):
    err = np.abs(c_gpu.astype(np.float64) - c_ref)
    # the second term is the rounding floor of the oracle's own double-precision sum
    bound = rtol * absref + 1e-12 * max(1.0, float(absref.max()))
    if floor is not None:
        bound = bound + floor
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err / bound), err.shape)
        raise AssertionError("%s: %d elements outside rtol=%g of the magnitude reference; worst at %s: "
                             "gpu=%r ref=%r absref=%r" % (what, bad.sum(), rtol, i, c_gpu[i], c_ref[i], absref[i]))
    return float((err / bound).max()) * rtol
