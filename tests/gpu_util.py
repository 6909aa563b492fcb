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


# Where the floor may decide: only outputs whose group dots (nearly) all vanish, i.e. whose magnitude
# reference R = sum_g |deltaA deltaW D_g| is a small fraction of F = sum_k |A~||W~|.
FLOOR_ONLY_BELOW_R_OVER_F = 0.02


def expected_paths(K: int, beta_a: int, beta_w: int):
    """Contraction paths that must take two packed operands (the support rules the header states); every
    other path must refuse them with HBMM_ERR_UNSUPPORTED.  POPC and AUTO take everything."""
    one_a, one_w = beta_a >= K, beta_w >= K
    paths = {hbmm.PATH_POPC, hbmm.PATH_AUTO}
    if (one_a or beta_a % 128 == 0) and (one_w or beta_w % 128 == 0):
        paths.add(hbmm.PATH_B1MMA)                 # legacy b1 instruction: segments of whole 128-bit chunks
    if K % 32 == 0:
        paths.add(hbmm.PATH_FOLDED)                # any supported group size, K in whole words
        if (one_a or beta_a % 32 == 0) and (one_w or beta_w % 32 == 0):
            paths.add(hbmm.PATH_TENSOR)            # groups of whole words
    return paths


def auto_runs_folded(K: int, beta_a: int, beta_w: int) -> bool:
    """HBMM_PATH_AUTO with a workspace takes the folded-scale kernel when K is whole words and the finer
    grouping has at most 128 elements (the header's rule); otherwise the e4m3 kernel or the integer pipe."""
    return K % 32 == 0 and min(eff_beta(beta_a, K), eff_beta(beta_w, K)) <= 128


def assert_close_rel_absref(c_gpu: np.ndarray, c_ref: np.ndarray, absref: np.ndarray, rtol: float, what="", fine=None):
    """|c_gpu - c_ref| <= rtol * absref (+ the oracle's own double-rounding floor).  With `fine` (F, see
    elementwise_magnitude) the bound gains FOLDED_FLOOR_ULPS * 2^-24 * F, and every output that needs that
    term must be one whose group dots nearly all cancel (R < 0.02 F).  Returns the number of such outputs."""
    err = np.abs(c_gpu.astype(np.float64) - c_ref)
    # the second term is the rounding floor of the oracle's own double-precision sum
    strict = rtol * absref + 1e-12 * max(1.0, float(absref.max()))
    bound = strict if fine is None else strict + FOLDED_FLOOR_ULPS * U * fine
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err / bound), err.shape)
        raise AssertionError("%s: %d elements outside rtol=%g of the magnitude reference; worst at %s: "
                             "gpu=%r ref=%r absref=%r" % (what, bad.sum(), rtol, i, c_gpu[i], c_ref[i], absref[i]))
    if fine is None:
        return 0
    by_floor = err > strict
    if by_floor.any():
        assert (absref[by_floor] < FLOOR_ONLY_BELOW_R_OVER_F * fine[by_floor]).all(), \
            "%s: the absolute floor decided an output whose group dots do not cancel" % what
    return int(by_floor.sum())


def random_sign_words(rows: int, K: int, ld_words: int, seed: int) -> np.ndarray:
    """Random packed sign rows [rows, ld_words] (uint32), bits past K and padding words zero."""
    rng = np.random.default_rng(seed)
    nw = (K + 31) // 32
    bits = np.zeros((rows, ld_words), dtype=np.uint32)
    bits[:, :nw] = rng.integers(0, 2 ** 32, size=(rows, nw), dtype=np.uint64).astype(np.uint32)
    if K % 32:
        bits[:, nw - 1] &= np.uint32((1 << (K % 32)) - 1)
    return bits


def signs_of_words(bits: np.ndarray, K: int) -> np.ndarray:
    """+-1 (float32) of packed rows: element k is bit k % 32 (least significant first) of word k / 32, 1 <=> +1.
    Plain numpy bit unpacking, independent of the library and of the oracle's packer."""
    b = np.unpackbits(np.ascontiguousarray(bits).view(np.uint8), axis=1, bitorder="little")[:, :K]
    return b.astype(np.float32) * 2.0 - 1.0


def check_next_operand(nxt, z_ref: np.ndarray, band: np.ndarray, bn: int, bf16_scales: bool):
    """A packed operand written by a fused epilogue against the reference rows z_ref (double): signs where |z| is
    outside the product's own error band (inside it the fp32 value the kernel computed decides), more than 99 %
    of them decided; exact zero padding; every group scale to the band's mean over the group plus the rounding
    of a pairwise fp32 tree (and of bf16 storage)."""
    import oracle
    M, N = z_ref.shape
    bits = host_bits(nxt.bits)
    lw = bits.shape[1]
    got_sign = ((bits[:, np.arange(N) // 32] >> (np.arange(N) % 32).astype(np.uint32)) & 1).astype(np.int8) * 2 - 1
    want_sign = np.where(z_ref >= 0, 1, -1)
    decided = np.abs(z_ref) > band
    assert (got_sign[decided] == want_sign[decided]).all()
    assert decided.mean() > 0.99
    assert np.array_equal(bits, oracle.pack(got_sign.astype(np.int8), lw))       # bits past N and words past ceil(N / 32) are zero
    G = -(-N // bn)
    sc = nxt.scales.float().cpu().numpy().astype(np.float64)
    assert np.all(sc[:, G:] == 0.0)
    tree = (int(np.ceil(np.log2(bn))) + 3) * U + (2.0 ** -8 if bf16_scales else 0.0)
    for g in range(G):
        sl = slice(g * bn, min((g + 1) * bn, N))
        want = np.abs(z_ref[:, sl]).mean(axis=1)
        tol = band[:, sl].mean(axis=1) + tree * want
        assert (np.abs(sc[:, g] - want) <= tol).all(), g
