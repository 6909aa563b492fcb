"""CPU-only pins of the oracle against facts fixed by the paper or by mathematics.

None of these tests compares the oracle with itself: expected values come from exact
rational arithmetic in pure Python, closed forms, numpy/torch library routines on the
special cases that reduce to them, Python's own bit counting, or values the paper prints.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if ":" in line:
                k, v = line.split(":", 1)
                out[k.strip()] = v.strip()
    return out


# ---------------------------------------------------------------- exact rational brute force
def _frac_quantize(row, beta):
    """Eq. 1-4 in exact rationals: list of (delta per element, sign per element)."""
    K = len(row)
    deltas, signs = [], []
    for k in range(K):
        g0 = (k // beta) * beta
        seg = row[g0:min(g0 + beta, K)]
        deltas.append(sum(abs(Fraction(float(v))) for v in seg) / len(seg))
        signs.append(1 if row[k] >= 0 else -1)
    return deltas, signs


def _frac_hbmm(a, w, beta_a, beta_w):
    M, N = len(a), len(w)
    c = [[Fraction(0)] * N for _ in range(M)]
    qa = [_frac_quantize(r, beta_a) for r in a]
    qw = [_frac_quantize(r, beta_w) for r in w]
    for m in range(M):
        for n in range(N):
            c[m][n] = sum(qa[m][0][k] * qa[m][1][k] * qw[n][0][k] * qw[n][1][k] for k in range(len(a[m])))
    return c


@pytest.mark.parametrize("M,N,K,ba,bw", [(3, 2, 8, 2, 2), (2, 3, 7, 2, 4), (4, 1, 5, 5, 1), (1, 4, 6, 3, 2),
                                         (3, 5, 8, 8, 4), (2, 2, 1, 2, 2)])
def test_brute_force_exact_rationals(M, N, K, ba, bw):
    rng = np.random.default_rng(100 + M * 31 + N * 7 + K)
    # quarter-integers: every mean is an exact double, so the oracle must match to the last bit
    a = (rng.integers(-8, 9, size=(M, K)) / 4.0).astype(np.float32)
    w = (rng.integers(-8, 9, size=(N, K)) / 4.0).astype(np.float32)
    c, _ = oracle.hbmm(a, w, ba, bw)
    ref = _frac_hbmm(a.tolist(), w.tolist(), ba, bw)
    for m in range(M):
        for n in range(N):
            assert abs(Fraction(float(c[m, n])) - ref[m][n]) <= abs(ref[m][n]) * Fraction(1, 2 ** 48), (m, n)


def test_all_sign_patterns_k4():
    """Every sign pattern of two length-4 vectors with unit magnitudes and beta = 2:
    the product is the sum over the two groups of (signed dot of the group) since delta = 1."""
    vals = []
    for pa in range(16):
        vals.append([1.0 if (pa >> i) & 1 else -1.0 for i in range(4)])
    a = np.array(vals, dtype=np.float32)
    c, _ = oracle.hbmm(a, a, 2, 2)
    for i in range(16):
        for j in range(16):
            agree = sum(1 for k in range(4) if vals[i][k] == vals[j][k])
            assert c[i, j] == 2 * agree - 4


def test_hand_worked_example_beta2():
    """beta_a = beta_w = 2 on two length-6 vectors, worked by hand from Eq. 2, 4 and 7:
    A = [1,-3, 2,2, -.5,.5]  -> delta_A = [2, 2, .5], signs + - | + + | - +
    W = [-2,-2, 1,3, 4,-4]   -> delta_W = [2, 2, 4],  signs - - | + + | + -
    signed group dots: (+1)(-1)+(-1)(-1) = 0 ; 1+1 = 2 ; (-1)(+1)+(+1)(-1) = -2
    O = 2*2*0 + 2*2*2 + .5*4*(-2) = 4."""
    a = np.array([[1, -3, 2, 2, -0.5, 0.5]], dtype=np.float32)
    w = np.array([[-2, -2, 1, 3, 4, -4]], dtype=np.float32)
    da, sa = oracle.quantize(a, 2)
    dw, sw = oracle.quantize(w, 2)
    assert da.tolist() == [[2.0, 2.0, 0.5]] and dw.tolist() == [[2.0, 2.0, 4.0]]
    assert sa.tolist() == [[1, -1, 1, 1, -1, 1]] and sw.tolist() == [[-1, -1, 1, 1, 1, -1]]
    d, absref = oracle.partials(sa, sw, 2, 2, da, dw)
    assert d.tolist() == [[[0, 2, -2]]]
    c, _ = oracle.hbmm(a, w, 2, 2)
    assert c[0, 0] == 4.0
    assert absref[0, 0] == 12.0  # |0| + |8| + |-4|


# ---------------------------------------------------------------- dense-matmul identity (library routine)
def _np_hadamard(x, beta):
    rows, K = x.shape
    G = -(-K // beta)
    xp = np.zeros((rows, G * beta))
    xp[:, :K] = np.abs(x.astype(np.float64))
    cnt = np.minimum(beta, K - np.arange(G) * beta)
    delta = xp.reshape(rows, G, beta).sum(-1) / cnt
    return np.repeat(delta, beta, axis=1)[:, :K] * np.where(x >= 0, 1.0, -1.0)


@pytest.mark.parametrize("M,N,K,ba,bw", [(37, 11, 100, 32, 64), (5, 64, 576, 32, 32), (16, 9, 333, 128, 32),
                                         (8, 8, 64, 64, 64), (3, 7, 50, 7, 5)])
def test_equals_dense_matmul_of_hadamard_operands(M, N, K, ba, bw):
    rng = np.random.default_rng(7 * M + N + K)
    a = rng.standard_normal((M, K)).astype(np.float32)
    w = rng.standard_normal((N, K)).astype(np.float32)
    c, absref = oracle.hbmm(a, w, ba, bw)
    ref = _np_hadamard(a, ba) @ _np_hadamard(w, bw).T
    assert c.shape == (M, N)
    np.testing.assert_allclose(c, ref, rtol=0, atol=1e-12 * K)
    assert np.all(absref >= np.abs(c) - 1e-9)


# ---------------------------------------------------------------- popcount identity, packing
def _popc(x):
    return bin(int(x)).count("1")


@pytest.mark.parametrize("K,ba,bw", [(64, 32, 32), (100, 32, 64), (45, 32, 32), (256, 128, 64), (96, 96, 32)])
def test_popcount_identity_on_packed_words(K, ba, bw):
    """dot(+-1) over a segment == n_valid - 2*popc(xor of the packed words restricted to it)."""
    rng = np.random.default_rng(K)
    a = rng.standard_normal((6, K)).astype(np.float32)
    w = rng.standard_normal((5, K)).astype(np.float32)
    _, sa = oracle.quantize(a, ba)
    _, sw = oracle.quantize(w, bw)
    d, _ = oracle.partials(sa, sw, ba, bw)
    ba_bits, bw_bits = oracle.pack(sa), oracle.pack(sw)
    seg = min(ba, bw)
    assert max(ba, bw) % seg == 0
    T = -(-K // seg)
    assert d.shape == (6, 5, T)
    for m in range(6):
        for n in range(5):
            for t in range(T):
                k0, k1 = t * seg, min((t + 1) * seg, K)
                ham = 0
                for k in range(k0, k1):
                    xa = (int(ba_bits[m, k // 32]) >> (k % 32)) & 1
                    xw = (int(bw_bits[n, k // 32]) >> (k % 32)) & 1
                    ham += xa ^ xw
                assert d[m, n, t] == (k1 - k0) - 2 * ham
            # whole-word form: pad bits are zero in both operands, so they never count
            tot = sum(_popc(int(ba_bits[m, j]) ^ int(bw_bits[n, j])) for j in range(ba_bits.shape[1]))
            assert d[m, n].sum() == K - 2 * tot


def test_packing_polarity_matches_paper_example():
    g = _golden("packing_example.txt")
    vec = [int(t) for t in g["vector"].split()]
    bits = oracle.pack(np.array([vec], dtype=np.int8))
    got = "".join(str((int(bits[0, 0]) >> k) & 1) for k in range(len(vec)))
    assert got == g["bits"]
    assert int(bits[0, 0]) >> len(vec) == 0 and not bits[0, 1:].any()
    assert oracle.unpack(bits, len(vec)).tolist() == [vec]
    assert bits.shape[1] % 4 == 0


def test_pack_unpack_roundtrip_ragged():
    rng = np.random.default_rng(5)
    s = rng.choice(np.array([-1, 1], dtype=np.int8), size=(9, 131))
    b = oracle.pack(s)
    assert b.shape == (9, 8)
    assert np.array_equal(oracle.unpack(b, 131), s)
    # bit k of the row lives in word k//32 at position k%32
    assert ((int(b[3, 4]) >> 2) & 1) == (1 if s[3, 130] > 0 else 0)


# ---------------------------------------------------------------- special cases named by the paper
def test_unit_scales_reduce_to_xnor_popcount():
    """With every scale equal to 1 the product is the plain binary (XNOR-net style) dot K - 2*hamming."""
    rng = np.random.default_rng(11)
    K = 200
    sa = rng.choice(np.array([-1, 1], dtype=np.int8), size=(7, K))
    sw = rng.choice(np.array([-1, 1], dtype=np.int8), size=(4, K))
    ones_a = np.ones((7, oracle.n_groups(K, 32)))
    ones_w = np.ones((4, oracle.n_groups(K, 64)))
    c, absref = oracle.hbmm_from_quantized(ones_a, sa, 32, ones_w, sw, 64)
    ham = (sa[:, None, :] != sw[None, :, :]).sum(-1)
    assert np.array_equal(c, (K - 2 * ham).astype(np.float64))
    assert np.all(absref >= np.abs(c))


def test_beta_equals_k_is_xnor_net():
    """beta = nElement(row): one scalar per row, C = alpha_A[m] * alpha_W[n] * (K - 2*hamming)  (Section 5)."""
    rng = np.random.default_rng(12)
    K = 77
    a = rng.standard_normal((5, K)).astype(np.float32)
    w = rng.standard_normal((6, K)).astype(np.float32)
    c, _ = oracle.hbmm(a, w, K, K)
    alpha_a = np.abs(a.astype(np.float64)).mean(1)
    alpha_w = np.abs(w.astype(np.float64)).mean(1)
    ham = ((a >= 0)[:, None, :] != (w >= 0)[None, :, :]).sum(-1)
    np.testing.assert_allclose(c, alpha_a[:, None] * alpha_w[None, :] * (K - 2 * ham), rtol=1e-13)


def test_beta_one_is_full_precision():
    """beta = 1 (first/last layers in the paper) leaves the tensor unchanged: X~ = X."""
    rng = np.random.default_rng(13)
    x = rng.standard_normal((4, 19)).astype(np.float32)
    x[0, 0] = 0.0
    x[1, 1] = -0.0
    d, s = oracle.quantize(x, 1)
    assert np.array_equal(oracle.dequant(d, s, 1), x.astype(np.float64))
    assert s[0, 0] == 1 and s[1, 1] == 1  # Sign(0) = Sign(-0) = +1
    # and HBWN equals the dense product of A with W~
    w = rng.standard_normal((3, 19)).astype(np.float32)
    c, absref = oracle.hbwn(x, w, 4)
    np.testing.assert_allclose(c, x.astype(np.float64) @ _np_hadamard(w, 4).T, rtol=0, atol=1e-13)
    np.testing.assert_allclose(absref, np.abs(x.astype(np.float64)) @ np.abs(_np_hadamard(w, 4)).T, atol=1e-13)
    c2, _ = oracle.hbmm(x, w, 1, 4)
    np.testing.assert_allclose(c2, c, rtol=0, atol=1e-13)


def test_delta_is_l2_optimal_scale_of_each_segment():
    """(1/n)||W||_1 Sign(W) is the optimal binary estimate of a segment (Section 3.1.2):
    moving any one scale away from delta raises ||x - a*sign(x)||_2."""
    rng = np.random.default_rng(14)
    x = rng.standard_normal((3, 70)).astype(np.float32)
    beta = 32
    d, s = oracle.quantize(x, beta)
    base = np.sum((x - oracle.dequant(d, s, beta)) ** 2)
    for g in range(d.shape[1]):
        for eps in (-1e-3, 1e-3):
            d2 = d.copy()
            d2[1, g] += eps
            assert np.sum((x - oracle.dequant(d2, s, beta)) ** 2) > base


@pytest.mark.parametrize("beta", [1, 2, 4, 8, 16, 32, 64, 128])
def test_angle_closed_form(beta):
    """For x ~ N(0,1)^n: cos^2 angle(x, H_beta(x)) -> 2/pi + (1 - 2/pi)/beta, i.e. 0 deg at beta = 1
    rising to arccos(sqrt(2/pi)) = 37.07 deg; the paper reports saturation near 37 deg for beta > 8."""
    n = 1 << 20
    x = np.random.default_rng(15).standard_normal((1, n)).astype(np.float32)
    d, s = oracle.quantize(x, beta)
    xt = oracle.dequant(d, s, beta)[0]
    xd = x[0].astype(np.float64)
    cosang = xd @ xt / math.sqrt((xd @ xd) * (xt @ xt))
    ang = math.degrees(math.acos(min(1.0, cosang)))
    closed = math.degrees(math.acos(math.sqrt(2 / math.pi + (1 - 2 / math.pi) / beta)))
    assert abs(ang - closed) < 0.1
    if beta > 8:
        assert abs(ang - float(_golden("angle.txt")["saturation_degrees"])) < 2.0
    if beta == 1:
        assert ang < 1e-3


def test_tail_group_uses_its_own_length():
    x = np.array([[1, 2, 3, 4, 5, 6, 7]], dtype=np.float32)
    d, _ = oracle.quantize(x, 4)
    assert d.tolist() == [[2.5, 6.0]]
    assert oracle.n_groups(7, 4) == 2


def test_scale_storage_rounding():
    v = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 0.1, 3.0e-39])
    f = oracle.round_scales(v, "f32")
    assert np.array_equal(f, v.astype(np.float32).astype(np.float64))
    b = oracle.round_scales(v, "bf16")
    # bf16 has 8 significant bits: ties go to even, anything above the tie goes up
    assert b[0] == 1.0 and b[1] == 1.0 and b[2] == 1.0 + 2.0 ** -6 and b[3] == 1.0 + 2.0 ** -7
    import torch
    tb = torch.tensor(v, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(b, tb)


# ---------------------------------------------------------------- im2col index map
@pytest.mark.parametrize("B,C,H,W,kh,kw,st,pd", [(2, 3, 5, 6, 3, 3, 1, 1), (1, 4, 7, 7, 3, 3, 2, 0), (2, 2, 4, 5, 1, 1, 1, 0),
                                               (1, 2, 6, 6, 5, 3, 1, 2)])
def test_im2col_matches_unfold(B, C, H, W, kh, kw, st, pd):
    import torch
    x = np.random.default_rng(16).standard_normal((B, C, H, W)).astype(np.float32)
    got = oracle.im2col(x, kh, kw, (st, st), (pd, pd))
    ref = torch.nn.functional.unfold(torch.from_numpy(x), (kh, kw), padding=pd, stride=st)  # [B, C*kh*kw, L]
    ref = ref.permute(0, 2, 1).reshape(-1, C * kh * kw).numpy()
    assert np.array_equal(got, ref)


def test_hbwn_conv_equals_direct_convolution_with_binarized_filters():
    """beta_a = 1: the im2col product must equal a direct convolution with W~ reshaped back to
    (filters, c, kh, kw) -- this pins the k = (c, i, j) order against Reshape(W, (S[0], -1))."""
    import torch
    rng = np.random.default_rng(17)
    x = rng.standard_normal((2, 3, 6, 5)).astype(np.float32)
    w4 = rng.standard_normal((4, 3, 3, 3)).astype(np.float32)
    w2d = w4.reshape(4, -1)
    c, _ = oracle.conv_im2col(x, w2d, 3, 3, (1, 1), (1, 1), 1, 9)
    wt = _np_hadamard(w2d, 9).reshape(4, 3, 3, 3)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(wt), padding=1)
    ref = ref.permute(0, 2, 3, 1).reshape(-1, 4).numpy()  # NHWC rows
    np.testing.assert_allclose(c, ref, rtol=0, atol=1e-12)


def test_conv_hbmm_binarizes_im2col_rows_along_k():
    """beta_a > 1: activations are grouped along K of the im2col row (the form Eq. 7 is stated for)."""
    rng = np.random.default_rng(18)
    x = rng.standard_normal((1, 4, 4, 4)).astype(np.float32)
    w2d = rng.standard_normal((3, 36)).astype(np.float32)
    c, _ = oracle.conv_im2col(x, w2d, 3, 3, (1, 1), (1, 1), 4, 12)
    import torch
    cols = torch.nn.functional.unfold(torch.from_numpy(x), 3, padding=1).permute(0, 2, 1).reshape(-1, 36).numpy()
    ref = _np_hadamard(cols, 4) @ _np_hadamard(w2d, 12).T
    np.testing.assert_allclose(c, ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- gradient through the binarization (Eq. 5, Eq. 6)
def _hadamard_objective(x64, gy64, beta):
    """sum(gy * (delta (.) Sign(x))) in exact rational arithmetic is overkill here: float64 with values that
    are small dyadic rationals keeps every step exact."""
    rows, K = x64.shape
    total = 0.0
    for r in range(rows):
        for k0 in range(0, K, beta):
            seg = x64[r, k0:k0 + beta]
            d = np.abs(seg).sum() / len(seg)
            total += float((gy64[r, k0:k0 + beta] * d * np.where(seg >= 0, 1.0, -1.0)).sum())
    return total


def test_binarize_backward_hand_example():
    """x = (0.5, -2), gy = (1, 3), beta = 2: s = (+1, -1), delta = 1.25, sum gy*s = -2.
    First term (1/2) s_i (-2) = (-1, +1); estimator term delta*gy_i*[|x_i| <= 1] = (1.25, 0)."""
    gx = oracle.binarize_backward(np.array([[0.5, -2.0]], np.float32), np.array([[1.0, 3.0]], np.float32), 2)
    assert np.array_equal(gx, np.array([[0.25, 1.0]]))


@pytest.mark.parametrize("K,beta", [(12, 4), (10, 4), (9, 2), (16, 16), (7, 1), (5, 8)])
def test_binarize_backward_first_term_is_the_exact_derivative_with_signs_held(K, beta):
    """Away from |x| <= 1 the estimator term vanishes, and delta (.) Sign(x) is piecewise linear in x: a
    finite difference that does not cross zero gives dC/dx exactly (dyadic inputs: no rounding at all).
    Pins the group sum, its 1/n_g factor (tail group included), both sign factors and the row layout."""
    rng = np.random.default_rng(700 + K + beta)
    x = (rng.integers(9, 40, size=(3, K)) / 8.0 * rng.choice([-1.0, 1.0], size=(3, K))).astype(np.float32)   # 1.125 <= |x| < 5
    gy = (rng.integers(-16, 17, size=(3, K)) / 4.0).astype(np.float32)
    gx = oracle.binarize_backward(x, gy, beta)
    x64, gy64 = x.astype(np.float64), gy.astype(np.float64)
    f0 = _hadamard_objective(x64, gy64, beta)
    h = 2.0 ** -6
    for r in range(3):
        for i in range(K):
            xp = x64.copy()
            xp[r, i] += h * (1.0 if xp[r, i] > 0 else -1.0)          # away from zero
            fd = (_hadamard_objective(xp, gy64, beta) - f0) / h * (1.0 if x64[r, i] > 0 else -1.0)
            assert abs(fd - gx[r, i]) < 1e-9, (r, i, fd, gx[r, i])


def test_binarize_backward_estimator_term_and_its_threshold():
    """Eq. 5: the straight-through term delta_g * gy_i is added exactly where |x_i| <= 1 (inclusive)."""
    x = np.array([[1.0, -1.0, 1.0000001, -0.25, 0.0, 3.0, -1.5, 0.75]], np.float32)
    gy = np.array([[2.0, -3.0, 5.0, 7.0, -1.0, 4.0, 0.5, 8.0]], np.float32)
    beta = 4
    gx = oracle.binarize_backward(x, gy, beta)
    x64 = x.astype(np.float64)
    s = np.where(x64 >= 0, 1.0, -1.0)                                  # Sign(0) = +1
    for g in range(2):
        sl = slice(4 * g, 4 * g + 4)
        delta = np.abs(x64[0, sl]).mean()
        first = s[0, sl] * (gy[0, sl].astype(np.float64) * s[0, sl]).sum() / 4.0
        ste = gx[0, sl] - first
        expect = np.where(np.abs(x64[0, sl]) <= 1.0, delta * gy[0, sl], 0.0)
        np.testing.assert_allclose(ste, expect, rtol=0, atol=1e-12)
    assert gx[0, 2] - (s[0, 2] * (gy[0, :4] * s[0, :4]).sum() / 4.0) == 0.0     # 1.0000001 > 1: no estimator term


def test_binarize_backward_beta_one():
    """beta = 1: delta = |x| and X~ = X, so Eq. 6 gives gy_i * (1 + |x_i| [|x_i| <= 1])."""
    rng = np.random.default_rng(71)
    x = rng.standard_normal((4, 9)).astype(np.float32)
    gy = rng.standard_normal((4, 9)).astype(np.float32)
    gx = oracle.binarize_backward(x, gy, 1)
    x64, g64 = x.astype(np.float64), gy.astype(np.float64)
    np.testing.assert_allclose(gx, g64 * (1.0 + np.abs(x64) * (np.abs(x64) <= 1.0)), rtol=0, atol=1e-15)


# ---------------------------------------------------------------- Eq. 3 as printed: groups along the rows of the activation map
def test_binarize_map_hand_example():
    """A 2 x 4 map with beta_a = 2, worked by hand: (1,-3) -> delta 2; (0,2) -> delta 1 with Sign(0) = +1;
    (-.5,-.5) -> delta .5; (4,-2) -> delta 3."""
    x = np.array([[[[1.0, -3.0, 0.0, 2.0], [-0.5, -0.5, 4.0, -2.0]]]], dtype=np.float32)
    want = np.array([[[[2.0, -2.0, 1.0, 1.0], [-0.5, -0.5, 3.0, -3.0]]]])
    assert np.array_equal(oracle.binarize_map(x, 2), want)


def test_binarize_map_groups_run_along_the_width_only():
    """Each (batch, channel, height) line is binarized on its own: permuting lines permutes the result, the group
    sums of |A~| equal those of |A| (delta is the mean), and a tail run of one element is kept as it is."""
    rng = np.random.default_rng(31)
    x = rng.standard_normal((2, 3, 4, 7)).astype(np.float32)
    got = oracle.binarize_map(x, 3)
    perm = rng.permutation(4)
    assert np.array_equal(oracle.binarize_map(x[:, :, perm, :], 3), got[:, :, perm, :])
    assert np.array_equal(oracle.binarize_map(x.transpose(1, 0, 2, 3).copy(), 3), got.transpose(1, 0, 2, 3))
    for g0 in (0, 3):
        np.testing.assert_allclose(np.abs(got[..., g0:g0 + 3]).sum(-1), np.abs(x[..., g0:g0 + 3].astype(np.float64)).sum(-1), rtol=1e-15)
        assert np.all(np.abs(got[..., g0:g0 + 3]) == np.abs(got[..., g0:g0 + 1]))        # one magnitude per group
    assert np.array_equal(got[..., 6], x[..., 6].astype(np.float64))                      # tail group of length 1
    assert np.array_equal(np.signbit(got), np.signbit(x) & (x != 0))
    assert np.array_equal(oracle.binarize_map(x, 1), x.astype(np.float64))                # beta_a = 1: full precision
    assert np.array_equal(oracle.binarize_map(x, 64), oracle.binarize_map(x, 7))          # beta_a above the width: one group per line


def test_conv_of_map_binarized_activations_brute_force():
    """Direct convolution, written as plain loops, of a map binarized by plain loops with filters binarized by plain
    loops: strided, padded, width not a multiple of beta_a."""
    rng = np.random.default_rng(32)
    B, C, H, W, F, kh, kw, st, pd, ba, bw = 2, 2, 5, 6, 3, 3, 3, 2, 1, 4, 6
    x = (rng.integers(-8, 9, size=(B, C, H, W)) / 4.0).astype(np.float32)
    w4 = (rng.integers(-8, 9, size=(F, C, kh, kw)) / 8.0).astype(np.float32)
    at = np.zeros((B, C, H, W))
    for b in range(B):
        for c in range(C):
            for y in range(H):
                for x0 in range(0, W, ba):
                    seg = x[b, c, y, x0:x0 + ba].astype(np.float64)
                    d = sum(abs(v) for v in seg) / len(seg)
                    for t, v in enumerate(seg):
                        at[b, c, y, x0 + t] = d if v >= 0 else -d
    w2d = w4.reshape(F, -1)
    wt = np.zeros(w2d.shape)
    for f in range(F):
        for k0 in range(0, w2d.shape[1], bw):
            seg = w2d[f, k0:k0 + bw].astype(np.float64)
            d = sum(abs(v) for v in seg) / len(seg)
            for t, v in enumerate(seg):
                wt[f, k0 + t] = d if v >= 0 else -d
    wt4 = wt.reshape(F, C, kh, kw)
    Ho, Wo = (H + 2 * pd - kh) // st + 1, (W + 2 * pd - kw) // st + 1
    ref = np.zeros((B * Ho * Wo, F))
    for b in range(B):
        for yo in range(Ho):
            for xo in range(Wo):
                for f in range(F):
                    acc = 0.0
                    for c in range(C):
                        for i in range(kh):
                            for j in range(kw):
                                y, xx = yo * st + i - pd, xo * st + j - pd
                                if 0 <= y < H and 0 <= xx < W:
                                    acc += at[b, c, y, xx] * wt4[f, c, i, j]
                    ref[(b * Ho + yo) * Wo + xo, f] = acc
    got, absref = oracle.conv_map_binarized(x, w2d, kh, kw, (st, st), (pd, pd), ba, bw)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    assert np.all(absref >= np.abs(got) - 1e-12)


def test_conv_of_map_binarized_activations_special_cases():
    """beta_a = 1 is the HBWN convolution; and a map whose magnitudes are constant along every group is its own
    binarization, so the result is again the HBWN convolution of the map itself."""
    rng = np.random.default_rng(33)
    x = rng.standard_normal((2, 3, 6, 8)).astype(np.float32)
    w2d = rng.standard_normal((4, 27)).astype(np.float32)
    a, _ = oracle.conv_map_binarized(x, w2d, 3, 3, (1, 1), (1, 1), 1, 9)
    b, _ = oracle.conv_im2col(x, w2d, 3, 3, (1, 1), (1, 1), 1, 9)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    mags = np.repeat(rng.integers(1, 9, size=(2, 3, 6, 2)) / 8.0, 4, axis=-1)
    xs = (mags * np.where(rng.standard_normal((2, 3, 6, 8)) >= 0, 1.0, -1.0)).astype(np.float32)
    a, _ = oracle.conv_map_binarized(xs, w2d, 3, 3, (1, 1), (1, 1), 4, 9)
    b, _ = oracle.conv_im2col(xs, w2d, 3, 3, (1, 1), (1, 1), 1, 9)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_im2col_f64_matches_the_float_gather():
    rng = np.random.default_rng(34)
    x = rng.standard_normal((2, 3, 7, 5)).astype(np.float32)
    for kh, kw, st, pd in ((3, 3, (1, 1), (1, 1)), (3, 3, (2, 2), (0, 0)), (1, 1, (1, 1), (0, 0)), (5, 3, (1, 2), (2, 1))):
        assert np.array_equal(oracle.im2col_f64(x.astype(np.float64), kh, kw, st, pd), oracle.im2col(x, kh, kw, st, pd).astype(np.float64))
