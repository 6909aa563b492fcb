"""GPU parity: every result of the CUDA library is compared with the CPU oracle on the same seeded
inputs, through the C-ABI binding.  Bits and integer partials must match exactly; scales within the
bound of an fp32 pairwise sum; products within 1e-5 of the magnitude reference sum |deltaA*deltaW*D|."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_10759_b200 import inputs

pytestmark = pytest.mark.gpu

RTOL = 1e-5          # fp32 products (relative to sum_t |deltaA * deltaW * D_t|)
RTOL_BF16 = 1e-2     # paths whose inputs or scales are stored in bf16, end to end from raw data


@pytest.fixture(scope="module")
def hb():
    from paper_1905_10759_b200 import hbmm
    yield hbmm
    assert hbmm.last_device_error() == 0      # no bounded device-side wait expired during these tests


def _gu():
    import gpu_util
    return gpu_util


# ------------------------------------------------------------------ quantize / pack
QUANT_CASES = [
    # rows, K, beta, x bf16?, scale dtype, ldx pad
    (256, 256, 32, False, 0, 0),
    (37, 100, 32, False, 0, 0),
    (5, 45, 32, False, 0, 3),      # ragged K, unaligned rows -> scalar loads
    (64, 576, 32, False, 0, 0),
    (64, 576, 64, False, 1, 0),
    (33, 576, 128, False, 0, 0),   # 128 does not divide 576: tail group of 64
    (16, 1152, 256, False, 0, 0),  # general path
    (7, 384, 96, False, 0, 0),     # group of three words
    (9, 577, 577, False, 0, 0),    # one group per row, ragged
    (3, 4608, 4608, False, 1, 0),
    (130, 1000, 64, True, 0, 0),   # bf16 input
    (20, 333, 32, True, 1, 8),
    (11, 2048, 256, True, 0, 0),
    (1, 1, 32, False, 0, 0),
    # sub-word groups, the settings of the paper's experiments (Section 5: beta 2 .. 16)
    (64, 576, 16, False, 0, 0),
    (37, 100, 8, False, 0, 0),     # ragged K: 100 = 12 * 8 + 4, tail group of four
    (33, 333, 4, False, 1, 0),     # tail group of one element, bf16 scales
    (20, 576, 2, False, 0, 0),
    (5, 45, 2, False, 0, 3),       # unaligned rows -> scalar loads, odd K
    (130, 1000, 16, True, 0, 0),   # bf16 input: eight elements per thread
    (16, 264, 8, True, 1, 0),
    (9, 77, 4, True, 0, 8),
    (12, 512, 2, True, 0, 0),
    (4, 8, 16, False, 0, 0),       # beta >= K: one group per row
]


@pytest.mark.parametrize("rows,K,beta,xbf16,sdt,ldpad", QUANT_CASES)
def test_quantize_bits_exact_scales_within_bound(hb, rows, K, beta, xbf16, sdt, ldpad):
    gu = _gu()
    x = inputs.normal((rows, K), 1000 + rows + K + beta)
    x[0, 0] = 0.0
    if K > 2:
        x[rows // 2, 1] = -0.0
    if xbf16:
        xb, x = inputs.as_bf16(x)
    delta, sign = oracle.quantize(x, beta)
    xd = torch.zeros((rows, K + ldpad), dtype=torch.float32)
    xd[:, :K] = torch.from_numpy(x)
    xd = xd.cuda()
    if xbf16:
        xd = xd.to(torch.bfloat16)  # exact: values are bf16-representable
    out = hb.alloc_operand(rows, K, beta, sdt)
    out.bits.fill_(-1)
    out.scales.fill_(float("nan"))
    hb.quantize(xd[:, :K], out)
    torch.cuda.synchronize()
    bits = gu.host_bits(out.bits)
    assert np.array_equal(bits, oracle.pack(sign, bits.shape[1]))          # includes zero pad bits / words
    G = delta.shape[1]
    sc = out.scales.float().cpu().numpy().astype(np.float64)
    assert np.all(sc[:, G:] == 0.0)
    be = gu.eff_beta(beta, K)
    depth = int(np.ceil(np.log2(be))) + int(np.ceil(be / 1024)) + 2     # pairwise tree (+ lane-strided part)
    tol = depth * gu.U
    if sdt == hb.BF16:
        tol += 2.0 ** -8                                                  # half an ulp of bf16 (8 significant bits)
    np.testing.assert_allclose(sc[:, :G], delta, rtol=tol, atol=0)


def test_quantize_signs_of_special_values(hb):
    gu = _gu()
    x = np.zeros((2, 64), dtype=np.float32)
    x[0, :] = [(-1.0) ** k * 1e-38 * (k % 3) for k in range(64)]   # zeros, +-tiny
    x[1, ::2] = -0.0
    x[1, 1::2] = np.float32(3e36)   # 16 of them still sum below the fp32 maximum
    out = hb.alloc_operand(2, 64, 32, 0)
    hb.quantize(torch.from_numpy(x).cuda(), out)
    delta, sign = oracle.quantize(x, 32)
    assert np.array_equal(gu.host_bits(out.bits), oracle.pack(sign, 4))
    np.testing.assert_allclose(out.scales.cpu().numpy()[:, :2], delta, rtol=8 * gu.U)


# ------------------------------------------------------------------ integer partials (bit exact)
PARTIAL_CASES = [(33, 17, 256, 32, 32), (20, 9, 100, 32, 64), (8, 8, 576, 128, 32), (5, 6, 333, 333, 32),
                 (4, 3, 384, 96, 96), (6, 7, 77, 77, 77), (3, 5, 1024, 256, 64),
                 # sub-word segments: masked popcounts inside a word
                 (9, 7, 256, 16, 16), (6, 5, 100, 4, 4), (5, 4, 77, 2, 16), (4, 6, 128, 8, 64), (3, 3, 45, 45, 2)]


@pytest.mark.parametrize("M,N,K,ba,bw", PARTIAL_CASES)
def test_partials_bit_exact(hb, M, N, K, ba, bw):
    gu = _gu()
    a = inputs.normal((M, K), 2000 + M + K)
    w = inputs.normal((N, K), 3000 + N + K)
    A, _, sa = gu.oracle_operand(a, ba)
    W, _, sw = gu.oracle_operand(w, bw)
    d_ref, _ = oracle.partials(sa, sw, gu.eff_beta(ba, K), gu.eff_beta(bw, K))
    D = torch.empty(d_ref.shape, dtype=torch.int32, device="cuda")
    hb.gemm_partials(A, W, D, hb.PATH_POPC)
    assert np.array_equal(D.cpu().numpy(), d_ref)


@pytest.mark.parametrize("M,N,K,ba,bw", [(33, 17, 576, 128, 128), (20, 9, 1024, 256, 128), (6, 7, 77, 77, 77),
                                         (40, 70, 640, 128, 640), (65, 66, 200, 128, 128)])
def test_partials_bit_exact_on_the_b1_tensor_instruction(hb, M, N, K, ba, bw):
    gu = _gu()
    a = inputs.normal((M, K), 2100 + M + K)
    w = inputs.normal((N, K), 3100 + N + K)
    A, _, sa = gu.oracle_operand(a, ba)
    W, _, sw = gu.oracle_operand(w, bw)
    d_ref, _ = oracle.partials(sa, sw, gu.eff_beta(ba, K), gu.eff_beta(bw, K))
    D = torch.full(d_ref.shape, -12345, dtype=torch.int32, device="cuda")
    hb.gemm_partials(A, W, D, hb.PATH_B1MMA)
    assert np.array_equal(D.cpu().numpy(), d_ref)


# ------------------------------------------------------------------ packed x packed contraction
GEMM_CASES = [
    # M, N, K, beta_a, beta_w, scale dtype
    (256, 256, 256, 32, 32, 0),      # the 256^3 configuration
    (130, 70, 100, 32, 32, 0),       # ragged everywhere, tail segment of 4 bits
    (300, 64, 576, 32, 32, 0),       # narrow-N tile
    (129, 200, 576, 64, 64, 0),
    (77, 129, 576, 128, 128, 0),     # 576 = 4*128 + 64: short tail segment
    (64, 96, 1024, 256, 256, 0),
    (100, 100, 512, 32, 128, 0),     # beta_a < beta_w: finer segmentation decides
    (100, 100, 512, 128, 32, 1),     # and the other way, bf16 scales
    (65, 63, 384, 96, 96, 0),        # generic segment length
    (50, 60, 333, 333, 333, 0),      # XNOR-Net case, one scale per row
    (50, 60, 320, 320, 32, 0),       # one group per row against beta 32
    (40, 1000, 4096, 64, 64, 0),     # FC-style ragged N = 1000
    (1, 1000, 4096, 64, 64, 0),      # batch 1
    (3, 5, 31, 32, 32, 0),           # K below one word
    # at most eight activation rows: the matrix-vector kernel (one warp per weight row)
    (7, 129, 333, 32, 32, 0),        # ragged K: tail segment of 13 bits
    (8, 130, 576, 128, 32, 0),       # mixed groups, 576 = 4 * 128 + 64
    (5, 64, 320, 320, 64, 0),        # one activation group per row
    (2, 33, 200, 64, 64, 1),         # bf16 scales, tail segment of 8 bits
    (4, 1000, 9216, 64, 64, 0),      # the first fully connected layer's depth
    # sub-word groups (beta 2 .. 16, Section 5), alone and mixed as in the paper's tables (beta_a <= beta_w)
    (200, 72, 576, 16, 16, 0),
    (130, 140, 1152, 4, 4, 0),
    (70, 64, 256, 2, 16, 0),
    (65, 33, 320, 8, 64, 0),         # sub-word activations against word-multiple weight groups
    (40, 50, 384, 2, 2, 1),          # bf16 scales
    (33, 40, 100, 4, 8, 0),          # K no multiple of 32: integer-pipe path only
    (50, 60, 320, 320, 16, 0),       # one group per row against beta 16
    (300, 130, 640, 32, 8, 0),       # finer weight groups
    # sub-word activation groups whose scales reach the producers through shared memory (beta_a <= 8), several tiles,
    # ragged rows; 512 or more scales per row: the rows' largest scales come from a kernel of their own
    (300, 130, 1152, 8, 8, 0),
    (260, 72, 2048, 2, 16, 0),       # 1024 scales per row
    (150, 200, 4608, 8, 32, 0),      # 576 scales per row, tail stage of one word... K = 144 words
    (140, 64, 1056, 4, 4, 0),        # odd number of words: the last stage holds one word
]


def _paths(hb):
    return [hb.PATH_POPC, hb.PATH_B1MMA, hb.PATH_TENSOR, hb.PATH_FOLDED, hb.PATH_AUTO]


def _gemm_ws(hb, A, W):
    """Workspace of the contraction (the tensor-core path keeps its expanded weight operand there)."""
    n = hb.gemm_workspace_bytes(A, W)
    return torch.empty(max(n, 16), dtype=torch.uint8, device="cuda")


@pytest.mark.parametrize("M,N,K,ba,bw,sdt", GEMM_CASES)
def test_gemm_matches_oracle_on_every_path(hb, M, N, K, ba, bw, sdt):
    gu = _gu()
    a = inputs.normal((M, K), 4000 + M + K + ba)
    w = inputs.he_normal(N, K, 5000 + N + K + bw)
    A, da, sa = gu.oracle_operand(a, ba, sdt)
    W, dw, sw = gu.oracle_operand(w, bw, sdt)
    c_ref, absref = oracle.hbmm_from_quantized(da, sa, gu.eff_beta(ba, K), dw, sw, gu.eff_beta(bw, K))
    # the folded-scale kernel (what AUTO runs when it has the workspace) sums the individual products in
    # fp32: where every group dot is zero the magnitude reference is zero and a few ulps of F remain
    fine = gu.elementwise_magnitude(da, gu.eff_beta(ba, K), dw, gu.eff_beta(bw, K), K)
    must_run = gu.expected_paths(K, ba, bw)
    ws = _gemm_ws(hb, A, W)
    for path in _paths(hb):
        ldc = (N + 3) // 4 * 4 + 4
        C = torch.full((M, ldc), float("nan"), device="cuda")
        if path not in must_run:
            with pytest.raises(hb.HbmmError) as e:
                hb.gemm_ex(A, W, C, path, ws)
            assert e.value.status == hb.ERR_UNSUPPORTED
            continue
        hb.gemm_ex(A, W, C, path, ws)              # a path that takes these operands today must keep taking them
        out = C.cpu().numpy()
        assert np.isnan(out[:, N:]).all()          # nothing written beyond column N
        folded = path == hb.PATH_FOLDED or (path == hb.PATH_AUTO and gu.auto_runs_folded(K, ba, bw))
        gu.assert_close_rel_absref(out[:, :N], c_ref, absref, RTOL, "path %d" % path, fine if folded else None)


@pytest.mark.parametrize("M,N,K,beta", [(200, 130, 576, 32), (70, 64, 1152, 64), (33, 140, 640, 128)])
def test_unit_scales_give_exact_integers(hb, M, N, K, beta):
    """All scales 1: C must equal K - 2*popc(xor) exactly (every value is a small integer in fp32)."""
    gu = _gu()
    rng = np.random.default_rng(M + N)
    sa = rng.choice(np.array([-1, 1], dtype=np.int8), size=(M, K))
    sw = rng.choice(np.array([-1, 1], dtype=np.int8), size=(N, K))
    G = oracle.n_groups(K, beta)
    _, _, lw, ls = hb.operand_bytes(M, K, beta, hb.F32)
    A = hb.wrap_packed(gu.dev_bits(oracle.pack(sa, lw)), gu.scales_to_dev(np.ones((M, G)), hb.F32, ls), K, beta)
    W = hb.wrap_packed(gu.dev_bits(oracle.pack(sw, lw)), gu.scales_to_dev(np.ones((N, G)), hb.F32, ls), K, beta)
    ref = sa.astype(np.int32) @ sw.astype(np.int32).T
    ws = _gemm_ws(hb, A, W)
    must_run = gu.expected_paths(K, beta, beta)
    for path in _paths(hb):
        C = torch.empty((M, (N + 3) // 4 * 4), device="cuda")
        if path not in must_run:
            with pytest.raises(hb.HbmmError) as e:
                hb.gemm_ex(A, W, C, path, ws)
            assert e.value.status == hb.ERR_UNSUPPORTED
            continue
        hb.gemm_ex(A, W, C, path, ws)
        assert np.array_equal(C.cpu().numpy()[:, :N], ref.astype(np.float32)), path


def test_quantize_then_gemm_end_to_end(hb):
    """Raw fp32 inputs through hbmm_quantize and hbmm_gemm against the oracle from raw inputs."""
    gu = _gu()
    M, N, K = 256, 256, 256
    a = inputs.normal((M, K), inputs.SEEDS["square256"][0])
    w = inputs.normal((N, K), inputs.SEEDS["square256"][1])
    for sdt, rtol in [(hb.F32, RTOL), (hb.BF16, RTOL_BF16)]:
        A = hb.quantize(torch.from_numpy(a).cuda(), hb.alloc_operand(M, K, 32, sdt))
        W = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(N, K, 32, sdt))
        C = torch.empty((M, N), device="cuda")
        hb.gemm(A, W, C, _gemm_ws(hb, A, W))
        c_ref, absref = oracle.hbmm(a, w, 32, 32, None)       # exact scales: the GPU's rounding is inside rtol
        gu.assert_close_rel_absref(C.cpu().numpy(), c_ref, absref, rtol)


# ------------------------------------------------------------------ HBWN (beta_a = 1)
HBWN_CASES = [(130, 72, 576, 16, True), (65, 40, 320, 4, True), (40, 33, 100, 2, False), (70, 130, 256, 8, True),   # sub-word weight groups
              (256, 64, 576, 32, True), (100, 130, 1152, 32, True), (65, 70, 100, 32, True), (40, 33, 576, 64, False),
              (30, 40, 333, 333, True), (129, 256, 2304, 32, True), (8, 16, 64, 32, False), (300, 64, 576, 64, True),
              (130, 200, 672, 128, True), (70, 50, 96, 64, True), (257, 129, 1160, 1160, True), (33, 64, 40, 32, True),
              (64, 72, 384, 96, True)]


def _hbwn_rtol(gu, K, beta_w, two_pieces=False):
    be = gu.eff_beta(beta_w, K)
    rtol = (be + -(-K // be) + 4) * 2 * gu.U       # sequential fp32 sums inside and across groups, x2 margin
    if two_pieces:
        rtol += 2.0 ** -18                         # the default tensor-core kernel carries the weight scale in two bf16 pieces
    return rtol


@pytest.mark.parametrize("M,N,K,bw,abf16", HBWN_CASES)
def test_hbwn_matches_oracle(hb, M, N, K, bw, abf16):
    gu = _gu()
    a = inputs.normal((M, K), 6000 + M + K)
    w = inputs.he_normal(N, K, 7000 + N + K)
    if abf16:
        _, a = inputs.as_bf16(a)
    W, dw, sw = gu.oracle_operand(w, bw)
    c_ref, absref = oracle.hbwn_from_quantized(a, dw, sw, gu.eff_beta(bw, K))
    ad = torch.from_numpy(a).cuda()
    if abf16:
        ad = ad.to(torch.bfloat16)
    rtol = _hbwn_rtol(gu, K, bw)
    rtol2 = _hbwn_rtol(gu, K, bw, True)
    assert rtol2 < RTOL_BF16
    A = hb.wrap_dense(ad)
    ws = _gemm_ws(hb, A, W)
    ran = 0
    # TENSOR: tcgen05 kernel, three weight pieces; FOLDED (and AUTO with a workspace): two pieces;
    # B1MMA: warp-level bf16 mma.sync kernel; POPC: fp32 sign-select kernel
    for path, wsp in ((hb.PATH_AUTO, ws), (hb.PATH_AUTO, None), (hb.PATH_TENSOR, ws), (hb.PATH_FOLDED, ws), (hb.PATH_B1MMA, None),
                      (hb.PATH_POPC, None)):
        C = torch.full((M, (N + 3) // 4 * 4 + 4), float("nan"), device="cuda")
        try:
            hb.gemm_ex(A, W, C, path, wsp)
        except hb.HbmmError as e:
            # the two tensor-core kernels take bf16 activations whose rows start on 16-byte boundaries
            assert e.status == hb.ERR_UNSUPPORTED and path in (hb.PATH_TENSOR, hb.PATH_FOLDED, hb.PATH_B1MMA)
            if path in (hb.PATH_TENSOR, hb.PATH_FOLDED):
                assert not abf16 or K % 8 != 0
            continue
        ran += 1
        out = C.cpu().numpy()
        assert np.isnan(out[:, N:]).all()
        two = wsp is not None and path in (hb.PATH_AUTO, hb.PATH_FOLDED)
        gu.assert_close_rel_absref(out[:, :N], c_ref, absref, rtol2 if two else rtol, "hbwn path %d" % path)
    assert ran >= (4 if abf16 and K % 8 == 0 else 2)


def test_hbwn_tensor_path_needs_its_workspace(hb):
    gu = _gu()
    M, N, K = 64, 64, 128
    _, a = inputs.as_bf16(inputs.normal((M, K), 61))
    W, dw, sw = gu.oracle_operand(inputs.he_normal(N, K, 62), 32)
    A = hb.wrap_dense(torch.from_numpy(a).cuda().to(torch.bfloat16))
    assert hb.gemm_workspace_bytes(A, W) > 0
    C = torch.empty((M, N), device="cuda")
    with pytest.raises(hb.HbmmError) as e:
        hb.gemm_ex(A, W, C, hb.PATH_TENSOR)
    assert e.value.status == hb.ERR_WORKSPACE


# ------------------------------------------------------------------ convolution front end
CONV_CASES = [
    # B, C, H, W, N, kh, kw, stride, pad, beta_a, beta_w, signed, x bf16
    # sub-word groups (Section 5: beta_a / beta_w such as 2/16, 4/4, 1/4)
    (2, 64, 8, 8, 64, 3, 3, 1, 1, 16, 16, True, False),
    (2, 32, 6, 6, 16, 3, 3, 1, 1, 2, 16, True, False),
    (2, 20, 7, 7, 33, 3, 3, 1, 1, 4, 4, True, False),       # K = 180: no whole words, integer-pipe contraction
    (2, 64, 8, 8, 64, 3, 3, 1, 1, 1, 4, True, True),        # HBWN with beta_w = 4
    (2, 64, 8, 8, 64, 3, 3, 1, 1, 32, 32, True, False),
    (2, 64, 8, 8, 64, 3, 3, 1, 1, 32, 32, False, False),    # post-ReLU: every sign bit is 1
    (3, 32, 7, 9, 40, 3, 3, 1, 1, 64, 32, True, False),
    (2, 16, 9, 9, 20, 3, 3, 2, 0, 32, 32, True, False),     # stride 2, no padding
    (1, 8, 6, 6, 12, 5, 5, 1, 2, 200, 200, True, False),    # one group per row
    (2, 24, 5, 5, 16, 1, 1, 1, 0, 32, 32, True, True),      # 1x1, bf16 input, K = 24 below a word
    (2, 64, 8, 8, 64, 3, 3, 1, 1, 1, 32, True, True),       # HBWN
    (2, 20, 7, 7, 33, 3, 3, 1, 1, 1, 32, False, False),     # HBWN from fp32 input (rounded to bf16 rows)
    # packed front end with the input tile staged by tensor copies (fp32 input, W % 4 == 0, stride 1 along x)
    (2, 96, 20, 20, 40, 3, 3, 1, 1, 32, 32, True, False),   # several row blocks and channel ranges
    (2, 40, 8, 8, 24, 5, 5, 1, 2, 32, 32, True, False),     # 5x5, last chunk of 8 channels
    (1, 64, 12, 12, 16, 1, 1, 1, 0, 32, 32, True, False),   # 1x1
    (3, 70, 16, 12, 33, 3, 3, 1, 0, 32, 64, True, False),   # no padding, ragged channels, beta_w = 64
    (2, 64, 8, 8, 16, 3, 3, 1, 1, 32, 32, None, False),     # zeros of both signs in the input
    # ... and with whole channel planes staged by bulk copies when rows are not multiples of 16 bytes
    (2, 64, 7, 7, 24, 3, 3, 1, 1, 32, 32, True, False),
    (3, 96, 14, 14, 40, 3, 3, 1, 1, 32, 32, True, False),
    (2, 32, 9, 10, 16, 1, 1, 1, 0, 32, 32, True, False),
    (2, 64, 7, 7, 24, 3, 3, 1, 0, 32, 32, None, False),     # no padding, zeros of both signs
    # the same front end with groups shorter than a word (means stored from the gather) and of several words (sums of
    # the words' sums), tiles with halo and whole planes, full and short last chunks, channel ranges
    (2, 96, 20, 20, 40, 3, 3, 1, 1, 4, 4, True, False),
    (2, 96, 20, 20, 40, 3, 3, 1, 1, 64, 64, True, False),
    (2, 128, 12, 12, 24, 3, 3, 1, 1, 128, 32, True, False),  # 1152 = 9 groups of 128
    (3, 70, 16, 12, 33, 3, 3, 1, 0, 8, 32, True, False),     # last chunk of 6 channels, K = 630: last group of 6
    (3, 70, 16, 12, 33, 3, 3, 1, 0, 128, 64, True, False),   # K = 630: last group of 118
    (2, 40, 8, 8, 24, 5, 5, 1, 2, 16, 16, True, False),      # 5x5
    (1, 64, 12, 12, 16, 1, 1, 1, 0, 8, 8, True, False),      # 1x1
    (2, 64, 7, 7, 24, 3, 3, 1, 1, 2, 2, None, False),        # whole planes, zeros of both signs
    (3, 96, 14, 14, 40, 3, 3, 1, 1, 96, 32, True, False),    # groups of three words
    # HBWN with whole 64-channel blocks: no im2col matrix, tiles fetched by im2col-mode tensor copies
    (3, 128, 7, 7, 72, 3, 3, 1, 1, 1, 32, True, False),     # two channel blocks, tiles span images, ragged M and N
    (2, 64, 9, 9, 40, 3, 3, 2, 0, 1, 32, True, True),       # stride 2, no padding
    (2, 64, 10, 10, 64, 3, 3, 2, 1, 1, 64, True, True),     # stride 2 with padding
    (1, 64, 12, 12, 16, 1, 1, 1, 0, 1, 64, True, True),     # 1x1
    (2, 64, 6, 6, 24, 5, 5, 1, 2, 1, 1600, True, True),     # 5x5, one weight group per row
    (5, 192, 14, 14, 130, 3, 3, 1, 1, 1, 96, False, True),  # three blocks, several tiles per image, post-ReLU
    # HBWN, 64 channels, at most 64 filters, stride 1, more row tiles than SMs: every tap reads one staged run of
    # input rows (positions numbered over the padded image; tiles cross image rows, images and the end)
    (8, 64, 50, 50, 40, 3, 3, 1, 1, 1, 32, True, True),     # ragged filters
    (10, 64, 47, 45, 64, 3, 3, 1, 0, 1, 64, True, False),   # no padding, odd extents, fp32 input
    (6, 64, 56, 56, 24, 3, 3, 1, 2, 1, 32, False, True),    # padding wider than the filter needs, post-ReLU
    (8, 64, 51, 51, 33, 2, 2, 1, 0, 1, 32, True, True),     # 2 x 2 filter
    (6, 64, 60, 60, 16, 1, 1, 1, 0, 1, 32, True, True),     # 1 x 1: no halo at all
]


@pytest.mark.parametrize("B,C,H,W,N,kh,kw,st,pd,ba,bw,signed,xbf16", CONV_CASES)
def test_conv_im2col_matches_oracle(hb, B, C, H, W, N, kh, kw, st, pd, ba, bw, signed, xbf16):
    gu = _gu()
    shape = inputs.ConvShape("t", B, C, H, W, N, kh, kw, st, pd)
    x = inputs.conv_activation(shape, 8000 + C + H, signed=bool(signed) or signed is None)
    if signed is None:
        # Sign(+0) = Sign(-0) = +1: plant zeros of both signs
        flat = x.reshape(-1)
        flat[::7] = 0.0
        flat[3::11] = -0.0
    if xbf16 or ba == 1:
        _, xr = inputs.as_bf16(x)     # HBWN rows are bf16: the oracle sees the same rounded values
    else:
        xr = x
    if xbf16:
        x = xr
    K = C * kh * kw
    w = inputs.he_normal(N, K, 9000 + N)
    Wop, dw, sw = gu.oracle_operand(w, bw)
    a_rows = oracle.im2col(xr, kh, kw, (st, st), (pd, pd))
    fine = None
    if ba == 1:
        c_ref, absref = oracle.hbwn_from_quantized(a_rows, dw, sw, gu.eff_beta(bw, K))
        rtol = _hbwn_rtol(gu, K, bw, True)
    else:
        da, sa = oracle.quantize(a_rows, gu.eff_beta(ba, K))
        c_ref, absref = oracle.hbmm_from_quantized(da, sa, gu.eff_beta(ba, K), dw, sw, gu.eff_beta(bw, K))
        rtol = RTOL
        # the contraction that follows the front end is the folded-scale kernel when K is whole words
        if gu.auto_runs_folded(K, ba, bw):
            fine = gu.elementwise_magnitude(da, gu.eff_beta(ba, K), dw, gu.eff_beta(bw, K), K)
    geom = hb.make_geom(B, C, H, W, kh, kw, (st, st), (pd, pd))
    xd = torch.from_numpy(x).cuda()
    if xbf16:
        xd = xd.to(torch.bfloat16)
    nbytes = hb.conv_workspace_bytes(geom, ba, hb.F32, Wop)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    M = c_ref.shape[0]
    Cout = torch.full((M, (N + 3) // 4 * 4), float("nan"), device="cuda")
    hb.conv_im2col(xd, geom, ba, hb.F32, Wop, Cout, ws)
    gu.assert_close_rel_absref(Cout.cpu().numpy()[:, :N], c_ref, absref, rtol, "", fine)
    if ba > 1:
        # the packed activation operand left in the workspace: bits exact
        _, _, lw, ls = hb.operand_bytes(M, K, ba, hb.F32)
        bits = ws[: M * lw * 4].view(torch.int32).reshape(M, lw)
        assert np.array_equal(gu.host_bits(bits), oracle.pack(sa, lw))


def test_tensor_path_needs_its_workspace_and_auto_falls_back(hb):
    """Without a workspace the tensor-core path is refused before any launch, and the automatic choice
    runs the integer-pipe kernel instead; with one, both give the oracle's result."""
    gu = _gu()
    M, N, K = 96, 80, 256
    a = inputs.normal((M, K), 77)
    w = inputs.he_normal(N, K, 78)
    A, da, sa = gu.oracle_operand(a, 32)
    W, dw, sw = gu.oracle_operand(w, 32)
    c_ref, absref = oracle.hbmm_from_quantized(da, sa, 32, dw, sw, 32)
    assert hb.gemm_workspace_bytes(A, W) > 0
    C = torch.empty((M, N), device="cuda")
    with pytest.raises(hb.HbmmError) as e:
        hb.gemm_ex(A, W, C, hb.PATH_TENSOR)
    assert e.value.status == hb.ERR_WORKSPACE
    hb.gemm(A, W, C)                                   # no workspace: integer-pipe path
    gu.assert_close_rel_absref(C.cpu().numpy(), c_ref, absref, RTOL)
    C.zero_()
    hb.gemm(A, W, C, _gemm_ws(hb, A, W))
    gu.assert_close_rel_absref(C.cpu().numpy(), c_ref, absref, RTOL)


def test_prepared_weights_path_repeats_the_tensor_path_bit_for_bit(hb):
    """HBMM_PATH_TENSOR_PREPARED skips the weight expansion and reuses what the previous call left in the
    workspace: same kernel, same operands, so the results are identical."""
    gu = _gu()
    M, N, K = 300, 136, 640
    a = inputs.normal((M, K), 91)
    w = inputs.he_normal(N, K, 92)
    A, da, sa = gu.oracle_operand(a, 32)
    W, dw, sw = gu.oracle_operand(w, 64)
    ws = _gemm_ws(hb, A, W)
    C1 = torch.empty((M, N), device="cuda")
    C2 = torch.full((M, N), float("nan"), device="cuda")
    hb.gemm_ex(A, W, C1, hb.PATH_TENSOR, ws)
    hb.gemm_ex(A, W, C2, hb.PATH_TENSOR_PREPARED, ws)
    assert torch.equal(C1, C2)
    with pytest.raises(hb.HbmmError) as e:
        hb.gemm_ex(A, W, C2, hb.PATH_TENSOR_PREPARED)
    assert e.value.status == hb.ERR_WORKSPACE
    # the folded-scale kernel
    C2.fill_(float("nan"))
    hb.gemm_ex(A, W, C1, hb.PATH_FOLDED, ws)
    hb.gemm_ex(A, W, C2, hb.PATH_FOLDED_PREPARED, ws)
    assert torch.equal(C1, C2)
    # dense activations (HBWN)
    _, ab = inputs.as_bf16(a)
    Ad = hb.wrap_dense(torch.from_numpy(ab).cuda().to(torch.bfloat16))
    wsd = _gemm_ws(hb, Ad, W)
    hb.gemm_ex(Ad, W, C1, hb.PATH_TENSOR, wsd)
    C2.fill_(float("nan"))
    hb.gemm_ex(Ad, W, C2, hb.PATH_TENSOR_PREPARED, wsd)
    assert torch.equal(C1, C2)
    c_ref, absref = oracle.hbwn_from_quantized(ab, dw, sw, 64)
    gu.assert_close_rel_absref(C2.cpu().numpy(), c_ref, absref, _hbwn_rtol(gu, K, 64))
    hb.gemm_ex(Ad, W, C1, hb.PATH_FOLDED, wsd)
    C2.fill_(float("nan"))
    hb.gemm_ex(Ad, W, C2, hb.PATH_FOLDED_PREPARED, wsd)
    assert torch.equal(C1, C2)
    gu.assert_close_rel_absref(C2.cpu().numpy(), c_ref, absref, _hbwn_rtol(gu, K, 64, True))


@pytest.mark.parametrize("spread", [0, 8, 16])
def test_folded_path_keeps_the_tolerance_when_group_scales_differ_by_orders_of_magnitude(hb, spread):
    """The folded-scale kernel normalises every row by a power of two and carries each group scale in two
    fp16 pieces; scales up to 2^17 below the largest of their row keep 22 significant bits.  Rows whose
    groups differ by up to 2^spread, rows that are zero, and very large / very small rows must all
    stay inside the 1e-5 bound."""
    gu = _gu()
    M, N, K, beta = 140, 72, 640, 32
    rng = np.random.default_rng(300 + spread)
    a = inputs.normal((M, K), 301 + spread)
    w = inputs.he_normal(N, K, 302 + spread)
    G = K // beta
    for x in (a, w):
        f = np.exp2(rng.integers(-spread, 1, size=(x.shape[0], G))).astype(np.float32)
        x *= np.repeat(f, beta, axis=1)
    a[3] = 0.0                       # an all-zero row
    a[5] *= np.float32(2.0 ** 60)    # rows far from 1: the normalisation is per row
    a[7] *= np.float32(2.0 ** -60)
    w[2] *= np.float32(2.0 ** 40)
    w[9] *= np.float32(2.0 ** -50)
    A, da, sa = gu.oracle_operand(a, beta)
    W, dw, sw = gu.oracle_operand(w, beta)
    c_ref, absref = oracle.hbmm_from_quantized(da, sa, beta, dw, sw, beta)
    C = torch.full((M, N), float("nan"), device="cuda")
    hb.gemm_ex(A, W, C, hb.PATH_FOLDED, _gemm_ws(hb, A, W))
    out = C.cpu().numpy()
    assert np.all(out[3] == 0.0)
    fine = gu.elementwise_magnitude(da, beta, dw, beta, K)
    # compared block by block, so that the floor of the bound follows each block's own magnitude
    rows_n = np.array([r for r in range(M) if r not in (3, 5, 7)])
    cols_n = np.array([c for c in range(N) if c not in (2, 9)])
    for rows in (rows_n, np.array([5]), np.array([7])):
        for cols in (cols_n, np.array([2]), np.array([9])):
            ix = np.ix_(rows, cols)
            gu.assert_close_rel_absref(out[ix], c_ref[ix], absref[ix], RTOL, "folded, spread 2^%d" % spread, fine[ix])


@pytest.mark.parametrize("beta_a,xbf16,C,H", [(32, False, 64, 12), (1, True, 64, 8), (32, False, 96, 7), (16, False, 32, 6)])
def test_conv_with_prepared_weights_repeats_the_plain_call_bit_for_bit(hb, beta_a, xbf16, C, H):
    """HBMM_CONV_WEIGHTS_PREPARED skips the weight expansion and reuses what an earlier call left in the
    workspace; a second batch through the same workspace must give exactly what the plain call gives."""
    shape = inputs.ConvShape("t", 3, C, H, H, 72, 3, 3, 1, 1)
    K = C * 9
    w = inputs.he_normal(72, K, 511)
    Wop = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(72, K, 32))
    geom = hb.make_geom(3, C, H, H, 3, 3, (1, 1), (1, 1))
    ws = torch.empty(hb.conv_workspace_bytes(geom, beta_a, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty_like(ws)
    outs = []
    for seed in (512, 513):
        x = torch.from_numpy(inputs.conv_activation(shape, seed, signed=True)).cuda()
        if xbf16:
            x = x.to(torch.bfloat16)
        plain = torch.full((shape.M, 72), float("nan"), device="cuda")
        hb.conv_im2col(x, geom, beta_a, hb.F32, Wop, plain, ws2)
        fast = torch.full((shape.M, 72), float("nan"), device="cuda")
        # first batch fills the workspace, every later one states that the weights are still there
        hb.conv_im2col(x, geom, beta_a, hb.F32, Wop, fast, ws, flags=hb.CONV_WEIGHTS_PREPARED if outs else 0)
        assert torch.equal(plain, fast)
        outs.append(fast)
    assert not torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("C,H,beta_a", [(64, 12, 32), (96, 7, 32), (32, 6, 16), (40, 9, 64)])
def test_conv_pack_only_leaves_the_operand_the_contraction_would_read(hb, C, H, beta_a):
    """HBMM_CONV_PACK_ONLY stops after the front end: the packed activation operand in the workspace equals the
    oracle's binarization of the im2col rows, and hbmm_gemm on it repeats the one-call convolution bit for bit."""
    gu = _gu()
    shape = inputs.ConvShape("t", 2, C, H, H, 72, 3, 3, 1, 1)
    K = C * 9
    x = inputs.conv_activation(shape, 640 + C, signed=True)
    Wop = hb.quantize(torch.from_numpy(inputs.he_normal(72, K, 641)).cuda(), hb.alloc_operand(72, K, 32))
    geom = hb.make_geom(2, C, H, H, 3, 3, (1, 1), (1, 1))
    ws = torch.empty(hb.conv_workspace_bytes(geom, beta_a, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)
    xd = torch.from_numpy(x).cuda()
    hb.conv_im2col(xd, geom, beta_a, hb.F32, Wop, None, ws, flags=hb.CONV_PACK_ONLY)
    M = shape.M
    bb, sb, lw, ls = hb.operand_bytes(M, K, beta_a, hb.F32)
    bits = ws[:bb].view(torch.int32).reshape(M, lw)
    off = (bb + 255) // 256 * 256
    scales = ws[off: off + sb].view(torch.float32).reshape(M, ls)
    da, sa = oracle.quantize(oracle.im2col(x, 3, 3, (1, 1), (1, 1)), beta_a)
    assert np.array_equal(gu.host_bits(bits), oracle.pack(sa, lw))
    G = da.shape[1]
    sc = scales.cpu().numpy().astype(np.float64)
    assert np.all(sc[:, G:] == 0.0)
    np.testing.assert_allclose(sc[:, :G], da, rtol=(int(np.ceil(np.log2(beta_a))) + 3) * gu.U, atol=0)
    A = hb.wrap_packed(bits, scales, K, beta_a)
    two = torch.empty((M, 72), device="cuda")
    hb.gemm(A, Wop, two, _gemm_ws(hb, A, Wop))
    one = torch.empty((M, 72), device="cuda")
    ws2 = torch.empty_like(ws)
    hb.conv_im2col(xd, geom, beta_a, hb.F32, Wop, one, ws2)
    assert torch.equal(one, two)
    with pytest.raises(hb.HbmmError) as e:      # a dense activation operand is never left behind
        hb.conv_im2col(xd.to(torch.bfloat16), geom, 1, hb.F32, Wop, None, ws, flags=hb.CONV_PACK_ONLY)
    assert e.value.status == hb.ERR_INVALID_ARG


# ------------------------------------------------------------------ gradient through the binarization (Eq. 5, Eq. 6)
BACKWARD_CASES = [
    # rows, K, beta, row padding of the inputs
    (64, 576, 2, 0), (33, 1152, 4, 0), (20, 256, 8, 0), (17, 512, 16, 0), (130, 576, 32, 0), (9, 1024, 128, 0), (40, 100, 1, 0),
    (7, 333, 4, 0),      # ragged K: tail group of one element -> general kernel
    (12, 96, 96, 0),     # one group per row
    (5, 45, 7, 3),       # odd everything, padded rows
    (16, 128, 256, 0),   # beta > K
]


@pytest.mark.parametrize("rows,K,beta,pad", BACKWARD_CASES)
def test_binarize_backward_matches_oracle(hb, rows, K, beta, pad):
    gu = _gu()
    x = inputs.normal((rows, K), 9100 + rows + K)
    gy = inputs.normal((rows, K), 9200 + rows + beta)
    x[0, :4] = [1.0, -1.0, 0.0, -0.0]                       # estimator threshold (inclusive) and Sign(+-0) = +1
    ref = oracle.binarize_backward(x, gy, beta)
    xd = torch.zeros((rows, K + pad)); xd[:, :K] = torch.from_numpy(x)
    gd = torch.zeros((rows, K + pad)); gd[:, :K] = torch.from_numpy(gy)
    out = torch.full((rows, K + pad), float("nan"), device="cuda")
    hb.binarize_backward(xd.cuda()[:, :K], gd.cuda()[:, :K], beta, out[:, :K])
    got = out.cpu().numpy()
    assert np.isnan(got[:, K:]).all()
    # both terms are fp32 trees over at most beta elements followed by one multiply and one add
    be = gu.eff_beta(beta, K)
    G = -(-K // be)
    x64, g64 = x.astype(np.float64), gy.astype(np.float64)
    mag = np.empty_like(x64)
    for g in range(G):
        sl = slice(g * be, min((g + 1) * be, K))
        n = sl.stop - sl.start
        mag[:, sl] = np.abs(g64[:, sl]).sum(axis=1, keepdims=True) / n + np.abs(x64[:, sl]).mean(axis=1, keepdims=True) * np.abs(g64[:, sl])
    tol = (int(np.ceil(np.log2(max(be, 2)))) + int(np.ceil(be / 32)) + 4) * gu.U
    err = np.abs(got[:, :K].astype(np.float64) - ref)
    assert (err <= tol * mag + 1e-30).all(), float((err / (mag + 1e-30)).max() / gu.U)


# ------------------------------------------------------------------ product fused with the next layer's binarization
FUSED_CASES = [
    # M, N, K, beta_a, beta_w, beta_next, next scale dtype, affine map?
    (200, 128, 576, 32, 32, 32, 0, True),
    (130, 1000, 1024, 64, 64, 64, 0, True),     # ragged N: tail group of 40 columns, absent columns in the last tile
    (70, 64, 256, 32, 32, 4, 0, True),          # narrow tile
    (65, 200, 320, 32, 128, 128, 0, False),     # group as wide as the tile
    (40, 72, 384, 32, 32, 16, 1, True),         # bf16 scales, two column tiles with a ragged second one
    (300, 130, 640, 32, 32, 2, 0, True),
    (129, 256, 2304, 32, 32, 8, 0, False),
]


@pytest.mark.parametrize("M,N,K,ba,bw,bn,sdt,affine", FUSED_CASES)
def test_gemm_binarize_next_matches_oracle(hb, M, N, K, ba, bw, bn, sdt, affine):
    """hbmm_gemm_binarize_next against the composition of the pinned oracle steps: product, affine map,
    binarization of its rows.  Signs are compared where z is outside the product's own error band (inside it
    the fp32 value the kernel computed decides, as the header says); scales to the band's mean plus the
    rounding of a pairwise fp32 tree."""
    gu = _gu()
    a = inputs.normal((M, K), 9300 + M + K)
    w = inputs.he_normal(N, K, 9400 + N + K)
    A, da, sa = gu.oracle_operand(a, ba)
    W, dw, sw = gu.oracle_operand(w, bw)
    c_ref, absref = oracle.hbmm_from_quantized(da, sa, gu.eff_beta(ba, K), dw, sw, gu.eff_beta(bw, K))
    fine = gu.elementwise_magnitude(da, gu.eff_beta(ba, K), dw, gu.eff_beta(bw, K), K)
    rng = np.random.default_rng(M + N)
    bs = (rng.uniform(0.5, 2.0, N) * rng.choice([-1.0, 1.0], N)).astype(np.float32) if affine else np.ones(N, np.float32)
    bh = (0.3 * rng.standard_normal(N)).astype(np.float32) if affine else np.zeros(N, np.float32)
    z_ref = c_ref * bs.astype(np.float64) + bh.astype(np.float64)
    band = np.abs(bs) * (RTOL * absref + gu.FOLDED_FLOOR_ULPS * gu.U * fine) + 4 * gu.U * (np.abs(c_ref * bs) + np.abs(bh)) + 1e-30
    nxt = hb.alloc_operand(M, N, bn, sdt)
    nxt.bits.fill_(-1)
    nxt.scales.fill_(float("nan"))
    ws = _gemm_ws(hb, A, W)
    hb.gemm_binarize_next(A, W, nxt, ws, torch.from_numpy(bs).cuda() if affine else None, torch.from_numpy(bh).cuda() if affine else None)
    torch.cuda.synchronize()
    gu.check_next_operand(nxt, z_ref, band, bn, sdt == hb.BF16)


# ------------------------------------------------------------------ the rest of the layer in the epilogue (Section 5's order)
FUSED_DENSE_CASES = [
    # M, N, K, beta_a (1 = dense bf16 activations), beta_w, ReLU?, affine?, bf16 output?
    (200, 128, 576, 32, 32, True, True, True),
    (130, 1000, 1024, 64, 64, False, True, False),    # ragged N, fp32 out
    (70, 64, 256, 32, 32, True, False, True),         # narrow tile
    (65, 200, 320, 32, 128, True, True, False),
    (300, 130, 640, 1, 32, True, True, True),         # HBWN kernel, ragged N: scalar bf16 stores at the edge
    (129, 256, 1152, 1, 32, False, True, False),
    (40, 64, 128, 1, 64, True, False, True),
]


@pytest.mark.parametrize("M,N,K,ba,bw,relu,affine,obf16", FUSED_DENSE_CASES)
def test_gemm_fused_dense_output_matches_oracle(hb, M, N, K, ba, bw, relu, affine, obf16):
    """hbmm_gemm_fused with a dense output: product -> activation -> per-column affine map -> fp32 or bf16 rows,
    against the same chain applied to the oracle's product in double.  The bound is the product's own tolerance
    carried through the map plus the fp32 arithmetic of the map (and half a bf16 ulp for bf16 rows)."""
    gu = _gu()
    a = inputs.normal((M, K), 9600 + M + K)
    w = inputs.he_normal(N, K, 9700 + N + K)
    W, dw, sw = gu.oracle_operand(w, bw)
    if ba == 1:
        _, a = inputs.as_bf16(a)
        A = hb.wrap_dense(torch.from_numpy(a).cuda().to(torch.bfloat16))
        c_ref, absref = oracle.hbwn_from_quantized(a, dw, sw, gu.eff_beta(bw, K))
        tol_c = _hbwn_rtol(gu, K, bw, True) * absref
    else:
        A, da, sa = gu.oracle_operand(a, ba)
        c_ref, absref = oracle.hbmm_from_quantized(da, sa, gu.eff_beta(ba, K), dw, sw, gu.eff_beta(bw, K))
        fine = gu.elementwise_magnitude(da, gu.eff_beta(ba, K), dw, gu.eff_beta(bw, K), K)
        tol_c = RTOL * absref + gu.FOLDED_FLOOR_ULPS * gu.U * fine
    rng = np.random.default_rng(M + N)
    bs = (rng.uniform(0.5, 2.0, N) * rng.choice([-1.0, 1.0], N)).astype(np.float32) if affine else np.ones(N, np.float32)
    bh = (0.3 * rng.standard_normal(N)).astype(np.float32) if affine else np.zeros(N, np.float32)
    y_ref = np.maximum(c_ref, 0.0) if relu else c_ref
    z_ref = y_ref * bs.astype(np.float64) + bh.astype(np.float64)
    bound = np.abs(bs) * tol_c + 4 * gu.U * (np.abs(y_ref * bs) + np.abs(bh)) + 1e-30
    if obf16:
        bound = bound + 2.0 ** -8 * np.abs(z_ref)
    ld = (N + 7) // 8 * 8 + 8
    out = torch.full((M, ld), float("nan"), device="cuda", dtype=torch.bfloat16 if obf16 else torch.float32)
    ep = hb.make_epilogue(hb.ACT_RELU if relu else hb.ACT_NONE, torch.from_numpy(bs).cuda() if affine else None,
                          torch.from_numpy(bh).cuda() if affine else None, out=out[:, :N])
    hb.gemm_fused(A, W, ep, _gemm_ws(hb, A, W))
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isnan(got[:, N:]).all()                  # nothing written beyond column N
    err = np.abs(got[:, :N] - z_ref)
    assert (err <= bound).all(), float((err / bound).max())


def test_gemm_fused_packed_output_after_relu_from_dense_activations(hb):
    """HBWN product -> ReLU -> affine map -> rows binarized for the next layer, in the tensor-core HBWN kernel."""
    gu = _gu()
    M, N, K, bw, bn = 200, 136, 576, 32, 32
    _, a = inputs.as_bf16(inputs.normal((M, K), 9801))
    w = inputs.he_normal(N, K, 9802)
    W, dw, sw = gu.oracle_operand(w, bw)
    A = hb.wrap_dense(torch.from_numpy(a).cuda().to(torch.bfloat16))
    c_ref, absref = oracle.hbwn_from_quantized(a, dw, sw, bw)
    rng = np.random.default_rng(5)
    bs = rng.uniform(0.5, 2.0, N).astype(np.float32)
    bh = (-0.4 + 0.2 * rng.standard_normal(N)).astype(np.float32)       # shifts the rectified values around zero
    y_ref = np.maximum(c_ref, 0.0)
    z_ref = y_ref * bs.astype(np.float64) + bh.astype(np.float64)
    band = np.abs(bs) * _hbwn_rtol(gu, K, bw, True) * absref + 4 * gu.U * (np.abs(y_ref * bs) + np.abs(bh)) + 1e-30
    nxt = hb.alloc_operand(M, N, bn, hb.F32)
    nxt.bits.fill_(-1)
    nxt.scales.fill_(float("nan"))
    ep = hb.make_epilogue(hb.ACT_RELU, torch.from_numpy(bs).cuda(), torch.from_numpy(bh).cuda(), nxt=nxt)
    hb.gemm_fused(A, W, ep, _gemm_ws(hb, A, W))
    torch.cuda.synchronize()
    gu.check_next_operand(nxt, z_ref, band, bn, False)


def _nhwc_to_nchw(z, B, Ho, Wo):
    return np.ascontiguousarray(z.reshape(B, Ho, Wo, -1).transpose(0, 3, 1, 2))


@pytest.mark.parametrize("B,C,H,F1,F2", [(3, 64, 12, 64, 72), (2, 128, 7, 128, 40), (7, 64, 54, 64, 48)])
def test_two_dense_activation_convolutions_chained_through_the_epilogue(hb, B, C, H, F1, F2):
    """Layer 1: convolution (bf16 activations x Hadamard-binary weights) -> ReLU -> the next block's batch-norm map ->
    NHWC bf16, written by the epilogue.  Layer 2 reads that tensor as it is (HBMM_CONV_INPUT_NHWC).  Layer 1 is held to
    the composed oracle (product tolerance carried through the map, half a bf16 ulp); layer 2 to the oracle's
    convolution of exactly the values layer 1 stored."""
    gu = _gu()
    s1 = inputs.ConvShape("l1", B, C, H, H, F1)
    x = inputs.conv_activation(s1, 9900 + C, signed=True)
    _, xb = inputs.as_bf16(x)
    w1 = inputs.he_normal(F1, C * 9, 9901)
    w2 = inputs.he_normal(F2, F1 * 9, 9902)
    W1 = hb.quantize(torch.from_numpy(w1).cuda(), hb.alloc_operand(F1, C * 9, 32))
    W2 = hb.quantize(torch.from_numpy(w2).cuda(), hb.alloc_operand(F2, F1 * 9, 32))
    rng = np.random.default_rng(C)
    bs = rng.uniform(0.5, 2.0, F1).astype(np.float32)
    bh = (0.2 * rng.standard_normal(F1)).astype(np.float32)
    g1 = hb.make_geom(B, C, H, H, 3, 3, (1, 1), (1, 1))
    g2 = hb.make_geom(B, F1, H, H, 3, 3, (1, 1), (1, 1))
    ws1 = torch.empty(hb.conv_workspace_bytes(g1, 1, hb.F32, W1), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(hb.conv_workspace_bytes(g2, 1, hb.F32, W2), dtype=torch.uint8, device="cuda")
    M = B * H * H
    z = torch.full((M, F1), float("nan"), device="cuda", dtype=torch.bfloat16)
    ep = hb.make_epilogue(hb.ACT_RELU, torch.from_numpy(bs).cuda(), torch.from_numpy(bh).cuda(), out=z)
    hb.conv_im2col_fused(torch.from_numpy(xb).cuda().to(torch.bfloat16), g1, 1, hb.F32, W1, ep, ws1)
    out = torch.full((M, (F2 + 3) // 4 * 4), float("nan"), device="cuda")
    hb.conv_im2col(z.view(B, H, H, F1), g2, 1, hb.F32, W2, out, ws2, flags=hb.CONV_INPUT_NHWC)
    torch.cuda.synchronize()
    # layer 1
    c1, abs1 = oracle.conv_im2col(xb, w1, 3, 3, (1, 1), (1, 1), 1, 32)
    y1 = np.maximum(c1, 0.0)
    z_ref = y1 * bs.astype(np.float64) + bh.astype(np.float64)
    z_gpu = z.float().cpu().numpy()
    bound = np.abs(bs) * _hbwn_rtol(gu, C * 9, 32, True) * abs1 + 4 * gu.U * (np.abs(y1 * bs) + np.abs(bh)) + 2.0 ** -8 * np.abs(z_ref) + 1e-30
    assert (np.abs(z_gpu - z_ref) <= bound).all()
    # layer 2 from the stored values
    c2, abs2 = oracle.conv_im2col(_nhwc_to_nchw(z_gpu, B, H, H), w2, 3, 3, (1, 1), (1, 1), 1, 32)
    gu.assert_close_rel_absref(out.cpu().numpy()[:, :F2], c2, abs2, _hbwn_rtol(gu, F1 * 9, 32, True), "layer 2")


def test_packed_convolution_feeding_a_pointwise_layer_through_the_epilogue(hb):
    """Layer 1: 3 x 3 convolution as HBMM (beta_a = beta_w = 32) -> ReLU -> batch-norm map -> rows binarized along the
    output channels by the epilogue (the fp32 product never stored).  Layer 2: a 1 x 1 convolution = hbmm_gemm on that
    packed operand.  Layer 1 is checked like hbmm_gemm_binarize_next; layer 2 against the oracle's product of the
    operand layer 1 actually wrote."""
    gu = _gu()
    B, C, H, F1, F2, bn = 2, 64, 12, 128, 96, 32
    s1 = inputs.ConvShape("l1", B, C, H, H, F1)
    x = inputs.conv_activation(s1, 9950, signed=True)
    w1 = inputs.he_normal(F1, C * 9, 9951)
    w2 = inputs.he_normal(F2, F1, 9952)
    W1, dw1, sw1 = gu.oracle_operand(w1, 32)
    W2, dw2, sw2 = gu.oracle_operand(w2, bn)
    rng = np.random.default_rng(11)
    bs = rng.uniform(0.5, 2.0, F1).astype(np.float32)
    bh = (-0.3 + 0.2 * rng.standard_normal(F1)).astype(np.float32)
    g1 = hb.make_geom(B, C, H, H, 3, 3, (1, 1), (1, 1))
    ws1 = torch.empty(hb.conv_workspace_bytes(g1, 32, hb.F32, W1), dtype=torch.uint8, device="cuda")
    M = B * H * H
    nxt = hb.alloc_operand(M, F1, bn, hb.F32)
    nxt.bits.fill_(-1)
    nxt.scales.fill_(float("nan"))
    ep = hb.make_epilogue(hb.ACT_RELU, torch.from_numpy(bs).cuda(), torch.from_numpy(bh).cuda(), nxt=nxt)
    hb.conv_im2col_fused(torch.from_numpy(x).cuda(), g1, 32, hb.F32, W1, ep, ws1)
    out = torch.full((M, F2), float("nan"), device="cuda")
    hb.gemm(nxt, W2, out, _gemm_ws(hb, nxt, W2))
    torch.cuda.synchronize()
    rows = oracle.im2col(x, 3, 3, (1, 1), (1, 1))
    da, sa = oracle.quantize(rows, 32)
    c1, abs1 = oracle.hbmm_from_quantized(da, sa, 32, dw1, sw1, 32)
    fine = gu.elementwise_magnitude(da, 32, dw1, 32, C * 9)
    y1 = np.maximum(c1, 0.0)
    z_ref = y1 * bs.astype(np.float64) + bh.astype(np.float64)
    band = np.abs(bs) * (RTOL * abs1 + gu.FOLDED_FLOOR_ULPS * gu.U * fine) + 4 * gu.U * (np.abs(y1 * bs) + np.abs(bh)) + 1e-30
    gu.check_next_operand(nxt, z_ref, band, bn, False)
    # layer 2 from what was stored
    sg = oracle.unpack(gu.host_bits(nxt.bits), F1)
    dg = nxt.scales.cpu().numpy().astype(np.float64)[:, : F1 // bn]
    c2, abs2 = oracle.hbmm_from_quantized(dg, sg, bn, dw2, sw2, bn)
    gu.assert_close_rel_absref(out.cpu().numpy(), c2, abs2, RTOL, "pointwise layer",
                               gu.elementwise_magnitude(dg, bn, dw2, bn, F1))


@pytest.mark.parametrize("beta_a,xbf16", [(32, False), (1, True)])
def test_back_to_back_calls_on_one_workspace_do_not_disturb_each_other(hb, beta_a, xbf16):
    """The kernels of a convolution call are launched so that their set-up may overlap the tail of the kernel
    before them.  A second call that reuses the workspace right behind the first must still wait for it:
    the results of a burst of calls equal those of calls separated by device synchronisation."""
    shape = inputs.ConvShape("t", 8, 64, 28, 28, 72, 3, 3, 1, 1)
    K = 64 * 9
    Wop = hb.quantize(torch.from_numpy(inputs.he_normal(72, K, 611)).cuda(), hb.alloc_operand(72, K, 32))
    geom = hb.make_geom(8, 64, 28, 28, 3, 3, (1, 1), (1, 1))
    ws = torch.empty(hb.conv_workspace_bytes(geom, beta_a, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    xs = []
    for seed in range(4):
        x = torch.from_numpy(inputs.conv_activation(shape, 620 + seed, signed=True)).cuda()
        xs.append(x.to(torch.bfloat16) if xbf16 else x)
    calm = []
    for x in xs:
        out = torch.empty((shape.M, 72), device="cuda")
        hb.conv_im2col(x, geom, beta_a, hb.F32, Wop, out, ws)
        torch.cuda.synchronize()
        calm.append(out)
    burst = [torch.empty((shape.M, 72), device="cuda") for _ in xs]
    for _ in range(3):
        for x, out in zip(xs, burst):
            hb.conv_im2col(x, geom, beta_a, hb.F32, Wop, out, ws)
    torch.cuda.synchronize()
    for a, b in zip(calm, burst):
        assert torch.equal(a, b)


def test_two_products_on_two_streams_equal_their_serial_results(hb):
    """HBMM and HBWN calls that share no buffer may run on different streams at the same time (the schedule
    the benchmark times): the library keeps no scratch of its own between them, so the results are those of
    the calls made one after the other."""
    shapes = [inputs.ConvShape("a", 16, 64, 28, 28, 128, 3, 3, 1, 1), inputs.ConvShape("b", 16, 128, 14, 14, 256, 3, 3, 1, 1)]
    jobs = []
    for i, s in enumerate(shapes):
        K = s.C * 9
        Wop = hb.quantize(torch.from_numpy(inputs.he_normal(s.N, K, 700 + i)).cuda(), hb.alloc_operand(s.N, K, 32))
        geom = hb.make_geom(s.B, s.C, s.H, s.W, 3, 3, (1, 1), (1, 1))
        x = torch.from_numpy(inputs.conv_activation(s, 710 + i, signed=True)).cuda()
        for beta_a, xin in ((32, x), (1, x.to(torch.bfloat16))):
            ws = torch.empty(hb.conv_workspace_bytes(geom, beta_a, hb.F32, Wop), dtype=torch.uint8, device="cuda")
            jobs.append(dict(x=xin, geom=geom, beta_a=beta_a, W=Wop, ws=ws, M=s.M, N=s.N))
    calm = []
    for j in jobs:
        out = torch.empty((j["M"], j["N"]), device="cuda")
        hb.conv_im2col(j["x"], j["geom"], j["beta_a"], hb.F32, j["W"], out, j["ws"])
        torch.cuda.synchronize()
        calm.append(out)
    outs = [torch.empty_like(c) for c in calm]
    streams = {32: torch.cuda.Stream(), 1: torch.cuda.Stream()}
    torch.cuda.synchronize()
    for _ in range(5):
        for j, out in zip(jobs, outs):
            with torch.cuda.stream(streams[j["beta_a"]]):
                hb.conv_im2col(j["x"], j["geom"], j["beta_a"], hb.F32, j["W"], out, j["ws"])
    torch.cuda.synchronize()
    assert hb.last_device_error() == 0
    for a, b in zip(calm, outs):
        assert torch.equal(a, b)


# ------------------------------------------------------------------ Eq. 3 as printed: the binarized tensor written out dense
DENSE_CASES = [
    # rows, K, beta, row padding
    (64, 576, 2, 0), (33, 1152, 4, 0), (20, 256, 8, 0), (17, 512, 16, 0), (130, 576, 32, 0), (9, 1024, 128, 0), (40, 100, 1, 0),
    (7, 333, 4, 0),      # ragged K: tail group of one element -> general kernel
    (1000, 56, 8, 0),    # a 56-wide map line, 7 groups of 8
    (1000, 28, 16, 0),   # tail group of 12
    (300, 7, 4, 0),      # conv5-sized map line
    (5, 45, 7, 3),       # odd everything, padded rows
    (16, 128, 256, 0),   # beta > K
]


@pytest.mark.parametrize("rows,K,beta,pad", DENSE_CASES)
def test_binarize_dense_matches_oracle(hb, rows, K, beta, pad):
    gu = _gu()
    x = inputs.normal((rows, K), 9300 + rows + K)
    x[0, :4] = [1.0, -1.0, 0.0, -0.0]                       # Sign(+-0) = +1
    be = gu.eff_beta(beta, K)
    delta, sign = oracle.quantize(x, be)
    ref = oracle.dequant(delta, sign, be)
    xd = torch.zeros((rows, K + pad)); xd[:, :K] = torch.from_numpy(x)
    xg = xd.cuda()[:, :K]
    out = torch.full((rows, K + pad), float("nan"), device="cuda")
    hb.binarize_dense(xg, beta, hb.F32, out[:, :K])
    got = out.cpu().numpy()
    assert np.isnan(got[:, K:]).all()
    got = got[:, :K]
    assert np.array_equal(np.signbit(got), sign < 0)                          # signs are bit-exact, zeros positive
    # the scale is an fp32 tree over at most beta non-negative terms and one multiply
    tol = (int(np.ceil(np.log2(max(be, 2)))) + int(np.ceil(be / 32)) + 2) * gu.U
    assert (np.abs(np.abs(got.astype(np.float64)) - np.abs(ref)) <= tol * np.abs(ref)).all()
    # bf16 output: the same fp32 values rounded to nearest even
    outb = torch.full((rows, K + pad), float("nan"), device="cuda", dtype=torch.bfloat16)
    hb.binarize_dense(xg, beta, hb.BF16, outb[:, :K])
    assert torch.isnan(outb[:, K:]).all()
    assert torch.equal(outb[:, :K], out[:, :K].to(torch.bfloat16))


MAP_CONV_CASES = [
    # B, C, H, W, filters, stride, beta_a, beta_w
    (4, 64, 28, 28, 72, 1, 4, 32),
    (2, 64, 56, 56, 64, 1, 8, 32),
    (3, 128, 14, 14, 130, 2, 16, 64),      # tail group of 14 along the map line, strided
    (2, 32, 9, 11, 40, 1, 3, 32),          # odd width, groups of three
]


@pytest.mark.parametrize("B,C,H,W,F,st,ba,bw", MAP_CONV_CASES)
def test_convolution_of_the_map_binarized_as_in_eq3(hb, B, C, H, W, F, st, ba, bw):
    """Eq. 3 groups the activations along the rows of the map, before the gather.  The path: hbmm_binarize_dense
    on the map (bf16 out), then hbmm_conv_im2col with beta_a = 1 on it.  The activation values are A~ rounded
    to bf16 (2^-9 relative, as for any bf16 activation of the HBWN path); the rest is the HBWN tolerance."""
    gu = _gu()
    shape = inputs.ConvShape("t", B, C, H, W, F, 3, 3, st, 1)
    K = C * 9
    x = inputs.conv_activation(shape, 9400 + C + W, signed=True)
    w = inputs.he_normal(F, K, 9500 + F)
    ref, absref = oracle.conv_map_binarized(x, w, 3, 3, (st, st), (1, 1), ba, bw)
    Wop = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(F, K, bw))
    geom = hb.make_geom(B, C, H, W, 3, 3, (st, st), (1, 1))
    at = hb.binarize_map(torch.from_numpy(x).cuda(), ba, hb.BF16)
    ws = torch.empty(hb.conv_workspace_bytes(geom, 1, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    out = torch.full((shape.M, (F + 3) // 4 * 4), float("nan"), device="cuda")
    hb.conv_im2col(at, geom, 1, hb.F32, Wop, out, ws)
    torch.cuda.synchronize()
    assert hb.last_device_error() == 0
    rtol = 2.0 ** -9 + _hbwn_rtol(gu, K, bw, True)
    gu.assert_close_rel_absref(out.cpu().numpy()[:, :F], ref, absref, rtol, "eq3 conv")
    # and the map itself against the oracle: signs exact, magnitudes to bf16 rounding
    a64 = oracle.binarize_map(x, ba)
    ag = at.float().cpu().numpy()
    assert np.array_equal(np.signbit(ag), a64 < 0)
    assert (np.abs(np.abs(ag) - np.abs(a64)) <= 2.0 ** -8 * np.abs(a64)).all()
