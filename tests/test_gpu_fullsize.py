"""GPU parity at full workload sizes, in the launch configuration the benchmark times: the library runs
the whole problem, the CPU oracle recomputes sampled output rows one by one from the same seeded
inputs (whole images for the convolutions, scattered rows for the matrix products)."""
import functools

import numpy as np
import pytest
import torch

import oracle
from paper_1905_10759_b200 import inputs

pytestmark = pytest.mark.gpu

RTOL = 1e-5
BETA = 32


@pytest.fixture(scope="module")
def hb():
    from paper_1905_10759_b200 import hbmm
    yield hbmm
    assert hbmm.last_device_error() == 0


def _gu():
    import gpu_util
    return gpu_util


def _sample_rows(M, n, seed):
    """First and last rows, rows around 128-row tile borders, and random ones."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 129, M // 2, M - 129, M - 128, M - 2, M - 1]
    rows = set(r for r in fixed if 0 <= r < M)
    while len(rows) < min(n, M):
        rows.add(int(rng.integers(0, M)))
    return np.array(sorted(rows))


# ------------------------------------------------------------------ the benchmark's convolutions, batch 64
@pytest.mark.parametrize("li", [0, 1, 2, 3])
@pytest.mark.parametrize("signed", [False, True])
def test_resnet_conv_hbmm_full_batch(hb, li, signed):
    gu = _gu()
    s = inputs.resnet18_convs(64)[li]
    x = inputs.conv_activation(s, inputs.SEEDS["resnet_hbmm"][0] + li, signed=signed)
    w = inputs.he_normal(s.N, s.K, inputs.SEEDS["resnet_hbmm"][1] + li)
    Wop = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(s.N, s.K, BETA, hb.F32))
    geom = hb.make_geom(s.B, s.C, s.H, s.W, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
    ws = torch.empty(hb.conv_workspace_bytes(geom, BETA, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    C = torch.empty((s.M, s.N), device="cuda")
    hb.conv_im2col(torch.from_numpy(x).cuda(), geom, BETA, hb.F32, Wop, C, ws)
    torch.cuda.synchronize()
    _, _, lw, ls = hb.operand_bytes(s.M, s.K, BETA, hb.F32)
    bits = ws[: s.M * lw * 4].view(torch.int32).reshape(s.M, lw)
    per_image = s.M // s.B
    for b in (0, s.B // 2, s.B - 1):                       # whole images: first, middle, last
        rows = oracle.im2col(x[b:b + 1], s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
        da, sa = oracle.quantize(rows, BETA)
        dw, sw = oracle.quantize(w, BETA)
        c_ref, absref = oracle.hbmm_from_quantized(oracle.round_scales(da, "f32"), sa, BETA, oracle.round_scales(dw, "f32"), sw, BETA)
        lo = b * per_image
        assert np.array_equal(gu.host_bits(bits[lo: lo + per_image]), oracle.pack(sa, lw)), "packed activations of image %d" % b
        gu.assert_close_rel_absref(C[lo: lo + per_image].cpu().numpy(), c_ref, absref, RTOL, "%s image %d" % (s.name, b))


@pytest.mark.parametrize("li,ba,bw", [(0, 4, 4), (1, 2, 16), (2, 16, 16), (3, 64, 64), (1, 128, 32)])
def test_resnet_conv_hbmm_full_batch_at_other_group_sizes(hb, li, ba, bw):
    """The paper's own group sizes (Section 5: beta_a / beta_w of 2 .. 16) and groups of several words through the
    convolution entry at batch 64: packed activations bit for bit, their scales to the quantizer's bound, the product
    to 1e-5 R, on whole images."""
    gu = _gu()
    s = inputs.resnet18_convs(64)[li]
    x = inputs.conv_activation(s, inputs.SEEDS["resnet_hbmm"][0] + 70 + li, signed=True)
    w = inputs.he_normal(s.N, s.K, inputs.SEEDS["resnet_hbmm"][1] + 70 + li)
    Wop = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(s.N, s.K, bw, hb.F32))
    geom = hb.make_geom(s.B, s.C, s.H, s.W, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
    ws = torch.empty(hb.conv_workspace_bytes(geom, ba, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    C = torch.empty((s.M, s.N), device="cuda")
    hb.conv_im2col(torch.from_numpy(x).cuda(), geom, ba, hb.F32, Wop, C, ws)
    torch.cuda.synchronize()
    assert hb.last_device_error() == 0
    _, _, lw, ls = hb.operand_bytes(s.M, s.K, ba, hb.F32)
    bits_bytes = (s.M * lw * 4 + 255) // 256 * 256          # the scales follow the packed words on a 256-byte boundary
    bits = ws[: s.M * lw * 4].view(torch.int32).reshape(s.M, lw)
    scales = ws[bits_bytes: bits_bytes + s.M * ls * 4].view(torch.float32).reshape(s.M, ls)
    G = oracle.n_groups(s.K, ba)
    per_image = s.M // s.B
    dw, sw = oracle.quantize(w, bw)
    for b in (0, s.B - 1):
        rows = oracle.im2col(x[b:b + 1], s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
        da, sa = oracle.quantize(rows, ba)
        lo = b * per_image
        assert np.array_equal(gu.host_bits(bits[lo: lo + per_image]), oracle.pack(sa, lw)), "packed activations of image %d" % b
        sg = scales[lo: lo + per_image].cpu().numpy().astype(np.float64)
        assert np.all(sg[:, G:] == 0.0)
        assert np.all(np.abs(sg[:, :G] - da) <= 12 * gu.U * da + 1e-30)
        c_ref, absref = oracle.hbmm_from_quantized(sg[:, :G], sa, ba, oracle.round_scales(dw, "f32"), sw, bw)
        fine = gu.elementwise_magnitude(sg[:, :G], ba, dw, bw, s.K)
        gu.assert_close_rel_absref(C[lo: lo + per_image].cpu().numpy(), c_ref, absref, RTOL, "%s image %d beta %d/%d" % (s.name, b, ba, bw), fine)


@pytest.mark.parametrize("li", [0, 1, 2, 3])
def test_resnet_conv_hbwn_full_batch(hb, li):
    gu = _gu()
    s = inputs.resnet18_convs(64)[li]
    x = inputs.conv_activation(s, inputs.SEEDS["resnet_hbwn"][0] + li, signed=(li % 2 == 1))
    xb_bits, xb = inputs.as_bf16(x)
    w = inputs.he_normal(s.N, s.K, inputs.SEEDS["resnet_hbmm"][1] + li)
    Wop = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(s.N, s.K, BETA, hb.F32))
    geom = hb.make_geom(s.B, s.C, s.H, s.W, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
    ws = torch.empty(hb.conv_workspace_bytes(geom, 1, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    C = torch.empty((s.M, s.N), device="cuda")
    xd = torch.from_numpy(xb_bits.view(np.int16)).view(torch.bfloat16).cuda()
    hb.conv_im2col(xd, geom, 1, hb.F32, Wop, C, ws)
    torch.cuda.synchronize()
    dw, sw = oracle.quantize(w, BETA)
    dw = oracle.round_scales(dw, "f32")
    G = s.K // BETA
    rtol = (BETA + G + 4) * 2 * gu.U + 2.0 ** -18     # fp32 sums + the weight scale carried by two bf16 pieces
    per_image = s.M // s.B
    for b in (0, s.B // 2, s.B - 1):
        rows = oracle.im2col(xb[b:b + 1], s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
        c_ref, absref = oracle.hbwn_from_quantized(rows, dw, sw, BETA)
        lo = b * per_image
        gu.assert_close_rel_absref(C[lo: lo + per_image].cpu().numpy(), c_ref, absref, rtol, "%s image %d" % (s.name, b))


# ------------------------------------------------------------------ square products and the FC stack
@functools.lru_cache(maxsize=1)
def _square_inputs(n):
    """Raw inputs of one square size, shared by its six (group size, scale storage) combinations."""
    return (inputs.normal((n, n), inputs.SEEDS["square_sweep"][0] + n // 4096),
            inputs.normal((n, n), inputs.SEEDS["square_sweep"][1] + n // 4096))


# the whole sweep of the square configuration: two sizes x three group sizes x two scale storage types
@pytest.mark.parametrize("sdt", [0, 1], ids=["f32scales", "bf16scales"])
@pytest.mark.parametrize("beta", [32, 64, 128])
@pytest.mark.parametrize("n", [4096, 8192])
def test_square_quantize_then_gemm_sampled_rows(hb, n, beta, sdt):
    gu = _gu()
    a, w = _square_inputs(n)
    A = hb.quantize(torch.from_numpy(a).cuda(), hb.alloc_operand(n, n, beta, sdt))
    W = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(n, n, beta, sdt))
    C = torch.empty((n, n), device="cuda")
    ws = torch.empty(max(hb.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
    hb.gemm(A, W, C, ws)
    torch.cuda.synchronize()
    rows = _sample_rows(n, 24, n + beta)
    # the oracle binarizes the same raw rows; stored scales are compared through the rounding the storage type applies
    name = "f32" if sdt == hb.F32 else "bf16"
    da, sa = oracle.quantize(a[rows], beta)
    dw, sw = oracle.quantize(w, beta)
    lw = A.bits.shape[1]
    assert np.array_equal(gu.host_bits(A.bits[torch.from_numpy(rows).cuda()]), oracle.pack(sa, lw))
    # products from the scales the GPU actually stored (isolates the contraction from the scale rounding)
    G = n // beta
    sa_gpu = A.scales[torch.from_numpy(rows).cuda()][:, :G].float().cpu().numpy().astype(np.float64)
    sw_gpu = W.scales[:, :G].float().cpu().numpy().astype(np.float64)
    tol_s = (int(np.ceil(np.log2(beta))) + 3) * gu.U + (2.0 ** -8 if name == "bf16" else 0.0)
    assert np.all(np.abs(sa_gpu - da) <= tol_s * da + 1e-30)
    c_ref, absref = oracle.hbmm_from_quantized(sa_gpu, sa, beta, sw_gpu, sw, beta)
    gu.assert_close_rel_absref(C[torch.from_numpy(rows).cuda()].cpu().numpy(), c_ref, absref, RTOL, "square %d" % n)


@pytest.mark.parametrize("batch", [1, 256])
def test_alexnet_fc_stack(hb, batch):
    gu = _gu()
    beta = 64
    for i, (K, N) in enumerate(inputs.ALEXNET_FC):
        a = inputs.normal((batch, K), inputs.SEEDS["alexnet_fc"][0] + i)
        w = inputs.he_normal(N, K, inputs.SEEDS["alexnet_fc"][1] + i)
        A, da, sa = gu.oracle_operand(a, beta)
        W, dw, sw = gu.oracle_operand(w, beta)
        ldc = (N + 3) // 4 * 4
        C = torch.empty((batch, ldc), device="cuda")
        ws = torch.empty(max(hb.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
        hb.gemm(A, W, C, ws)
        rows = _sample_rows(batch, 16, K + N)
        c_ref, absref = oracle.hbmm_from_quantized(da[rows], sa[rows], beta, dw, sw, beta)
        gu.assert_close_rel_absref(C[torch.from_numpy(rows).cuda()].cpu().numpy()[:, :N], c_ref, absref, RTOL,
                                   "fc %dx%d batch %d" % (K, N, batch))


@pytest.mark.parametrize("ba,bw", [(16, 16), (4, 4), (2, 16)])
def test_subword_groups_on_the_conv3_matrix_sampled_rows(hb, ba, bw):
    """The paper's own group sizes (Section 5: beta_a / beta_w = 2 .. 16, mixed) at a benchmark shape
    (M = 50176, N = 128, K = 1152), through hbmm_quantize and the automatic contraction path."""
    gu = _gu()
    M, N, K = 50176, 128, 1152
    a = inputs.normal((M, K), inputs.SEEDS["resnet_hbmm"][0] + 40 + ba)
    w = inputs.he_normal(N, K, inputs.SEEDS["resnet_hbmm"][1] + 40 + bw)
    A = hb.quantize(torch.from_numpy(a).cuda(), hb.alloc_operand(M, K, ba, hb.F32))
    W = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(N, K, bw, hb.F32))
    C = torch.empty((M, N), device="cuda")
    ws = torch.empty(max(hb.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
    hb.gemm(A, W, C, ws)
    torch.cuda.synchronize()
    rows = _sample_rows(M, 48, M + ba)
    rows_d = torch.from_numpy(rows).cuda()
    da, sa = oracle.quantize(a[rows], ba)
    dw, sw = oracle.quantize(w, bw)
    assert np.array_equal(gu.host_bits(A.bits[rows_d]), oracle.pack(sa, A.bits.shape[1]))
    # products from the scales the GPU stored (they are checked against the oracle's to their own bound)
    sa_gpu = A.scales[rows_d][:, : K // ba].float().cpu().numpy().astype(np.float64)
    sw_gpu = W.scales[:, : K // bw].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(sa_gpu - da) <= 8 * gu.U * da + 1e-30) and np.all(np.abs(sw_gpu - dw) <= 8 * gu.U * dw + 1e-30)
    c_ref, absref = oracle.hbmm_from_quantized(sa_gpu, sa, ba, sw_gpu, sw, bw)
    # no absolute floor: at this size no output's group dots all cancel, so 1e-5 R alone must hold
    gu.assert_close_rel_absref(C[rows_d].cpu().numpy(), c_ref, absref, RTOL, "conv3 matrix beta %d/%d" % (ba, bw))


# ------------------------------------------------------------------ Eq. 3 grouping (along map rows) at the benchmark's sizes
@pytest.mark.parametrize("li,beta_a", [(0, 8), (2, 2), (3, 4)])
def test_resnet_conv_of_map_binarized_activations_full_batch(hb, li, beta_a):
    """hbmm_binarize_dense on the whole batch-64 map (bf16 out), then the HBWN convolution; the oracle redoes
    three whole images.  conv5_x with beta_a = 4: lines of 7, a tail run of 3 in every line."""
    gu = _gu()
    s = inputs.resnet18_convs(64)[li]
    x = inputs.conv_activation(s, inputs.SEEDS["resnet_hbwn"][0] + 40 + li, signed=True)
    w = inputs.he_normal(s.N, s.K, inputs.SEEDS["resnet_hbmm"][1] + li)
    Wop = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(s.N, s.K, BETA, hb.F32))
    geom = hb.make_geom(s.B, s.C, s.H, s.W, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad))
    ws = torch.empty(hb.conv_workspace_bytes(geom, 1, hb.F32, Wop), dtype=torch.uint8, device="cuda")
    C = torch.empty((s.M, s.N), device="cuda")
    at = hb.binarize_map(torch.from_numpy(x).cuda(), beta_a, hb.BF16)
    hb.conv_im2col(at, geom, 1, hb.F32, Wop, C, ws)
    torch.cuda.synchronize()
    G = s.K // BETA
    rtol = 2.0 ** -9 + (BETA + G + 4) * 2 * gu.U + 2.0 ** -18     # A~ rounded to bf16; fp32 sums; two-piece weight scales
    per_image = s.M // s.B
    for b in (0, s.B // 2, s.B - 1):
        a64 = oracle.binarize_map(x[b:b + 1], beta_a)
        ag = at[b:b + 1].float().cpu().numpy()
        assert np.array_equal(np.signbit(ag), a64 < 0)
        assert (np.abs(np.abs(ag) - np.abs(a64)) <= 2.0 ** -8 * np.abs(a64)).all()
        c_ref, absref = oracle.conv_map_binarized(x[b:b + 1], w, s.kh, s.kw, (s.stride, s.stride), (s.pad, s.pad), beta_a, BETA)
        lo = b * per_image
        gu.assert_close_rel_absref(C[lo: lo + per_image].cpu().numpy(), c_ref, absref, rtol, "%s image %d" % (s.name, b))


# ------------------------------------------------------------------ two layers chained through the epilogue, batch 64
def test_conv3_chain_through_the_epilogue_full_batch(hb):
    """conv3_x -> ReLU -> the next block's batch-norm map -> NHWC bf16 (all in the first contraction's epilogue), then a
    second conv3_x that reads that tensor directly (HBMM_CONV_INPUT_NHWC).  Three whole images are redone by the
    oracle: layer 1 from the raw input, layer 2 from exactly the values layer 1 stored."""
    gu = _gu()
    s = inputs.resnet18_convs(64)[1]
    B, C, H, N = s.B, s.C, s.H, s.N
    x = inputs.conv_activation(s, inputs.SEEDS["resnet_hbwn"][0] + 70, signed=True)
    xb_bits, xb = inputs.as_bf16(x)
    w1 = inputs.he_normal(N, s.K, inputs.SEEDS["resnet_hbmm"][1] + 70)
    w2 = inputs.he_normal(N, N * 9, inputs.SEEDS["resnet_hbmm"][1] + 71)
    W1 = hb.quantize(torch.from_numpy(w1).cuda(), hb.alloc_operand(N, s.K, BETA, hb.F32))
    W2 = hb.quantize(torch.from_numpy(w2).cuda(), hb.alloc_operand(N, N * 9, BETA, hb.F32))
    rng = np.random.default_rng(70)
    bs = rng.uniform(0.5, 2.0, N).astype(np.float32)
    bh = (0.2 * rng.standard_normal(N)).astype(np.float32)
    geom = hb.make_geom(B, C, H, H, 3, 3, (1, 1), (1, 1))
    ws1 = torch.empty(hb.conv_workspace_bytes(geom, 1, hb.F32, W1), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(hb.conv_workspace_bytes(geom, 1, hb.F32, W2), dtype=torch.uint8, device="cuda")
    z = torch.empty((s.M, N), device="cuda", dtype=torch.bfloat16)
    ep = hb.make_epilogue(hb.ACT_RELU, torch.from_numpy(bs).cuda(), torch.from_numpy(bh).cuda(), out=z)
    xd = torch.from_numpy(xb_bits.view(np.int16)).view(torch.bfloat16).cuda()
    hb.conv_im2col_fused(xd, geom, 1, hb.F32, W1, ep, ws1)
    out = torch.empty((s.M, N), device="cuda")
    hb.conv_im2col(z.view(B, H, H, N), geom, 1, hb.F32, W2, out, ws2, flags=hb.CONV_INPUT_NHWC)
    torch.cuda.synchronize()
    G = s.K // BETA
    rtol = (BETA + G + 4) * 2 * gu.U + 2.0 ** -18
    per_image = s.M // B
    for b in (0, B // 2, B - 1):
        lo = b * per_image
        c1, abs1 = oracle.conv_im2col(xb[b:b + 1], w1, 3, 3, (1, 1), (1, 1), 1, BETA)
        y1 = np.maximum(c1, 0.0)
        z_ref = y1 * bs.astype(np.float64) + bh.astype(np.float64)
        z_gpu = z[lo: lo + per_image].float().cpu().numpy()
        bound = np.abs(bs) * rtol * abs1 + 4 * gu.U * (np.abs(y1 * bs) + np.abs(bh)) + 2.0 ** -8 * np.abs(z_ref) + 1e-30
        assert (np.abs(z_gpu - z_ref) <= bound).all(), "layer 1, image %d" % b
        z_img = np.ascontiguousarray(z_gpu.reshape(1, H, H, N).transpose(0, 3, 1, 2))
        c2, abs2 = oracle.conv_im2col(z_img, w2, 3, 3, (1, 1), (1, 1), 1, BETA)
        gu.assert_close_rel_absref(out[lo: lo + per_image].cpu().numpy(), c2, abs2, rtol, "layer 2, image %d" % b)
