"""Integer exactness at the full sizes of the five workload configurations.

With every group scale equal to one, Eq. 7 collapses to the signed dot product of the two sign rows,
C[m,n] = K - 2 popcount(a xor w): a small integer that fp32 holds exactly (|C| <= K < 2^24).  Every
contraction path must therefore reproduce it BIT FOR BIT, whatever order it sums in.  The reference is
formed here on the host from randomly drawn packed words -- numpy bit unpacking and a matrix product of
+-1 values (exact in float32: every partial sum is an integer below 2^24) -- by neither the library nor
the checker under oracle/.  Sampled rows are compared for the large shapes.  The integer term of Eq. 7 on
its own (hbmm_gemm_partials) is checked against the checker's multiply-add partials on sampled rows of a
full-size operand the library binarized itself.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_10759_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_1905_10759_b200 import hbmm
    yield hbmm
    assert hbmm.last_device_error() == 0


def _gu():
    import gpu_util
    return gpu_util


def _rows(M, n, seed):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 129, M // 2, M - 129, M - 128, M - 2, M - 1]
    rows = set(r for r in fixed if 0 <= r < M)
    while len(rows) < min(n, M):
        rows.add(int(rng.integers(0, M)))
    return np.array(sorted(rows))


def _unit_operand(hb, gu, rows, K, beta, seed):
    _, _, lw, ls = hb.operand_bytes(rows, K, beta, hb.F32)
    words = gu.random_sign_words(rows, K, lw, seed)
    G = oracle.n_groups(K, beta)
    scales = torch.zeros((rows, ls), device="cuda")
    scales[:, :G] = 1.0
    return hb.wrap_packed(gu.dev_bits(words), scales, K, beta), words


_conv = {s.name: (s.M, s.N, s.K) for s in inputs.resnet18_convs(64)}
UNIT_CASES = [
    # name, M, N, K, beta
    ("square256", 256, 256, 256, 32),
    ("square4096_beta32", 4096, 4096, 4096, 32),
    ("square4096_beta128", 4096, 4096, 4096, 128),          # also the legacy b1 tensor instruction
    ("square8192_beta64", 8192, 8192, 8192, 64),
    ("conv2_x", *_conv["conv2_x"], 32),
    ("conv3_x", *_conv["conv3_x"], 32),
    ("conv4_x", *_conv["conv4_x"], 32),
    ("conv5_x", *_conv["conv5_x"], 32),
    ("conv3_x_beta128", *_conv["conv3_x"], 128),            # b1 path at a convolution shape (1152 = 9 x 128)
    ("fc6_b256", 256, 4096, 9216, 64), ("fc7_b256", 256, 4096, 4096, 64), ("fc8_b256", 256, 1000, 4096, 64),
    ("fc6_b1", 1, 4096, 9216, 64), ("fc7_b1", 1, 4096, 4096, 64), ("fc8_b1", 1, 1000, 4096, 64),
]


@pytest.mark.parametrize("name,M,N,K,beta", UNIT_CASES, ids=[c[0] for c in UNIT_CASES])
def test_unit_scales_are_exact_integers_on_every_path_at_full_size(hb, name, M, N, K, beta):
    gu = _gu()
    A, a_words = _unit_operand(hb, gu, M, K, beta, 31000 + M + K)
    W, w_words = _unit_operand(hb, gu, N, K, beta, 32000 + N + K)
    rows = _rows(M, 32, M + N)
    ref = gu.signs_of_words(a_words[rows], K) @ gu.signs_of_words(w_words, K).T      # exact integers in float32
    assert np.array_equal(ref, np.rint(ref)) and np.abs(ref).max() <= K
    ws = torch.empty(max(hb.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
    rows_d = torch.from_numpy(rows).cuda()
    ldc = (N + 3) // 4 * 4
    must_run = gu.expected_paths(K, beta, beta)
    for path in (hb.PATH_POPC, hb.PATH_B1MMA, hb.PATH_TENSOR, hb.PATH_FOLDED, hb.PATH_AUTO):
        C = torch.full((M, ldc), float("nan"), device="cuda")
        if path not in must_run:
            with pytest.raises(hb.HbmmError) as e:
                hb.gemm_ex(A, W, C, path, ws)
            assert e.value.status == hb.ERR_UNSUPPORTED
            continue
        hb.gemm_ex(A, W, C, path, ws)
        got = C[rows_d][:, :N].cpu().numpy()
        assert np.array_equal(got, ref), "%s path %d: %d outputs differ" % (name, path, int((got != ref).sum()))
        # the rest of the matrix: finite integers of the right parity (K even => every dot is even)
        whole = C[:, :N]
        assert bool(torch.isfinite(whole).all()) and bool((whole == whole.round()).all())
        assert bool((whole.abs() <= K).all()) and bool(((whole.to(torch.int64) - K) % 2 == 0).all())


@pytest.mark.parametrize("li", [0, 1, 2, 3])
def test_hbwn_unit_scales_integer_activations_are_exact_at_the_conv_shapes(hb, li):
    """HBWN analogue: weight scales all one and small-integer bf16 activations make every output an exact
    integer (|C| <= 8 K < 2^24), so every dense x packed path must agree bit for bit with the host product."""
    gu = _gu()
    s = inputs.resnet18_convs(64)[li]
    M, N, K = s.M, s.N, s.K
    rng = np.random.default_rng(33000 + li)
    a = rng.integers(-8, 9, size=(M, K), dtype=np.int8)
    W, w_words = _unit_operand(hb, gu, N, K, 32, 34000 + li)
    A = hb.wrap_dense(torch.from_numpy(a).cuda().to(torch.bfloat16))
    rows = _rows(M, 32, M + li)
    ref = a[rows].astype(np.float32) @ gu.signs_of_words(w_words, K).T
    assert np.abs(ref).max() < 2 ** 24
    ws = torch.empty(max(hb.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
    rows_d = torch.from_numpy(rows).cuda()
    for path, wsp in ((hb.PATH_AUTO, ws), (hb.PATH_TENSOR, ws), (hb.PATH_FOLDED, ws), (hb.PATH_B1MMA, None), (hb.PATH_POPC, None)):
        C = torch.full((M, N), float("nan"), device="cuda")
        hb.gemm_ex(A, W, C, path, wsp)
        got = C[rows_d].cpu().numpy()
        assert np.array_equal(got, ref), "%s path %d: %d outputs differ" % (s.name, path, int((got != ref).sum()))
        assert bool((C == C.round()).all())


@pytest.mark.parametrize("li,beta,path_name", [(1, 32, "POPC"), (1, 128, "B1MMA"), (0, 32, "POPC"), (3, 16, "POPC")])
def test_integer_partials_of_sampled_rows_of_a_full_size_conv_matrix(hb, li, beta, path_name):
    """hbmm_quantize binarizes the whole batch-64 im2col-shaped matrix; the integer term of Eq. 7 is then
    written for a sample of its rows (a row-sliced operand) against all filters and must equal the
    checker's multiply-add partials of the same raw rows bit for bit."""
    gu = _gu()
    s = inputs.resnet18_convs(64)[li]
    M, N, K = s.M, s.N, s.K
    a = inputs.normal((M, K), inputs.SEEDS["resnet_hbmm"][0] + 60 + li)
    w = inputs.he_normal(N, K, inputs.SEEDS["resnet_hbmm"][1] + 60 + li)
    A = hb.quantize(torch.from_numpy(a).cuda(), hb.alloc_operand(M, K, beta, hb.F32))
    W = hb.quantize(torch.from_numpy(w).cuda(), hb.alloc_operand(N, K, beta, hb.F32))
    rows = _rows(M, 40, M + beta)
    rows_d = torch.from_numpy(rows).cuda()
    Asub = hb.wrap_packed(A.bits[rows_d].contiguous(), A.scales[rows_d].contiguous(), K, beta)
    _, sa = oracle.quantize(a[rows], beta)
    _, sw = oracle.quantize(w, beta)
    d_ref, _ = oracle.partials(sa, sw, beta, beta)
    D = torch.full(d_ref.shape, -12345, dtype=torch.int32, device="cuda")
    hb.gemm_partials(Asub, W, D, getattr(hb, "PATH_" + path_name))
    assert np.array_equal(D.cpu().numpy(), d_ref)
