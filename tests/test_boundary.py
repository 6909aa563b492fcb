"""CPU-only checks of the C-ABI boundary: exported symbols, storage arithmetic, host-side validation.
No kernel is launched: every call here returns from the argument checks."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hb():
    from paper_1905_10759_b200 import build
    build.build_lib()
    from paper_1905_10759_b200 import hbmm
    return hbmm


def test_library_exports_every_declared_symbol(hb):
    header = open(os.path.join(ROOT, "include", "hbmm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(hbmm_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    lib = ctypes.CDLL(hb.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(hb.EXPORTS)
    assert hb.version() >= 100
    assert hb.status_string(hb.OK) == "ok"


def _golden_storage():
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", "storage_ratio.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                b, frac = line.split()
                rows.append((b, float(frac)))
    return rows


def test_storage_matches_paper_memory_column(hb):
    """bits per element = 1 + 32/beta with fp32 scales (beta*X/(beta+X) saving, X = 32): the paper's
    Table 2 prints ~.28, ~.16, ~.09 of full precision for beta_w = 4, 8, 16 and ~.03 for one scale per
    tensor.  The library stores whole-word groups, so the ratio is checked on beta = 32..K and the printed
    small-beta fractions are checked against the same closed form."""
    for b, frac in _golden_storage():
        closed = (1.0 / 32.0) if b == "inf" else (1.0 + 32.0 / int(b)) / 32.0
        assert abs(closed - frac) < 0.006, (b, closed, frac)
    rows, K = 512, 4096
    for beta, sdt, sbits in [(32, hb.F32, 32), (64, hb.F32, 32), (128, hb.F32, 32), (32, hb.BF16, 16), (4096, hb.F32, 32)]:
        bb, sb, lw, ls = hb.operand_bytes(rows, K, beta, sdt)
        bits_per_elt = 8.0 * (bb + sb) / (rows * K)
        g = -(-K // beta)
        pad = ls - g
        expect = 1.0 + sbits / beta + sbits * pad / K
        assert abs(bits_per_elt - expect) < 1e-12
        assert lw == K // 32 and lw % 4 == 0
    # ratio of the paper at beta = 32: 32*32/(32+32) = 16x smaller than fp32
    bb, sb, _, _ = hb.operand_bytes(rows, K, 32, hb.F32)
    assert abs(rows * K * 4 / (bb + sb) - 16.0) < 1e-9


def test_operand_bytes_padding_and_errors(hb):
    bb, sb, lw, ls = hb.operand_bytes(3, 100, 32, hb.F32)
    assert (lw, ls) == (4, 4) and bb == 3 * 4 * 4 and sb == 3 * 4 * 4
    _, _, lw, ls = hb.operand_bytes(3, 577, 64, hb.BF16)
    assert lw == 20 and ls == 16
    _, _, lw, ls = hb.operand_bytes(1, 77, 77, hb.F32)
    assert (lw, ls) == (4, 4)
    for args in [(0, 10, 32, 0), (10, 0, 32, 0), (10, 10, 1, 0), (10, 10, 32, 7)]:
        with pytest.raises(hb.HbmmError) as e:
            hb.operand_bytes(*args)
        assert e.value.status == hb.ERR_INVALID_ARG


def _fake_packed(hb, rows, K, beta, sdt=0, bits=0x1000, scales=0x2000, lw=None, ls=None):
    d = hb.hbmm_operand()
    _, _, lw0, ls0 = hb.operand_bytes(rows, K, max(beta, 2), sdt)
    d.rows, d.K, d.beta, d.scale_dtype = rows, K, beta, sdt
    d.bits, d.scales = bits, scales
    d.ld_words, d.ld_scales = lw0 if lw is None else lw, ls0 if ls is None else ls
    return hb.Operand(d)


def test_host_validation_rejects_before_launch(hb):
    """Fake (never dereferenced) device addresses: every call must fail in the host checks."""
    lib = hb._lib
    A = _fake_packed(hb, 8, 64, 32)
    W = _fake_packed(hb, 4, 64, 32)
    c = ctypes.c_void_p(0x3000)

    def gemm(a, w, cptr=c, ldc=4, path=0):
        return lib.hbmm_gemm_ex(ctypes.byref(a.desc), ctypes.byref(w.desc), cptr, ldc, None, 0, path, None)

    assert gemm(A, _fake_packed(hb, 4, 96, 32)) == hb.ERR_INVALID_ARG           # K mismatch
    assert gemm(A, W, ldc=3) == hb.ERR_INVALID_ARG                               # ldc < N
    assert gemm(A, W, cptr=ctypes.c_void_p(0x3004)) == hb.ERR_ALIGNMENT          # C not 16-byte aligned
    assert gemm(A, W, ldc=6) == hb.ERR_ALIGNMENT                                 # ldc % 4
    assert gemm(A, W, cptr=None) == hb.ERR_INVALID_ARG
    assert gemm(_fake_packed(hb, 8, 64, 12), W) == hb.ERR_UNSUPPORTED            # sub-word beta that is no power of two
    assert gemm(_fake_packed(hb, 8, 64, 32, bits=0x1004), W) == hb.ERR_ALIGNMENT
    assert gemm(_fake_packed(hb, 8, 64, 32, lw=2), W) == hb.ERR_ALIGNMENT        # ld_words % 4
    assert gemm(_fake_packed(hb, 8, 64, 32, lw=1), W) == hb.ERR_INVALID_ARG      # ld_words too small
    assert gemm(_fake_packed(hb, 8, 64, 32, ls=1), W) == hb.ERR_INVALID_ARG
    assert gemm(A, W, path=9) == hb.ERR_INVALID_ARG
    a192 = _fake_packed(hb, 8, 384, 64)
    w192 = _fake_packed(hb, 4, 384, 96)
    assert gemm(a192, w192) == hb.ERR_UNSUPPORTED                                 # 96 is no multiple of 64
    dense_w = hb.Operand(hb.hbmm_operand(rows=4, K=64, beta=1))
    assert gemm(A, dense_w) == hb.ERR_UNSUPPORTED                                 # weights must be packed
    both_dense = hb.Operand(hb.hbmm_operand(rows=8, K=64, beta=1))
    assert gemm(both_dense, W) == hb.ERR_INVALID_ARG                              # dense pointer missing
    assert lib.hbmm_gemm_ex(None, ctypes.byref(W.desc), c, 4, None, 0, 0, None) == hb.ERR_INVALID_ARG

    q = _fake_packed(hb, 8, 64, 32)
    x = ctypes.c_void_p(0x5000)
    assert lib.hbmm_quantize(x, 0, 8, 64, 32, ctypes.byref(q.desc), None) == hb.ERR_INVALID_ARG   # ldx < K
    assert lib.hbmm_quantize(x, 0, 9, 64, 64, ctypes.byref(q.desc), None) == hb.ERR_INVALID_ARG   # rows mismatch
    assert lib.hbmm_quantize(None, 0, 8, 64, 64, ctypes.byref(q.desc), None) == hb.ERR_INVALID_ARG
    assert lib.hbmm_quantize(x, 5, 8, 64, 64, ctypes.byref(q.desc), None) == hb.ERR_INVALID_ARG
    q24 = _fake_packed(hb, 8, 64, 24)
    assert lib.hbmm_quantize(x, 0, 8, 64, 64, ctypes.byref(q24.desc), None) == hb.ERR_UNSUPPORTED

    g = hb.make_geom(2, 4, 8, 8, 3, 3, (1, 1), (1, 1))
    Wc = _fake_packed(hb, 4, 36, 36)
    n = ctypes.c_size_t()
    assert lib.hbmm_conv_workspace_bytes(ctypes.byref(g), 36, 0, ctypes.byref(Wc.desc), ctypes.byref(n)) == hb.OK
    assert n.value > 0
    ws = ctypes.c_void_p(0x10000)
    call = lambda geom, w, wsp, wsb, beta_a=36: lib.hbmm_conv_im2col(x, 0, ctypes.byref(geom), beta_a, 0, ctypes.byref(w.desc), c, 4, wsp, wsb, None)
    assert call(g, Wc, ws, n.value - 1) == hb.ERR_WORKSPACE
    assert call(g, Wc, None, n.value) == hb.ERR_WORKSPACE
    assert call(g, Wc, ctypes.c_void_p(0x10010), n.value) == hb.ERR_ALIGNMENT
    assert call(g, _fake_packed(hb, 4, 40, 40), ws, n.value) == hb.ERR_INVALID_ARG    # K != C*kh*kw
    bad = hb.make_geom(2, 4, 2, 2, 5, 5, (1, 1), (0, 0))
    assert call(bad, Wc, ws, n.value) == hb.ERR_INVALID_ARG                           # filter larger than image
    assert call(g, Wc, ws, n.value, beta_a=12) == hb.ERR_UNSUPPORTED
    assert lib.hbmm_conv_im2col_ex(x, 0, ctypes.byref(g), 36, 0, ctypes.byref(Wc.desc), c, 4, ws, n.value, 4, None) == hb.ERR_INVALID_ARG  # unknown flag
    assert lib.hbmm_conv_im2col_ex(x, 0, ctypes.byref(g), 1, 0, ctypes.byref(Wc.desc), c, 4, ws, n.value, hb.CONV_PACK_ONLY,
                                   None) == hb.ERR_INVALID_ARG             # only a packed operand can be left behind
    fz = lib.hbmm_gemm_binarize_next
    nx = _fake_packed(hb, 8, 4, 2)
    assert fz(ctypes.byref(A.desc), ctypes.byref(W.desc), None, None, ctypes.byref(nx.desc), None, 0, None) == hb.ERR_WORKSPACE
    assert fz(ctypes.byref(A.desc), ctypes.byref(W.desc), None, None, ctypes.byref(_fake_packed(hb, 8, 5, 2).desc), None, 0, None) == hb.ERR_INVALID_ARG   # K of next != rows of W
    assert fz(ctypes.byref(A.desc), ctypes.byref(W.desc), None, None, ctypes.byref(_fake_packed(hb, 8, 4, 4).desc), None, 0, None) == hb.ERR_UNSUPPORTED   # group as long as the row
    bw = lib.hbmm_binarize_backward
    assert bw(x, 64, x, 64, 8, 64, 4, c, 32, None) == hb.ERR_INVALID_ARG          # output rows shorter than K
    assert bw(x, 64, x, 64, 8, 64, 0, c, 64, None) == hb.ERR_INVALID_ARG          # beta < 1
    assert bw(None, 64, x, 64, 8, 64, 4, c, 64, None) == hb.ERR_INVALID_ARG
    assert bw(ctypes.c_void_p(0x5002), 64, x, 64, 8, 64, 4, c, 64, None) == hb.ERR_ALIGNMENT
    bd = lib.hbmm_binarize_dense
    assert bd(x, 64, 8, 64, 4, c, hb.F32, 32, None) == hb.ERR_INVALID_ARG            # output rows shorter than K
    assert bd(x, 64, 8, 64, 0, c, hb.F32, 64, None) == hb.ERR_INVALID_ARG            # beta < 1
    assert bd(x, 64, 8, 64, 4, c, 7, 64, None) == hb.ERR_INVALID_ARG                 # unknown output type
    assert bd(x, 64, 8, 64, 4, None, hb.F32, 64, None) == hb.ERR_INVALID_ARG
    assert bd(x, 64, 8, 64, 4, ctypes.c_void_p(0x5002), hb.F32, 64, None) == hb.ERR_ALIGNMENT
    assert bd(x, 64, 8, 64, 4, ctypes.c_void_p(0x5001), hb.BF16, 64, None) == hb.ERR_ALIGNMENT
