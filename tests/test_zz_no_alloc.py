"""hbmm_conv_im2col_static: the convolution entry point for callers that cannot allocate device
memory (their framework owns the device, or they run where cudaMalloc is not allowed).  Its scratch
is a fixed array inside the library, so the checks here are: same results as hbmm_conv_im2col with a
caller workspace, on two calls in a row that reuse the shared array (the second smaller than the
first, so stale contents of the first are still lying behind it), and a clean refusal of a problem
that does not fit.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_1905_10759_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_1905_10759_b200 import hbmm
    return hbmm


def _both(hb, shape, seed, beta):
    x = torch.from_numpy(inputs.conv_activation(shape, seed, signed=True)).cuda()
    w = torch.from_numpy(inputs.he_normal(shape.N, shape.K, seed + 1)).cuda()
    W = hb.quantize(w, hb.alloc_operand(shape.N, shape.K, beta))
    geom = hb.make_geom(shape.B, shape.C, shape.H, shape.W, shape.kh, shape.kw, (shape.stride,) * 2, (shape.pad,) * 2)
    ws = torch.empty(hb.conv_workspace_bytes(geom, beta, hb.F32, W), dtype=torch.uint8, device="cuda")
    ref = torch.empty((shape.M, shape.N), device="cuda")
    hb.conv_im2col(x, geom, beta, hb.F32, W, ref, ws)
    out = torch.full((shape.M, shape.N), float("nan"), device="cuda")
    hb.conv_im2col_static(x, geom, beta, hb.F32, W, out)
    torch.cuda.synchronize()
    return out.cpu().numpy(), ref.cpu().numpy()


def test_static_scratch_matches_workspace_entry_point_twice(hb):
    first = inputs.ConvShape("a", 4, 64, 14, 14, 96)
    second = inputs.ConvShape("b", 2, 32, 9, 7, 40)          # smaller: sits on top of the first call's leftovers
    for shape, seed, beta in ((first, 31, 32), (second, 47, 64)):
        out, ref = _both(hb, shape, seed, beta)
        # the same kernels on the same inputs, only the scratch differs: the tolerance of the other GPU tests
        # (1e-5 relative) holds with room to spare, because the two results are bit-identical
        scale = np.abs(ref).max()
        np.testing.assert_allclose(out, ref, rtol=1e-5, atol=1e-5 * scale)
        assert np.array_equal(out, ref)


def test_static_entry_point_leaves_device_memory_as_it_found_it(hb):
    """After the first call on a device (which may load the part of the library that holds the array) further
    calls must not change the amount of free device memory: the entry point allocates and frees nothing."""
    shape = inputs.ConvShape("c", 2, 64, 12, 12, 48)
    x = torch.from_numpy(inputs.conv_activation(shape, 53, signed=True)).cuda()
    W = hb.quantize(torch.from_numpy(inputs.he_normal(shape.N, shape.K, 54)).cuda(), hb.alloc_operand(shape.N, shape.K, 32))
    geom = hb.make_geom(shape.B, shape.C, shape.H, shape.W, 3, 3, (1, 1), (1, 1))
    out = torch.empty((shape.M, shape.N), device="cuda")
    hb.conv_im2col_static(x, geom, 32, hb.F32, W, out)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        hb.conv_im2col_static(x, geom, 32, hb.F32, W, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_static_scratch_rejects_problems_that_do_not_fit(hb):
    big = inputs.ConvShape("big", 128, 64, 56, 56, 64)
    W = hb.alloc_operand(big.N, big.K, 32)
    geom = hb.make_geom(big.B, big.C, big.H, big.W, 3, 3, (1, 1), (1, 1))
    assert hb.conv_workspace_bytes(geom, 32, hb.F32, W) > hb.STATIC_SCRATCH_BYTES
    x = torch.empty(1, device="cuda")        # never read: the size check comes before any launch
    out = torch.empty((4, 64), device="cuda")
    with pytest.raises(hb.HbmmError) as e:
        hb._check(hb._lib.hbmm_conv_im2col_static(x.data_ptr(), hb.F32, geom, 32, hb.F32, W.desc, out.data_ptr(), 64, None),
                  "hbmm_conv_im2col_static")
    assert e.value.status == hb.ERR_WORKSPACE
