"""The failure path of the bounded device-side waits, exercised without starving any real kernel.

Every wait in the tensor-core kernels and in the packed convolution front end gives up after a poll
limit, records a code in a device-side health word and lets the kernel return.  Here the limit is lowered
through the library's test hook and a one-block self-test kernel lets a single thread wait on a barrier
that nobody arrives at and that guards nothing; the wait must run out, the health word must report it as
HBMM_ERR_TIMEOUT (code 309), stay set until it is cleared, and a real contraction launched afterwards with
the default limit restored must be correct and leave the word clean.  Collected after every other test
file except the no-allocation one, so that a word left set by mistake cannot fail unrelated tests.
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
    assert hbmm.last_device_error() == 0
    yield hbmm
    hbmm.debug_set_wait_limit(0)
    hbmm.clear_device_error()
    assert hbmm.last_device_error() == 0


def test_a_wait_that_nobody_satisfies_runs_out_and_is_reported_then_cleared(hb):
    import gpu_util as gu
    hb.debug_set_wait_limit(300)
    hb.debug_expire_wait()
    torch.cuda.synchronize()                       # the kernel returned by itself
    code = hb._i32(0)
    assert hb._lib.hbmm_last_device_error(code) == hb.ERR_TIMEOUT
    assert code.value == 309
    # sticky: a second query still reports it, and a second expiry keeps the first code
    hb.debug_expire_wait()
    assert hb.last_device_error() == 309
    hb.clear_device_error()
    assert hb._lib.hbmm_last_device_error(code) == hb.OK and code.value == 0
    hb.debug_set_wait_limit(0)                     # back to the default limit

    # the context is intact: a real tensor-core contraction right behind it is correct and clean
    M, N, K, beta = 300, 136, 640, 32
    a = inputs.normal((M, K), 9901)
    w = inputs.he_normal(N, K, 9902)
    A, da, sa = gu.oracle_operand(a, beta)
    W, dw, sw = gu.oracle_operand(w, beta)
    c_ref, absref = oracle.hbmm_from_quantized(da, sa, beta, dw, sw, beta)
    ws = torch.empty(max(hb.gemm_workspace_bytes(A, W), 16), dtype=torch.uint8, device="cuda")
    for path in (hb.PATH_FOLDED, hb.PATH_TENSOR):
        C = torch.full((M, N), float("nan"), device="cuda")
        hb.gemm_ex(A, W, C, path, ws)
        gu.assert_close_rel_absref(C.cpu().numpy(), c_ref, absref, 1e-5, "after an expired wait, path %d" % path)
    assert hb.last_device_error() == 0


def test_the_wait_limit_hook_rejects_values_that_do_not_fit(hb):
    with pytest.raises(hb.HbmmError) as e:
        hb.debug_set_wait_limit(0xFFFFFFFF)
    assert e.value.status == hb.ERR_INVALID_ARG
