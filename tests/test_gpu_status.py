"""The give-up path of the tensor-core kernels, exercised without hanging or faulting anything.

Every wait inside those kernels is bounded.  ``bnn_wait_probe`` enqueues a one-warp launch that
waits on a barrier on which nothing ever arrives: with a short limit its wait runs out, the kernel
returns normally and sets the device status word.  The test reads the word in stream order
(``bnn_query_status``) and through the synchronising call, resets it, and checks that the next
ordinary launch is bit-exact."""
import numpy as np
import pytest

from oracle import bnn_oracle as o
from paper_1706_09453_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available()
    from paper_1706_09453_b200 import build, binding, model
    build.build()
    return torch, binding, model


def test_wait_that_runs_out_sets_the_status_word_and_leaves_the_context_usable(env):
    torch, B, model = env
    assert B.bnn_device_status() == 0
    word = torch.full((4,), -1, dtype=torch.int32, device="cuda:0")
    prev = B.bnn_set_option(B.OPT_WAIT_LIMIT_US, 50)      # 50 us = 1e5 clocks
    try:
        B.bnn_query_status(word[0:1])                      # before: 0
        B.bnn_wait_probe()
        B.bnn_query_status(word[1:2])                      # after the probe, in stream order: 1
        B.bnn_reset_status()
        B.bnn_query_status(word[2:3])                      # after the reset: 0
        B.bnn_wait_probe()
        torch.cuda.synchronize()                           # the launches returned: nothing hangs
        assert word.cpu().tolist()[:3] == [0, 1, 0]
        assert B.bnn_device_status() == 1                  # the second probe set it again
        assert B.raw_call("bnn_device_status", B.C.byref(B.C.c_int(0))) == B.ERR_TIMEOUT
        B.bnn_reset_status()
        assert B.bnn_device_status() == 0
    finally:
        B.bnn_set_option(B.OPT_WAIT_LIMIT_US, prev)
    # the context is intact: an ordinary tensor-core launch right after is bit-exact
    m, n, k = 300, 257, 1000
    ap = wl.make_bit_planes(m, k, 0.5, [1, m, n, k], B.packed_pitch(k))
    wp = wl.make_bit_planes(n, k, 0.5, [2, m, n, k], B.packed_pitch(k))
    c = torch.empty((m, n), dtype=torch.int32, device="cuda:0")
    B.bnn_xnor_gemm(model.to_dev(ap), model.to_dev(wp), k, C_out=c)
    np.testing.assert_array_equal(c.cpu().numpy(), o.xnor_gemm(ap, wp, k))
    assert B.bnn_device_status() == 0


def test_wait_limit_option_bounds(env):
    torch, B, model = env
    with pytest.raises(ValueError):
        B.bnn_set_option(B.OPT_WAIT_LIMIT_US, 0)
    prev = B.bnn_set_option(B.OPT_WAIT_LIMIT_US, 1234)
    assert B.bnn_set_option(B.OPT_WAIT_LIMIT_US, prev) == 1234
