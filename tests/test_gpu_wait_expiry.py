"""A bounded wait that runs out: the kernel must record a code, drain and return, and the library must stay usable.

Every wait inside the tensor-core kernels is bounded.  Here the single-CTA contraction kernel (one CTA) and the
CTA-pair kernel (one pair) are launched on one tile of one k-block with their producers switched off
(pd_debug_withhold_loads) and the limit cut to one millisecond: the warp that feeds the tensor core waits for an
operand stage nobody fills, gives up, and the kernel returns.  Nothing faults or hangs: no copy and no product is
in flight when the wait gives up."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import dev_bf16, host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("tile_mode,M", [(1, 128), (2, 256)], ids=["single_cta_kernel", "cta_pair_kernel"])
def test_expired_wait_is_reported_and_the_next_launch_is_correct(tile_mode, M):
    from paper_2511_03586_b200 import api
    N, K = 256, 64                                            # one tile (128 or 256 rows x 256 columns), one k-block
    p = inputs.gemm_integer_inputs(M, N, K, seed=5)
    a, b = dev_bf16(p["a_bits"][0]), dev_bf16(p["b_bits"][0])
    ref = oracle.gemm(p["a"][0], p["b"][0])
    api.pd_clear_device_status()
    api.pd_set_gemm_tile_mode(tile_mode)
    try:
        api.pd_debug_set_wait_limit_ns(1_000_000)              # 1 ms
        api.pd_debug_withhold_loads(True)
        c = torch.full((M, N), -3.0, dtype=torch.float32, device="cuda")
        api.pd_gemm_bf16(a, b, c)                              # enqueues; PD_OK only says so
        code = api.pd_get_device_status()                      # synchronises
        assert 101 <= code <= 104, code                        # 102: the wait for an operand stage
        assert api._lib.pd_get_device_status(ctypes.byref(ctypes.c_int(0))) == 7   # PD_ERR_DEVICE_TIMEOUT
        assert bool((c == -3.0).all())                         # the aborted kernel wrote nothing
    finally:
        api.pd_debug_withhold_loads(False)
        api.pd_debug_set_wait_limit_ns(2_000_000_000)
    api.pd_clear_device_status()
    try:
        # the context is intact: the same launch now completes and is exact, and the status word stays clear
        c = api.pd_gemm_bf16(a, b, c_dtype=torch.float32)
        assert np.array_equal(host(c), ref)
        assert api.pd_get_device_status() == 0
    finally:
        api.pd_set_gemm_tile_mode(0)


def test_debug_switch_arguments():
    from paper_2511_03586_b200 import api
    assert api._lib.pd_debug_set_wait_limit_ns(10) == 2        # below 1 us: PD_ERR_BAD_SHAPE
    assert api._lib.pd_debug_withhold_loads(2) == 2
    assert api._lib.pd_debug_withhold_loads(0) == 0
