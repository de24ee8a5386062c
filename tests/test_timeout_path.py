"""The failure path of the kernels' bounded waits, exercised without starving a real kernel.

forge_debug_wait_timeout launches one warp that runs the library's wait routine, with a short clock
budget, on a barrier that nothing completes.  The warp must give up, set the device's status word and
return; forge_check_status then reports FORGE_ERR_TIMEOUT once, and FORGE_OK afterwards, and the
context stays usable (a real operator call still gives the right answer).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device


def test_budget_is_validated_on_the_host():
    lib = binding.load()
    assert lib.forge_debug_wait_timeout(-1, None) == binding.ERR_INVALID_ARG
    assert lib.forge_debug_wait_timeout(10**12, None) == binding.ERR_INVALID_ARG


@pytest.mark.gpu
def test_expired_wait_is_reported_once_and_the_context_survives():
    lib = binding.load()
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.forge_check_status(stream) == binding.OK
    binding.debug_wait_timeout(1_000_000)  # about half a millisecond of SM clocks
    assert lib.forge_check_status(stream) == binding.ERR_TIMEOUT
    assert lib.forge_status_string(binding.ERR_TIMEOUT) == b"FORGE_ERR_TIMEOUT"
    assert lib.forge_check_status(stream) == binding.OK  # the flag was cleared by the report
    with pytest.raises(binding.ForgeError) as e:
        binding.debug_wait_timeout(1_000)
        binding.check_status()
    assert e.value.status == binding.ERR_TIMEOUT
    # the device is still fine
    w = wl.linear_workload("t", 34, 130, 72, 64, w_std=1.0 / 8)
    y = binding.linear_bias_gelu(to_device(w.x), to_device(w.w), to_device(w.b))
    binding.check_status()
    assert_close_bf16(y, oracle.linear_bias_gelu(w.x.values, w.w.values, w.b.values))
    torch.cuda.synchronize()
