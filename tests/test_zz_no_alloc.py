"""The decode entry point that allocates nothing (forge_attn_decode_splitkv_static).

It serves callers that cannot allocate device memory (frozen memory plans, hosted plugins,
latency paths that must not hit cudaMalloc's synchronisation), so its split partials live in a
fixed array inside the library instead of a caller workspace.  The checks: through the C ABI it
gives what forge_attn_decode_splitkv gives, twice in a row on different problems (the array keeps
the first call's contents, which must not leak into the second), and it refuses problems whose
partials exceed the array.  This file sorts last so that a run that stops at the first failure
has already run every other test.
"""
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device, to_f64

P = 0x10000  # fake aligned pointer for calls that must be refused before anything is touched


def test_too_large_problem_is_refused_before_any_device_work():
    lib = binding.load()
    assert lib.forge_attn_decode_workspace_bytes(64, 64, 128, 64) > binding.DECODE_STATIC_SCRATCH_BYTES
    st = lib.forge_attn_decode_splitkv_static(P, P, P, P, 64, 64, 8, 4096, 128, P, 64, 1.0, None)
    assert st == binding.ERR_WORKSPACE
    st = lib.forge_attn_decode_splitkv_static(None, P, P, P, 1, 8, 2, 64, 128, P, 4, 1.0, None)
    assert st == binding.ERR_INVALID_ARG


@pytest.mark.gpu
def test_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    lib = binding.load()
    stream = torch.cuda.current_stream().cuda_stream
    cases = [
        # long sequences cut into many pieces, so the partials really go through the fixed array (the
        # first call may use up to 6.2 MiB of it, the second a small corner)
        wl.decode_workload("first", 61, 16, 32, 8, 1024, 128, 24, 128 ** -0.5, (300, 1024)),
        wl.decode_workload("second", 62, 3, 8, 2, 700, 64, 20, 0.125, (1, 700)),
    ]
    for w in cases:
        q, k, v = to_device(w.q), to_device(w.k_cache), to_device(w.v_cache)
        lens = torch.from_numpy(w.lens).cuda()
        expect = binding.attn_decode_splitkv(q, k, v, lens, w.num_splits, w.scale)
        out = torch.full_like(q, float("nan"))
        st = lib.forge_attn_decode_splitkv_static(
            q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), w.B, w.Hq, w.Hkv, w.Smax, w.D,
            lens.data_ptr(), w.num_splits, float(w.scale), stream)
        assert st == binding.OK, lib.forge_status_string(st)
        binding.check_status()
        assert_close_bf16(out, to_f64(expect))
        assert torch.equal(out, expect)  # same kernels, same order of operations
        # and both are right: the oracle on the same inputs
        assert_close_bf16(out, oracle.attn_decode(w.q.values, w.k_cache.values, w.v_cache.values, w.lens, w.scale))


@pytest.mark.gpu
def test_too_large_problem_launches_nothing():
    w = wl.decode_workload("big", 63, 2, 8, 2, 64, 128, 4, 0.1, (10, 64))
    q, k, v = to_device(w.q), to_device(w.k_cache), to_device(w.v_cache)
    lens = torch.from_numpy(w.lens).cuda()
    before = binding.launch_count()
    # claim a batch whose counters and partials (4 slots of 130 floats per (batch, head)) exceed the 8 MiB array
    st = binding.load().forge_attn_decode_splitkv_static(
        q.data_ptr(), k.data_ptr(), v.data_ptr(), q.data_ptr(), 4096, 8, 2, 64, 128, lens.data_ptr(), 4, 0.1,
        torch.cuda.current_stream().cuda_stream)
    assert st == binding.ERR_WORKSPACE
    assert binding.launch_count() == before
