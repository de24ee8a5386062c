"""GPU parity: forge_attn_decode_splitkv against the fp64 oracle (bf16 tolerances)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device, to_pinned

pytestmark = pytest.mark.gpu


def _run(w, num_splits=None):
    ns = w.num_splits if num_splits is None else num_splits
    out = binding.attn_decode_splitkv(to_device(w.q), to_device(w.k_cache), to_device(w.v_cache),
                                      torch.from_numpy(w.lens).cuda(), ns, w.scale)
    ref = oracle.attn_decode(w.q.values, w.k_cache.values, w.v_cache.values, w.lens, w.scale)
    assert_close_bf16(out, ref)
    return out


def test_cfg5_full_size():
    w = wl.cfg5_gqa_decode()
    assert w.lens.min() >= 1024 and w.lens.max() <= 4096
    _run(w)


@pytest.mark.parametrize("num_splits", [1, 2, 16, 17])
def test_result_does_not_depend_on_num_splits(num_splits):
    w = wl.decode_workload("t", 21, 4, 8, 2, 700, 128, 16, 1.0 / np.sqrt(128.0), (1, 700))
    _run(w, num_splits)


@pytest.mark.parametrize("D,Hq,Hkv", [(64, 12, 12), (64, 8, 4), (128, 8, 1), (128, 32, 8), (64, 16, 2),
                                       (128, 28, 4), (64, 6, 2), (128, 10, 2), (64, 12, 2)])
def test_head_dims_and_group_sizes(D, Hq, Hkv):
    w = wl.decode_workload("t", 22, 3, Hq, Hkv, 333, D, 5, 1.0 / np.sqrt(D), (1, 333))
    _run(w)


def test_batch_larger_than_the_length_ranking_limit():
    """More than 64 sequences: the kernel deals the items in batch order instead of by cached length."""
    w = wl.decode_workload("t", 25, 80, 4, 2, 160, 64, 3, 0.125, (1, 160))
    _run(w)


@pytest.mark.parametrize("D", [32, 80, 96, 120])
def test_other_head_dimensions(D):
    """Head sizes other than 64 and 128 (multiples of 8) run on the next larger kernel with zero padding."""
    w = wl.decode_workload("t", 26, 3, 8, 2, 300, D, 5, 1.0 / np.sqrt(D), (1, 300))
    _run(w)


def test_short_and_degenerate_lengths():
    """Fewer rows than splits (empty splits), one row, zero rows, and lens beyond Smax (clamped)."""
    w = wl.decode_workload("t", 23, 5, 8, 2, 64, 128, 16, 0.1, (1, 64))
    w.lens = np.array([1, 3, 0, 64, 1000], dtype=np.int32)
    out = _run(w)
    assert (out[2] == 0).all()


def test_rows_beyond_lens_are_never_read_into_the_result():
    w = wl.decode_workload("t", 24, 2, 4, 1, 128, 64, 4, 0.125, (5, 100))
    k, v = to_device(w.k_cache), to_device(w.v_cache)
    lens = torch.from_numpy(w.lens).cuda()
    a = binding.attn_decode_splitkv(to_device(w.q), k, v, lens, 4, w.scale)
    for b in range(2):
        k[b, :, int(w.lens[b]):] = float("nan")
        v[b, :, int(w.lens[b]):] = float("inf")
    b2 = binding.attn_decode_splitkv(to_device(w.q), k, v, lens, 4, w.scale)
    assert torch.equal(a, b2)


def test_one_workspace_serves_call_after_call_with_other_shapes():
    """The arrival counters at the start of the workspace are cleared once; every call leaves them at zero,
    so the same (oversized) workspace works for any later call."""
    ws = torch.empty(binding.attn_decode_workspace_bytes(16, 32, 128, 16), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)
    binding.attn_decode_workspace_init(ws)
    for rep in range(2):
        for (B, Hq, Hkv, Smax, D, splits, lo) in [(6, 32, 8, 1500, 128, 16, 200), (3, 8, 2, 700, 64, 9, 1),
                                                  (16, 16, 8, 2100, 128, 4, 1800), (2, 8, 1, 4000, 128, 16, 3000)]:
            w = wl.decode_workload("t", 27, B, Hq, Hkv, Smax, D, splits, 1.0 / np.sqrt(D), (lo, Smax))
            out = binding.attn_decode_splitkv(to_device(w.q), to_device(w.k_cache), to_device(w.v_cache),
                                              torch.from_numpy(w.lens).cuda(), splits, w.scale, workspace=ws)
            binding.check_status()
            assert_close_bf16(out, oracle.attn_decode(w.q.values, w.k_cache.values, w.v_cache.values, w.lens, w.scale))


def test_more_pieces_than_workers():
    """A batch whose pieces outnumber the GPU's workers (7 per SM) even at the longest allowed piece: workers
    take several pieces each."""
    w = wl.decode_workload("t", 28, 200, 8, 8, 48, 64, 2, 0.125, (1, 48))
    _run(w)


def test_run_to_run_bitwise_identical():
    w = wl.cfg5_gqa_decode(B=8)
    q, k, v, lens = to_device(w.q), to_device(w.k_cache), to_device(w.v_cache), torch.from_numpy(w.lens).cuda()
    a = binding.attn_decode_splitkv(q, k, v, lens, w.num_splits, w.scale)
    b = binding.attn_decode_splitkv(q, k, v, lens, w.num_splits, w.scale)
    assert torch.equal(a, b)


def test_workspace_too_small_is_rejected():
    w = wl.decode_workload("t", 25, 1, 4, 1, 32, 64, 4, 0.125, (5, 32))
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.ForgeError) as e:
        binding.attn_decode_splitkv(to_device(w.q), to_device(w.k_cache), to_device(w.v_cache),
                                    torch.from_numpy(w.lens).cuda(), 4, w.scale, workspace=ws)
    assert e.value.status == binding.ERR_WORKSPACE


def test_host_buffer_variant():
    w = wl.decode_workload("t", 26, 2, 8, 2, 300, 128, 8, 0.09, (100, 300))
    q, k, v = to_pinned(w.q), to_pinned(w.k_cache), to_pinned(w.v_cache)
    out = torch.empty_like(q).pin_memory()
    scratch = torch.empty(binding.attn_decode_host_scratch_bytes(2, 8, 2, 300, 128, 8), dtype=torch.uint8,
                          device="cuda")
    binding.attn_decode_splitkv_host(q, k, v, torch.from_numpy(w.lens), 8, out, scratch, w.scale)
    binding.check_status()
    ref = oracle.attn_decode(w.q.values, w.k_cache.values, w.v_cache.values, w.lens, w.scale)
    assert_close_bf16(out, ref)


@pytest.mark.parametrize("num_splits", [130, 256])
def test_single_long_sequence_with_many_pieces(num_splits):
    """One sequence, two kv heads: the pieces of a sequence number more than 64 (the merge keeps eight (m, l) pairs
    per lane and head); 257 pieces are refused."""
    w = wl.decode_workload("t", 33, 1, 8, 2, 20000, 128, num_splits, 1.0 / np.sqrt(128), (19000, 20000))
    _run(w, num_splits)
    with pytest.raises(binding.ForgeError) as e:
        binding.attn_decode_splitkv(to_device(w.q), to_device(w.k_cache), to_device(w.v_cache),
                                    torch.from_numpy(w.lens).cuda(), 257, w.scale)
    assert e.value.status == binding.ERR_UNSUPPORTED
