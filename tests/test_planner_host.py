"""The library's host-side planner (forge_plan_liveness, forge_plan_linear_scan, forge_decoder_layer_plan)
against the planning oracle, integer for integer.  No GPU is involved: the planner is host code."""
import random

import pytest

from oracle import planner as oracle_planner
from paper_2604_16498_b200 import binding


def test_linear_scan_matches_the_oracle_on_random_intervals():
    rng = random.Random(11)
    for trial in range(300):
        n = rng.randint(1, 60)
        start = [rng.randint(0, 80) for _ in range(n)]
        end = [s + rng.randint(0, 20) for s in start]
        nbytes = [rng.randint(1, 1 << 20) for _ in range(n)]
        pinned = [rng.random() < 0.1 for _ in range(n)] if trial % 3 == 0 else None
        want, m = oracle_planner.linear_scan(start, end, pinned)
        got, buf_bytes, gm = binding.plan_linear_scan(start, end, nbytes, pinned)
        assert got == want and gm == m
        # every buffer is as large as its largest tenant
        for b in range(m):
            assert buf_bytes[b] == max(nbytes[r] for r in range(n) if got[r] == b)


def test_liveness_matches_the_oracle_on_random_programs():
    rng = random.Random(12)
    for trial in range(200):
        num_ops = rng.randint(1, 30)
        num_inputs = rng.randint(1, 3)
        num_regs = num_inputs + num_ops
        out_reg, reads = [], []
        for j in range(num_ops):
            avail = num_inputs + j
            reads.append(rng.sample(range(avail), rng.randint(1, min(3, avail))))
            out_reg.append(num_inputs + j if rng.random() < 0.95 else -1)
        assert binding.plan_liveness(out_reg, reads, num_regs) == tuple(oracle_planner.liveness(out_reg, reads, num_regs))


def test_empty_and_invalid_inputs():
    assert binding.plan_linear_scan([], []) == ([], [], 0)
    with pytest.raises(binding.ForgeError) as e:
        binding.plan_linear_scan([3], [2])          # an interval that ends before it starts
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.ForgeError):
        binding.plan_liveness([0, 0], [[], []], 1)  # two writers of one register
    with pytest.raises(binding.ForgeError):
        binding.plan_liveness([0], [[5]], 1)        # register index out of range


@pytest.mark.parametrize("dims", [(2, 256, 12, 12, 64, 3072, binding.MLP_GELU), (1, 2048, 32, 8, 128, 14336, binding.MLP_SWIGLU)])
def test_decoder_layer_plan(dims):
    B, S, Hq, Hkv, D, F, mlp = dims
    p = binding.decoder_layer_plan(B, S, Hq, Hkv, D, F, mlp)
    T, H = B * S, Hq * D
    reg_bytes = [T * (Hq + 2 * Hkv) * D * 2, T * H * 2, T * H * 2, T * F * 2]
    assert list(p.reg_bytes) == reg_bytes
    # the same intervals and the same assignment as the oracle's planner gives for this instruction list
    start, end = oracle_planner.liveness([1, 2, 3, 4, 5], [[0], [1], [2, 0], [3], [4, 3]], 6)
    assert list(p.reg_start) == start[1:5] and list(p.reg_end) == end[1:5]
    want, m = oracle_planner.linear_scan(start[1:5], end[1:5])
    assert list(p.buf_of) == want and p.num_bufs == m == 2 and p.num_regs == 4
    assert abs(p.rho_buf - oracle_planner.rho_buf(4, m)) < 1e-7
    assert p.buf_bytes[0] == max(reg_bytes[0], reg_bytes[2]) and p.buf_bytes[1] == max(reg_bytes[1], reg_bytes[3])
    assert p.buf_offset[0] == 0 and p.buf_offset[1] % 256 == 0 and p.buf_offset[1] >= p.buf_bytes[0]
    assert p.workspace_bytes >= p.buf_bytes[0] + p.buf_bytes[1] and p.workspace_bytes < p.unplanned_bytes
