"""CPU oracle for the buffer planning of a fixed operator sequence.  Test infrastructure only.

Plain Python restatements of Section 4.5: the live interval of a register (Eq. 14), the linear-scan
assignment of intervals to buffers (Algorithm 2) and the buffer reduction ratio (Eq. 15).  Shares no code
with the library's planner.
"""
from __future__ import annotations


def liveness(out_reg, in_regs_per_op, num_regs):
    """Eq. 14: s_r = the instruction that writes r, e_r = the last instruction that reads r.
    A register nobody writes has s = -1; a register nobody reads has e = s."""
    start = [-1] * num_regs
    end = [-1] * num_regs
    for j, (w, reads) in enumerate(zip(out_reg, in_regs_per_op)):
        for r in reads:
            end[r] = max(end[r], j)
        if w >= 0:
            assert start[w] < 0, "a register has one writer"
            start[w] = j
    for r in range(num_regs):
        if end[r] < start[r]:
            end[r] = start[r]
    return start, end


def linear_scan(start, end, pinned=None):
    """Algorithm 2: intervals by ascending start; expire the active ones that ended before the current start
    and put their buffers into the free pool; take a buffer from the pool (the one freed earliest) or, if the
    pool is empty or the register is pinned, a new one; the interval becomes active.  Returns (buf_of, M)."""
    n = len(start)
    pinned = pinned or [False] * n
    order = sorted(range(n), key=lambda r: (start[r], r))
    active = []     # (end, buffer) in the order the intervals were opened
    free_pool = []
    buf_of = [None] * n
    m = 0
    for r in order:
        still = []
        for e, b in active:
            if e < start[r]:
                free_pool.append(b)
            else:
                still.append((e, b))
        active = still
        if pinned[r] or not free_pool:
            b = m
            m += 1
        else:
            b = free_pool.pop(0)
        buf_of[r] = b
        active.append((end[r], b))
    return buf_of, m


def rho_buf(n, m):
    """Eq. 15."""
    return 1.0 - m / n
