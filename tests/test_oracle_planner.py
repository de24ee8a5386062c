"""Pins of the buffer-planning oracle (oracle/planner.py) against what the paper and the mathematics fix:
hand-worked examples, the optimum known for interval graphs, validity, and a hand-checked liveness case."""
import itertools
import os
import random

import pytest

from oracle import planner

HERE = os.path.dirname(os.path.abspath(__file__))


def _examples():
    out = []
    for line in open(os.path.join(HERE, "golden", "planner_examples.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, s, e, bufs, m = [f.strip() for f in line.split("|")]
        out.append((name, [int(x) for x in s.split()], [int(x) for x in e.split()], [int(x) for x in bufs.split()], int(m)))
    return out


@pytest.mark.parametrize("name,start,end,bufs,m", _examples())
def test_hand_examples(name, start, end, bufs, m):
    got, gm = planner.linear_scan(start, end)
    assert got == bufs and gm == m


def _overlap(a, b, start, end):
    return not (end[a] < start[b] or end[b] < start[a])


def _max_live(start, end):
    return max(sum(1 for r in range(len(start)) if start[r] <= t <= end[r]) for t in range(min(start), max(end) + 1))


def _chromatic_number(start, end):
    n = len(start)
    for k in range(1, n + 1):
        for colouring in itertools.product(range(k), repeat=n):
            if all(colouring[a] != colouring[b] for a in range(n) for b in range(a + 1, n) if _overlap(a, b, start, end)):
                return k
    return n


def test_no_two_live_registers_share_a_buffer_and_the_count_is_optimal():
    rng = random.Random(7)
    for trial in range(300):
        n = rng.randint(1, 7)
        start = [rng.randint(0, 8) for _ in range(n)]
        end = [s + rng.randint(0, 5) for s in start]
        bufs, m = planner.linear_scan(start, end)
        assert sorted(set(bufs)) == list(range(m))
        for a in range(n):
            for b in range(a + 1, n):
                if _overlap(a, b, start, end):
                    assert bufs[a] != bufs[b]
        # greedy by start time is optimal on interval graphs: M = the largest number of registers live at once
        assert m == _max_live(start, end)
        if n <= 6:
            assert m == _chromatic_number(start, end)


def test_larger_random_cases_reach_the_clique_bound():
    rng = random.Random(8)
    for trial in range(50):
        n = rng.randint(20, 200)
        start = [rng.randint(0, 300) for _ in range(n)]
        end = [s + rng.randint(0, 40) for s in start]
        bufs, m = planner.linear_scan(start, end)
        assert m == _max_live(start, end)
        assert all(bufs[a] != bufs[b] for a in range(n) for b in range(a + 1, n) if _overlap(a, b, start, end))


def test_pinned_registers_get_a_fresh_buffer():
    start, end = [0, 1, 2], [0, 1, 2]
    assert planner.linear_scan(start, end) == ([0, 0, 0], 1)
    assert planner.linear_scan(start, end, pinned=[False, True, False]) == ([0, 1, 0], 2)


def test_liveness_of_a_small_program():
    # r0 = input; op0: r1 = f(r0); op1: r2 = f(r1); op2: r3 = f(r2, r0); op3: r4 = f(r3); op4: r5 = f(r4, r3)
    start, end = planner.liveness([1, 2, 3, 4, 5], [[0], [1], [2, 0], [3], [4, 3]], 6)
    assert start == [-1, 0, 1, 2, 3, 4]
    assert end == [2, 1, 2, 4, 4, 4]   # the result r5 is never read: dead right after its writer


def test_buffer_reduction_ratio():
    assert planner.rho_buf(4, 2) == 0.5
    assert planner.rho_buf(10, 10) == 0.0
    assert abs(planner.rho_buf(100, 52) - 0.48) < 1e-12   # the upper end of the range the paper reports
