"""Pins for the oracle's placement solver (Algorithm 1) and streaming bookkeeping."""
import itertools
import os

import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def brute(s, r, c, M):
    best = None
    for b in itertools.product((O.HOST, O.GPU), repeat=len(s)):
        if sum(si for si, bi in zip(s, b) if bi == O.GPU) > M:
            continue
        v = O.placement_objective(b, r, c)
        best = v if best is None else max(best, v)
    return best


def test_objective_definition_by_hand():
    # r on GPU tensors minus c_i at each boundary where the backend changes (c_1 never counts)
    assert O.placement_objective([1, 0, 1], [5, 1, 5], [9, 3, 4]) == 10 - 3 - 4
    assert O.placement_objective([0, 0, 0], [5, 1, 5], [9, 3, 4]) == 0
    assert O.placement_objective([1, 1, 1], [5, 1, 5], [9, 3, 4]) == 11
    assert O.placement_objective([0, 1, 1], [5, 1, 5], [9, 3, 4]) == 6 - 3


def test_hand_worked_instances():
    for line in open(os.path.join(GOLD, "placement_small.txt")):
        if line.startswith("#") or not line.strip():
            continue
        M, s, r, c, opt, bvec = [p.strip() for p in line.split("|")]
        s, r, c = [list(map(int, v.split())) for v in (s, r, c)]
        b, val = O.solve_knapsack_dp(s, r, c, int(M))
        assert val == int(opt) == O.placement_objective(b, r, c), line
        assert sum(si for si, bi in zip(s, b) if bi == O.GPU) <= int(M)
        if bvec != "-":
            assert ["HG"[x] for x in b] == bvec.split(), line


def test_dp_equals_brute_force_on_random_instances():
    rng = np.random.default_rng(0)
    for trial in range(250):
        n = int(rng.integers(1, 11))
        s = rng.integers(1, 6, size=n).tolist()
        r = rng.integers(0, 20, size=n).tolist()
        c = rng.integers(0, 8, size=n).tolist() if trial % 3 else [0] * n
        M = int(rng.integers(0, sum(s) + 2))
        b, val = O.solve_knapsack_dp(s, r, c, M)
        assert val == brute(s, r, c, M), (s, r, c, M)
        assert val == O.placement_objective(b, r, c)
        assert sum(si for si, bi in zip(s, b) if bi == O.GPU) <= M


def test_dp_limits_and_monotonicity():
    s, r, c = [3, 2, 4, 1], [6, 5, 9, 1], [0, 1, 2, 1]
    assert O.solve_knapsack_dp(s, r, c, 0)[0] == [O.HOST] * 4
    assert O.solve_knapsack_dp(s, r, c, 10)[0] == [O.GPU] * 4
    vals = [O.solve_knapsack_dp(s, r, c, M)[1] for M in range(12)]
    assert all(a <= b for a, b in zip(vals, vals[1:]))
    # huge switch cost -> at most one backend change never pays -> no change at all unless everything fits
    b, _ = O.solve_knapsack_dp(s, r, [0, 10 ** 6, 10 ** 6, 10 ** 6], 9)
    assert len(set(b)) == 1
    # c = 0 is the textbook 0/1 knapsack: compare with the classic one-dimensional DP
    rng = np.random.default_rng(4)
    s = rng.integers(1, 9, size=14).tolist()
    r = rng.integers(1, 30, size=14).tolist()
    M = 25
    best = [0] * (M + 1)
    for si, ri in zip(s, r):
        for m in range(M, si - 1, -1):
            best[m] = max(best[m], best[m - si] + ri)
    assert O.solve_knapsack_dp(s, r, [0] * 14, M)[1] == best[M]


def test_moe_partition_rule_both_branches():
    #            non  exp  non  exp
    s = [2, 5, 3, 4]
    r = [4, 9, 5, 8]
    c = [0, 0, 0, 0]
    is_exp = [False, True, False, True]
    # budget covers the non-expert tensors (5): they go to the GPU, DP over experts with the rest (4)
    b = O.static_placement(s, r, c, 9, is_exp)
    assert b == [O.GPU, O.HOST, O.GPU, O.GPU]
    # budget below the non-expert total: experts all stay on the host, DP over non-experts
    b = O.static_placement(s, r, c, 4, is_exp)
    assert b == [O.HOST, O.HOST, O.GPU, O.HOST]
    # dense model: same as the plain DP
    assert O.static_placement(s, r, c, 9, None) == O.solve_knapsack_dp(s, r, c, 9)[0]


def test_units_round_sizes_up_and_budget_down():
    G = 1 << 20
    assert O.size_units([1, G, G + 1, 2359296], G) == [1, 1, 2, 3]
    assert O.budget_units(3 * G - 1, G) == 2


def test_32_layer_dense_stack_at_60_percent():
    """The 32-layer stack of the dense workload at a 60 % byte budget, sizes = values = bytes, c = 0.
    Independent cross-checks: the result fills the budget's 2246 MiB units exactly and equals the
    textbook knapsack optimum; the resident/streamed byte split (2,326,265,856 resident /
    1,599,602,688 streamed) was also obtained by an independent numpy knapsack over the same sizes."""
    shape = W.DENSE_FULL
    nbytes = [W.q4_bytes(n, k) for _ in range(32) for (_, n, k) in shape.tensor_shapes()]
    total = sum(nbytes)
    assert total == 3925868544
    budget = int(0.60 * total)
    assert budget == 2355521126
    s, M = O.size_units(nbytes), O.budget_units(budget)
    assert M == 2246
    b = O.static_placement(s, nbytes, [0] * len(s), M)
    used = sum(si for si, bi in zip(s, b) if bi == O.GPU)
    assert used <= M
    resident = sum(x for x, bi in zip(nbytes, b) if bi == O.GPU)
    best = [0] * (M + 1)
    for si, ri in zip(s, nbytes):
        for m in range(M, si - 1, -1):
            if best[m - si] + ri > best[m]:
                best[m] = best[m - si] + ri
    assert resident == best[M]
    assert resident == 2326265856 and total - resident == 1599602688
    assert resident <= budget


def test_streaming_bookkeeping():
    nbytes = [100, 40, 40, 100]
    where = [O.GPU, O.HOST, O.GPU, O.HOST]
    assert O.streamed_dense(nbytes, where, 64) == (140, 1 + 2, [1, 3])
    # MoE: distinct host-placed experts over the batch, ascending; gate,up per expert then the downs
    ids = np.array([[5, 2, 7], [2, 3, 5]])
    odd_host = [[O.HOST if e % 2 else O.GPU for e in range(8)]] * 3
    nb, copies, order = O.streamed_moe(ids, odd_host, [10, 10, 12], 8)
    assert order == [(0, 3), (1, 3), (0, 5), (1, 5), (0, 7), (1, 7), (2, 3), (2, 5), (2, 7)]
    assert nb == 3 * 32 and copies == 3 * (2 + 2 + 2)
    # nothing selected on the host -> nothing moves
    assert O.streamed_moe(np.array([[0, 2]]), odd_host, [10, 10, 12], 8) == (0, 0, [])
