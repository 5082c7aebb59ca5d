"""Pins for the oracle's dynamic transfer scheduling (Algorithm 2) and re-scheduling gate (Algorithm 3).

The dynamic program is checked against things it does not compute itself: an exhaustive enumeration of every admissible
plan evaluated with the latency T of Section 4.4.1 (a closed-form sum, written out separately), hand-worked instances,
special cases with closed forms, and monotonicity.  Inputs are integer-valued so every sum is exact."""
import itertools

import numpy as np
import pytest

from oracle import ats_oracle as O

H, G = O.HOST, O.GPU


def admissible_starts(rb, b, i):
    """Legal transfer start points of promoted tensor i (0-based): the round start if nothing before i is promoted, or a
    host tensor executed on the host with nothing promoted between it and i."""
    promoted = [k for k in range(len(b)) if b[k] == H and rb[k] == G]
    prev = max([k for k in promoted if k < i], default=None)
    out = [O.ROUND_START] if prev is None else []
    lo = 0 if prev is None else prev + 1
    out += [j for j in range(lo, i) if b[j] == H and rb[j] == H]
    return out


def brute(b, tg, th, c, w):
    """Minimum of T over every admissible (assignment, start points) pair, by enumeration."""
    n = len(b)
    hosts = [i for i in range(n) if b[i] == H]
    best = None
    for bits in itertools.product((H, G), repeat=len(hosts)):
        rb = list(b)
        for i, v in zip(hosts, bits):
            rb[i] = v
        promoted = [i for i in hosts if rb[i] == G]
        choices = [admissible_starts(rb, b, i) for i in promoted]
        if any(len(ch) == 0 for ch in choices):
            continue
        for pick in itertools.product(*choices):
            start = [O.NO_TRANSFER] * n
            for i, j in zip(promoted, pick):
                start[i] = j
            t = O.transfer_latency(rb, start, b, tg, th, c, w)
            best = t if best is None else min(best, t)
    return best


def check_plan(b, rb, start):
    for i in range(len(b)):
        if b[i] == G:
            assert rb[i] == G and start[i] == O.NO_TRANSFER
        elif rb[i] == G:
            assert start[i] in admissible_starts(rb, b, i)
        else:
            assert start[i] == O.NO_TRANSFER


def random_instance(rng, n):
    b = [int(v) for v in rng.integers(0, 2, size=n)]
    tg = [float(v) for v in rng.integers(1, 20, size=n)]
    th = [float(tg[i] + rng.integers(0, 60)) for i in range(n)]
    c = [float(v) for v in rng.integers(0, 8, size=n)]
    w = [float(v) for v in rng.integers(0, 80, size=n)]
    return b, tg, th, c, w


def test_seg_and_latency_by_hand():
    # tensors 1..4 default on GPU, host, host, GPU; seg(j, i) adds what runs strictly between j and i on the default path
    b, tg, th, c = [G, H, H, G], [5.0, 2.0, 3.0, 7.0], [0.0, 20.0, 30.0, 0.0], [99.0, 1.0, 2.0, 4.0]
    assert O.seg_window(0, 1, b, tg, th, c) == 0
    assert O.seg_window(0, 2, b, tg, th, c) == 5                      # tensor 1 on the GPU, no predecessor
    assert O.seg_window(0, 3, b, tg, th, c) == 5 + (20 + 1)           # + tensor 2 on the host and the switch into it
    assert O.seg_window(2, 4, b, tg, th, c) == 30                     # tensor 3 on the host, same backend as tensor 2
    assert O.seg_window(1, 4, b, tg, th, c) == (20 + 1) + 30
    w = [0.0, 9.0, 40.0, 0.0]
    # nothing promoted: the default path
    assert O.transfer_latency(b, [O.NO_TRANSFER] * 4, b, tg, th, c, w) == 5 + 1 + 20 + 30 + 4 + 7
    # tensor 3 promoted, its transfer started after tensor 2: nothing lies between, all 40 exposed
    assert O.transfer_latency([G, H, G, G], [O.NO_TRANSFER, O.NO_TRANSFER, 1, O.NO_TRANSFER], b, tg, th, c, w) == 5 + 1 + 20 + 2 + 3 + 7 + 40
    # tensor 2 promoted from the round start: 9 - 5 exposed; tensor 3 stays on the host
    assert O.transfer_latency([G, G, H, G], [O.NO_TRANSFER, O.ROUND_START, O.NO_TRANSFER, O.NO_TRANSFER], b, tg, th, c, w) == 5 + 2 + 2 + 30 + 4 + 7 + 4


def test_hand_worked_promotion_hidden_and_exposed():
    b, tg, th, c = [G, G, H, G], [5.0, 5.0, 2.0, 5.0], [0.0, 0.0, 20.0, 0.0], [0.0, 1.0, 1.0, 1.0]
    # the window before tensor 3 is 10: a transfer of 8 hides completely, one of 14 exposes 4, one of 40 is not worth it
    for w3, want_t, want_rb in ((8.0, 17.0, [G, G, G, G]), (14.0, 21.0, [G, G, G, G]), (40.0, 37.0, [G, G, H, G])):
        t, rb, start = O.dynamic_transfer(b, tg, th, c, [0.0, 0.0, w3, 0.0])
        assert (t, rb) == (want_t, want_rb)
        check_plan(b, rb, start)


def test_closed_forms():
    rng = np.random.default_rng(5)
    n = 9
    tg = [float(v) for v in rng.integers(1, 9, size=n)]
    th = [float(v) for v in rng.integers(10, 50, size=n)]
    c = [float(v) for v in rng.integers(0, 5, size=n)]
    # everything resident: the sum of the GPU times, no switch, no transfer
    t, rb, start = O.dynamic_transfer([G] * n, tg, th, c, [7.0] * n)
    assert t == sum(tg) and rb == [G] * n and start == [O.NO_TRANSFER] * n
    # transfers too slow to ever pay: the default path
    b = [int(v) for v in rng.integers(0, 2, size=n)]
    default = O.transfer_latency(b, [O.NO_TRANSFER] * n, b, tg, th, c, [0.0] * n)
    t, rb, _ = O.dynamic_transfer(b, tg, th, c, [1e9] * n)
    assert t == default and rb == b
    # all tensors on the host, free transfers, no switch cost, GPU 1 vs host 10: a promoted tensor needs a host-executed
    # start point after the previous promotion, so at best every other tensor is promoted (starting with the first)
    for m in (1, 2, 5, 6):
        t, rb, start = O.dynamic_transfer([H] * m, [1.0] * m, [10.0] * m, [0.0] * m, [0.0] * m)
        assert t == 1.0 * ((m + 1) // 2) + 10.0 * (m // 2)
        check_plan([H] * m, rb, start)


def test_dp_equals_exhaustive_minimum():
    rng = np.random.default_rng(11)
    for trial in range(300):
        n = int(rng.integers(1, 8))
        b, tg, th, c, w = random_instance(rng, n)
        t, rb, start = O.dynamic_transfer(b, tg, th, c, w)
        check_plan(b, rb, start)
        assert t == O.transfer_latency(rb, start, b, tg, th, c, w), (b, tg, th, c, w)
        assert t == brute(b, tg, th, c, w), (b, tg, th, c, w)


def test_invariants():
    rng = np.random.default_rng(12)
    for trial in range(200):
        n = int(rng.integers(2, 30))
        b, tg, th, c, w = random_instance(rng, n)
        t, rb, start = O.dynamic_transfer(b, tg, th, c, w)
        check_plan(b, rb, start)
        assert t == O.transfer_latency(rb, start, b, tg, th, c, w)
        # never worse than promoting nothing; faster transfers never hurt
        assert t <= O.transfer_latency(b, [O.NO_TRANSFER] * n, b, tg, th, c, w)
        assert O.dynamic_transfer(b, tg, th, c, [v / 2 for v in w])[0] <= t
        # starting every transfer at the latest legal point (the last host-executed tensor before it) exposes at least as much
        late = list(start)
        for i in range(n):
            if b[i] == H and rb[i] == G:
                late[i] = admissible_starts(rb, b, i)[-1]
        assert O.transfer_latency(rb, late, b, tg, th, c, w) >= t


def test_deviation_and_gate():
    assert O.deviation([10.0, 20.0, 0.0], [10.0, 20.0, 0.0]) == 0.0
    assert O.deviation([10.0, 20.0], [11.0, 17.0]) == pytest.approx(0.15)
    assert O.deviation([0.0, 5.0], [1.0, 5.0]) == float("inf")
    b = [G, H, G]
    snap = lambda th2, w2: ([5.0, 2.0, 5.0], [0.0, th2, 0.0], [0.0, 1.0, 1.0], [0.0, w2, 0.0])
    m_prev = snap(20.0, 4.0)
    rb_prev = O.dynamic_transfer(b, *m_prev)[1]
    assert rb_prev == [G, G, G]
    # the paper's settings: eps = 15 %, minimum interval 5 x TPOT (40 ms) = 200 ms
    eps, tau = 0.15, 200.0
    slow_link = snap(20.0, 400.0)  # the transfer got 100 x slower: staying on the host wins now
    assert O.dynamic_transfer(b, *slow_link)[1] == [G, H, G]
    rb, ref, t_last, did = O.reschedule(b, rb_prev, m_prev, snap(20.0, 4.5), eps, tau, 1000.0, 0.0)      # 12.5 % < eps
    assert (rb, ref, t_last, did) == (rb_prev, m_prev, 0.0, False)
    rb, ref, t_last, did = O.reschedule(b, rb_prev, m_prev, slow_link, eps, tau, 199.0, 0.0)             # too soon
    assert (rb, ref, t_last, did) == (rb_prev, m_prev, 0.0, False)
    rb, ref, t_last, did = O.reschedule(b, rb_prev, m_prev, slow_link, eps, tau, 200.0, 0.0)             # interval reached
    assert (rb, ref, t_last, did) == ([G, H, G], slow_link, 200.0, True)
    rb, ref, t_last, did = O.reschedule(b, rb_prev, m_prev, snap(23.0, 4.0), eps, tau, 500.0, 0.0)       # exactly eps: re-plans
    assert did and ref == snap(23.0, 4.0) and t_last == 500.0
