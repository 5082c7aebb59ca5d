"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its host logic
(Algorithm 1, format repack) agrees with the oracle.  No GPU, no compute calls."""
import os
import re

import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _binding():
    from paper_2607_10183_b200 import build
    build.build()
    from paper_2607_10183_b200 import binding
    return binding


def test_library_exports_every_declared_symbol():
    B = _binding()
    header = open(os.path.join(ROOT, "include", "ats.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ats_[a-z0-9_]+)\s*\(", header))
    assert {"ats_register_tensor", "ats_set_placement", "ats_linear", "ats_moe_linear", "ats_layer_decode",
            "ats_layer_prefill"} <= declared
    for name in declared:
        assert hasattr(B.lib, name), f"{name} declared in ats.h but not exported"
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)


def test_struct_layouts_match_header_sizes():
    B = _binding()
    import ctypes as C
    assert C.sizeof(B.ats_config) == 72
    assert C.sizeof(B.ats_tensor_desc) == 40
    assert C.sizeof(B.ats_layer_desc) == 10 * 4 + 8 * 4 + 12
    assert C.sizeof(B.ats_stats) == 8 * 8 + 9 * 8 + 8 + 2 * 4 * B.ATS_STATS_LIST


def test_host_placement_matches_oracle_vector():
    B = _binding()
    rng = np.random.default_rng(3)
    for trial in range(200):
        n = int(rng.integers(1, 24))
        s = rng.integers(1, 7, size=n)
        r = rng.integers(0, 25, size=n)
        c = rng.integers(0, 9, size=n) if trial % 2 else np.zeros(n, dtype=np.int64)
        M = int(rng.integers(0, s.sum() + 2))
        exp = (rng.integers(0, 2, size=n).astype(bool) if trial % 5 == 0 else None)
        b, obj = B.host_solve_placement(s, r, c, M, exp)
        want = O.static_placement(s.tolist(), r.tolist(), c.tolist(), M, None if exp is None else exp.tolist())
        assert b.tolist() == want, (s, r, c, M, exp)
        assert obj == O.placement_objective(want, r.tolist(), c.tolist())


def test_host_placement_dense_stack_60_percent():
    B = _binding()
    nbytes = [W.q4_bytes(n, k) for _ in range(32) for (_, n, k) in W.DENSE_FULL.tensor_shapes()]
    s, M = O.size_units(nbytes), O.budget_units(int(0.60 * sum(nbytes)))
    b, _ = B.host_solve_placement(s, nbytes, [0] * len(s), M)
    assert b.tolist() == O.static_placement(s, nbytes, [0] * len(s), M)


def test_repack_round_trip_is_identity():
    B = _binding()
    packed, scales = W.q4_packed(93, 0, 0, 37, 96)
    sl = np.zeros(packed.size + scales.size * 2, dtype=np.uint8)
    assert B.ats_host_repack_q4(packed.ctypes.data, scales.ctypes.data, sl.ctypes.data, 37, 96) == 0
    p2, s2 = np.zeros_like(packed), np.zeros_like(scales)
    assert B.ats_host_unpack_q4(sl.ctypes.data, p2.ctypes.data, s2.ctypes.data, 37, 96) == 0
    assert np.array_equal(p2, packed) and np.array_equal(s2.view(np.uint16), scales.view(np.uint16))
    assert not np.array_equal(sl[:packed.size].reshape(packed.shape), packed)  # the internal order differs
    assert B.ats_host_repack_q4(packed.ctypes.data, scales.ctypes.data, sl.ctypes.data, 37, 40) == B.ATS_ERR_SHAPE


def test_group_pairs_is_the_stable_sort_by_expert():
    """Row order of the MoE prefill: against numpy's stable argsort, incl. empty experts, one expert taking everything,
    no pairs at all, and an id out of range."""
    from paper_2607_10183_b200 import binding as B
    rng = np.random.default_rng(4)
    for P, E in ((0, 4), (1, 1), (37, 5), (4096, 128), (300, 1024)):
        ids = rng.integers(0, E, size=P, dtype=np.int32)
        if P == 37:
            ids[:] = 3  # one expert takes every row
        order, pos, off, mx = B.host_group_pairs(ids, E)
        want = np.argsort(ids, kind="stable").astype(np.int32)
        assert np.array_equal(order, want)
        assert np.array_equal(pos[order], np.arange(P, dtype=np.int32))
        cnt = np.bincount(ids, minlength=E)
        assert np.array_equal(off, np.concatenate(([0], np.cumsum(cnt))).astype(np.int32))
        assert mx == (cnt.max() if P else 0)
    with pytest.raises(B.AtsError):
        B.host_group_pairs(np.array([0, 7], dtype=np.int32), 7)


def test_dynamic_transfer_matches_oracle():
    """Algorithm 2 in the library against the oracle: the optimal latency is unique and must agree exactly (integer-valued
    inputs: every sum is exact); the plan itself may differ among equally good ones, so it is checked for validity and for
    reaching that latency under the oracle's closed-form T.  Also real-valued inputs within rounding, and bad arguments."""
    B = _binding()
    rng = np.random.default_rng(21)
    for trial in range(150):
        n = int(rng.integers(1, 70))
        b = rng.integers(0, 2, size=n).astype(np.uint8)
        if trial % 10 == 0:
            b[:] = trial % 20 == 0  # all host / all resident
        tg = rng.integers(1, 20, size=n).astype(np.float64)
        th = tg + rng.integers(0, 60, size=n)
        c = rng.integers(0, 8, size=n).astype(np.float64)
        w = rng.integers(0, 120, size=n).astype(np.float64)
        want_t, want_rb, want_start = O.dynamic_transfer(list(b), list(tg), list(th), list(c), list(w))
        t, rb, start = B.host_dynamic_transfer(b, tg, th, c, w)
        assert t == want_t
        # the plan: resident tensors stay, start points are host tensors run on the host with no promotion in between
        last_promoted = -1
        for i in range(n):
            if b[i] == B.ATS_GPU:
                assert rb[i] == B.ATS_GPU and start[i] == B.ATS_NO_TRANSFER
            elif rb[i] == B.ATS_GPU:
                j = int(start[i])
                assert j == B.ATS_ROUND_START and last_promoted < 0 or (last_promoted < j < i and b[j] == B.ATS_HOST and rb[j] == B.ATS_HOST)
                last_promoted = i
            else:
                assert start[i] == B.ATS_NO_TRANSFER
        assert O.transfer_latency(list(rb), [int(v) for v in start], list(b), list(tg), list(th), list(c), list(w)) == want_t
        assert B.host_transfer_latency(rb, start, b, tg, th, c, w) == want_t
        assert B.host_transfer_latency(want_rb, want_start, b, tg, th, c, w) == want_t
        # the default path through the library's evaluator
        none = np.full(n, B.ATS_NO_TRANSFER, np.int32)
        assert B.host_transfer_latency(b, none, b, tg, th, c, w) == O.transfer_latency(list(b), list(none), list(b), list(tg), list(th), list(c), list(w))
    # measured times are not integers: agreement within rounding of the sums
    for trial in range(30):
        n = int(rng.integers(2, 200))
        b = rng.integers(0, 2, size=n).astype(np.uint8)
        tg, th = rng.random(n) * 50e-6, rng.random(n) * 900e-6
        c, w = rng.random(n) * 20e-6, rng.random(n) * 400e-6
        want_t = O.dynamic_transfer(list(b), list(tg), list(th), list(c), list(w))[0]
        t, rb, start = B.host_dynamic_transfer(b, tg, th, c, w)
        assert abs(t - want_t) <= 1e-12 * want_t
        assert abs(B.host_transfer_latency(rb, start, b, tg, th, c, w) - t) <= 1e-12 * t
    # empty round; bad arguments
    t, rb, start = B.host_dynamic_transfer([], [], [], [], [])
    assert t == 0.0 and rb.size == 0
    one = np.array([1.0])
    with pytest.raises(B.AtsError):
        B.host_dynamic_transfer([2], one, one, one, one)           # not a backend
    with pytest.raises(B.AtsError):
        B.host_dynamic_transfer([0], one, -one, one, one)          # negative time
    with pytest.raises(B.AtsError):
        B.host_dynamic_transfer([0], one, one, one, one * np.nan)
    with pytest.raises(B.AtsError):
        B.host_transfer_latency([0], [B.ATS_NO_TRANSFER], [1], one, one, one, one)   # resident tensor moved to the host
    with pytest.raises(B.AtsError):
        B.host_transfer_latency([1], [0], [0], one, one, one, one)                   # start point not before the tensor


def test_reschedule_gate_matches_oracle():
    """Algorithm 3 in the library against the oracle over a sequence of snapshots with drifting load: same decisions, same
    reference snapshot, same clock; and the deviation measure on its special cases."""
    B = _binding()
    assert B.host_deviation([10.0, 20.0, 0.0], [10.0, 20.0, 0.0]) == 0.0
    assert B.host_deviation([10.0, 20.0], [11.0, 17.0]) == O.deviation([10.0, 20.0], [11.0, 17.0])
    assert B.host_deviation([0.0, 5.0], [1.0, 5.0]) == float("inf")
    rng = np.random.default_rng(22)
    n = 24
    b = rng.integers(0, 2, size=n).astype(np.uint8)
    base = [rng.integers(1, 20, size=n).astype(np.float64), rng.integers(20, 80, size=n).astype(np.float64),
            rng.integers(0, 8, size=n).astype(np.float64), rng.integers(0, 120, size=n).astype(np.float64)]
    eps, tau = 0.15, 200.0
    m_ref_o = tuple(list(p) for p in base)
    _, rb_o, _ = O.dynamic_transfer(list(b), *m_ref_o)
    t_last_o = 0.0
    m_ref = np.concatenate(base)
    _, rb, start = B.host_dynamic_transfer(b, *base)
    t_last = 0.0
    replans = 0
    for step in range(60):
        t_now = 40.0 * (step + 1)
        load = 1.0 + (0.5 if 20 <= step < 40 else 0.0) + 0.02 * (step % 3)  # a burst of host load in the middle
        cur = [base[0], np.round(base[1] * load), base[2], base[3] * (3.0 if step >= 45 else 1.0)]
        rb_o, m_ref_o, t_last_o, did_o = O.reschedule(list(b), rb_o, m_ref_o, tuple(list(p) for p in cur), eps, tau, t_now, t_last_o)
        t_last, did = B.host_reschedule(b, m_ref, np.concatenate(cur), eps, tau, t_now, t_last, rb, start)
        assert (did, t_last) == (did_o, t_last_o)
        assert np.array_equal(m_ref, np.concatenate([np.asarray(p, dtype=np.float64) for p in m_ref_o]))
        # equally good plans may differ; their latency under the current reference may not
        ref = [list(p) for p in m_ref_o]
        if did:
            assert B.host_transfer_latency(rb, start, b, *ref) == O.dynamic_transfer(list(b), *ref)[0]
        replans += did
    assert 2 <= replans <= 12  # the burst's start, its end and the slower link each trigger one; the rate limit holds the rest back
