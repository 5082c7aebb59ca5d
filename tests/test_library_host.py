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
