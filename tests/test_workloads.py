"""The seeded generator is frozen and has the stated distributions."""
import importlib.util
import os

import numpy as np

from paper_2607_10183_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_generator_is_frozen():
    spec = importlib.util.spec_from_file_location("mk", os.path.join(GOLD, "make_generator_hash.py"))
    mk = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mk)
    want = dict(line.split() for line in open(os.path.join(GOLD, "generator_sha256.txt")))
    assert mk.digests() == want


def test_distributions_and_sizes():
    packed, scales = W.q4_packed(1, 0, W.ROLE_Q, 4096, 4096)
    assert packed.shape == (4096, 2048) and scales.shape == (4096, 128) and scales.dtype == np.float16
    lo, hi = packed & 0xF, packed >> 4
    for nib in (lo, hi):
        counts = np.bincount(nib.reshape(-1), minlength=16) / nib.size
        assert np.all(np.abs(counts - 1 / 16) < 2e-3)  # every code equally likely
    assert np.all(scales >= 0) and abs(float(scales.astype(np.float64).std()) - 0.02 * np.sqrt(1 - 2 / np.pi)) < 1e-3
    assert W.q4_bytes(4096, 4096) == 9437184
    assert sum(W.q4_bytes(n, k) for _, n, k in W.DENSE_FULL.tensor_shapes()) == 122683392
    assert W.q4_bytes(768, 2048) == 884736
    x = W.activations(1, 0, (1, 4096))
    assert x.dtype == np.float16 and abs(float(x.astype(np.float64).std()) - 1) < 0.05
