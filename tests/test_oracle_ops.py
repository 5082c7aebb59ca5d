"""Pins for the oracle's operator arithmetic: each check ties a function to something other than
itself (exact rational arithmetic, closed forms, invariants, library routines on special cases)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def frac16(v):
    return Fraction(float(np.float16(v)))


# ---------------------------------------------------------------- nibble layout / dequant (a1)
def test_nibble_golden_table():
    for line in open(os.path.join(GOLD, "nibbles.txt")):
        if line.startswith("#") or not line.strip():
            continue
        b, ce, co = line.split()
        got = O.unpack_codes(np.array([[int(b, 16)]], dtype=np.uint8))[0]
        assert (int(got[0]), int(got[1])) == (int(ce), int(co)), line


def test_all_256_bytes_roundtrip_through_generator_layout():
    allb = np.arange(256, dtype=np.uint8).reshape(1, 256)
    codes = O.unpack_codes(allb)
    assert codes.min() == -8 and codes.max() == 7
    assert np.array_equal(W.codes_to_packed(codes), allb)
    # every (even, odd) code pair appears exactly once
    pairs = set(zip(codes[0, 0::2].tolist(), codes[0, 1::2].tolist()))
    assert len(pairs) == 256


def test_dequant_exact_rational_and_block_indexing():
    rng = np.random.default_rng(1)
    codes = rng.integers(-8, 8, size=(3, 96), dtype=np.int8)
    scales = rng.normal(0, 0.02, size=(3, 3)).astype(np.float16)  # negative scales are legal
    w = O.dequantize(W.codes_to_packed(codes), scales)
    for n in range(3):
        for k in range(96):
            assert Fraction(float(w[n, k])) == frac16(scales[n, k // 32]) * int(codes[n, k])
    # exact in fp32 too (11-bit significand x 4-bit code)
    assert np.array_equal(w.astype(np.float32).astype(np.float64), w)


def test_dequant_zero_scale_block_is_zero_and_f16_mode_single_rounding():
    codes = np.full((2, 64), 7, dtype=np.int8)
    scales = np.array([[0.0, 0.01], [0.03, 0.0]], dtype=np.float16)
    w = O.dequantize(W.codes_to_packed(codes), scales)
    assert np.all(w[0, :32] == 0) and np.all(w[1, 32:] == 0) and np.all(w[0, 32:] != 0)
    # F16 mode: RN16 of the exact product; check against Fraction-based nearest search on a few scales
    for sbits in (0x0001, 0x03FF, 0x1234, 0x2D55, 0x3C01):
        s = np.array([[sbits]], dtype=np.uint16).view(np.float16)
        for code in (-8, -7, -3, 3, 5, 7):
            c = np.full((1, 32), code, dtype=np.int8)
            got = O.dequantize(W.codes_to_packed(c), s, O.WEIGHT_F16)[0, 0]
            exact = frac16(s[0, 0]) * code
            # nearest fp16 by brute force over the neighbours of the float64 value
            cand = np.float16(float(exact))
            nbrs = [np.nextafter(cand, np.float16(-np.inf)), cand, np.nextafter(cand, np.float16(np.inf))]
            best = min(abs(Fraction(float(x)) - exact) for x in nbrs)
            assert abs(Fraction(float(got)) - exact) == best


# ---------------------------------------------------------------- linear (a2, a3)
@pytest.mark.parametrize("N,K,M", [(1, 32, 1), (3, 64, 2), (17, 96, 3)])
def test_linear_exact_rational(N, K, M):
    rng = np.random.default_rng(N * 100 + K)
    codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    scales = np.abs(rng.normal(0, 0.02, size=(N, K // 32))).astype(np.float16)
    x = rng.normal(0, 1, size=(M, K)).astype(np.float16)
    y = O.linear(x, W.codes_to_packed(codes), scales)
    for m in range(M):
        for n in range(N):
            exact = sum(frac16(scales[n, k // 32]) * int(codes[n, k]) * frac16(x[m, k]) for k in range(K))
            assert abs(Fraction(float(y[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 45) + Fraction(1, 2 ** 60)


def test_linear_one_hot_picks_a_column_and_ones_give_row_sums():
    rng = np.random.default_rng(7)
    N, K = 5, 128
    codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    scales = np.abs(rng.normal(0, 0.02, size=(N, K // 32))).astype(np.float16)
    packed = W.codes_to_packed(codes)
    for k in (0, 1, 31, 32, 33, 127):
        x = np.zeros((1, K), dtype=np.float16)
        x[0, k] = 1
        y = O.linear(x, packed, scales)[0]
        want = scales[:, k // 32].astype(np.float64) * codes[:, k]
        assert np.array_equal(y, want), k
    ones_s = np.ones((N, K // 32), dtype=np.float16)
    y = O.linear(np.ones((1, K), dtype=np.float16), packed, ones_s)[0]
    assert np.array_equal(y, codes.astype(np.int64).sum(axis=1).astype(np.float64))


def test_linear_is_linear_in_activations_and_ignores_zero_scale_blocks():
    rng = np.random.default_rng(9)
    N, K = 8, 256
    packed, scales = W.q4_packed(90, 0, 0, N, K)
    x1 = rng.normal(0, 1, size=(2, K)).astype(np.float16)
    x2 = rng.normal(0, 1, size=(2, K)).astype(np.float16)
    a, b = 4.0, -0.5  # powers of two: scaling is exact
    lhs = O.linear(a * x1.astype(np.float64) + b * x2.astype(np.float64), packed, scales)
    rhs = a * O.linear(x1, packed, scales) + b * O.linear(x2, packed, scales)
    assert np.allclose(lhs, rhs, rtol=0, atol=1e-12)
    s0 = scales.copy()
    s0[:, 3] = 0
    xa = x1.copy()
    xb = x1.copy()
    xb[:, 96:128] = 100  # only touches the zero-scale block
    assert np.array_equal(O.linear(xa, packed, s0), O.linear(xb, packed, s0))


def test_standalone_output_rounding_is_fp16():
    packed, scales = W.q4_packed(90, 0, 1, 4, 64)
    x = W.activations(90, 0, (3, 64))
    y = O.linear(x, packed, scales, round_out=True)
    assert np.array_equal(y, y.astype(np.float16).astype(np.float64))


# ---------------------------------------------------------------- glue (a6)
def test_rmsnorm_closed_forms():
    # x = (3, 4): mean square 12.5 ; eps = 0
    h = O.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0)[0]
    assert np.allclose(h, [3 / np.sqrt(12.5), 8 / np.sqrt(12.5)], rtol=1e-15)
    # constant vector -> sign * gain (up to eps)
    g = np.array([0.5, -2.0, 3.0, 1.0])
    assert np.allclose(O.rmsnorm(np.full((1, 4), -7.0), g, 0.0)[0], -g, rtol=1e-15)
    # eps enters under the root: x = 0 stays 0, and eps = 3 with unit ms gives x/2
    assert np.allclose(O.rmsnorm(np.array([[1.0, -1.0]]), np.ones(2), 3.0)[0], [0.5, -0.5])


def test_rope_identities():
    rng = np.random.default_rng(3)
    d = 16
    u = rng.normal(size=(5, d))
    assert np.array_equal(O.rope(u, 0, 10000.0), u)  # position 0 is the identity
    assert np.array_equal(O.rope(u, 9, 0.0), u)  # theta = 0 disables
    # d = 2: a single pair rotated by the angle pos (theta^0 = 1)
    r = O.rope(np.array([1.0, 0.0]), 0.75, 10000.0)
    assert np.allclose(r, [np.cos(0.75), np.sin(0.75)], rtol=1e-15)
    # half-split pairing: element i pairs with i + d/2, frequency theta^(-2i/d)
    e = np.zeros(d)
    e[3] = 1.0
    r = O.rope(e, 5, 100.0)
    ang = 5 * 100.0 ** (-2 * 3 / d)
    want = np.zeros(d)
    want[3], want[3 + d // 2] = np.cos(ang), np.sin(ang)
    assert np.allclose(r, want, atol=1e-15)
    # norms preserved; <rope(q,m), rope(k,n)> depends on m - n only
    q, k = rng.normal(size=d), rng.normal(size=d)
    assert np.isclose(np.linalg.norm(O.rope(q, 37, 1e4)), np.linalg.norm(q))
    d1 = O.rope(q, 12, 1e4) @ O.rope(k, 5, 1e4)
    d2 = O.rope(q, 107, 1e4) @ O.rope(k, 100, 1e4)
    assert np.isclose(d1, d2, rtol=1e-12)
    # per-token positions broadcast: [T, heads, d] with pos [T, 1]
    uu = rng.normal(size=(3, 2, d))
    rr = O.rope(uu, np.array([[4.0], [5.0], [6.0]]), 1e4)
    assert np.allclose(rr[1, 1], O.rope(uu[1, 1], 5, 1e4))


def test_attention_special_cases():
    rng = np.random.default_rng(5)
    n_q, n_kv, d, cap = 4, 2, 8, 6
    q = rng.normal(size=(n_q, d))
    K = rng.normal(size=(n_kv, cap, d)).astype(np.float16)
    V = rng.normal(size=(n_kv, cap, d)).astype(np.float16)
    # one position: the output is that position's value, per kv group (heads 0,1 -> kv 0; 2,3 -> kv 1)
    a = O.attention_one(q, K, V, 1)
    assert np.array_equal(a[0], V[0, 0].astype(np.float64)) and np.array_equal(a[1], V[0, 0].astype(np.float64))
    assert np.array_equal(a[2], V[1, 0].astype(np.float64)) and np.array_equal(a[3], V[1, 0].astype(np.float64))
    # identical keys -> uniform weights -> mean of the values over the attended prefix only
    K2 = np.repeat(K[:, :1], cap, axis=1)
    a = O.attention_one(q, K2, V, 4)
    assert np.allclose(a[0], V[0, :4].astype(np.float64).mean(axis=0))
    assert np.allclose(a[3], V[1, :4].astype(np.float64).mean(axis=0))
    # scaling by 1/sqrt(d): two keys, scores s0, s1 -> weights from the logistic of (s0 - s1)/sqrt(d)
    a = O.attention_one(q, K, V, 2)
    s = (K[0, :2].astype(np.float64) @ q[1]) / np.sqrt(d)
    p0 = 1 / (1 + np.exp(s[1] - s[0]))
    assert np.allclose(a[1], p0 * V[0, 0].astype(np.float64) + (1 - p0) * V[0, 1].astype(np.float64))
    # softmax matches scipy's on random input
    from scipy.special import softmax as sp_softmax
    z = rng.normal(size=(3, 11)) * 30
    assert np.allclose(O.softmax(z), sp_softmax(z, axis=-1), rtol=1e-13)


def test_silu_and_swiglu():
    from scipy.special import expit
    z = np.linspace(-20, 20, 41)
    assert np.allclose(O.silu(z), z * expit(z), rtol=1e-14)
    assert O.silu(0.0) == 0.0


def _small_dense(seed_cfg=91, shape=W.DENSE_SMALL):
    L = W.dense_layer(seed_cfg, 0, shape)
    t = {"wq": L[W.ROLE_Q], "wk": L[W.ROLE_K], "wv": L[W.ROLE_V], "wo": L[W.ROLE_O],
         "w_gate": L[W.ROLE_GATE], "w_up": L[W.ROLE_UP], "w_down": L[W.ROLE_DOWN],
         "attn_norm": L[W.ROLE_ATTN_NORM], "ffn_norm": L[W.ROLE_FFN_NORM]}
    return t, shape


def test_prefill_equals_sequential_decode():
    """Pins the causal mask, append-before-attend and cache positions: a T-token prefill is
    T decode steps (same contract => equal up to fp64 rounding)."""
    t, shape = _small_dense()
    T, cap = 6, 16
    x = W.activations(91, 0, (T, shape.hidden))
    for edges in (frozenset(), frozenset(O.EDGES)):
        Kp, Vp = W.kv_cache(91, 0, shape.n_kv_heads, cap, shape.head_dim, 3)
        Ks, Vs = Kp.copy(), Vp.copy()
        yp = O.dense_layer(x, t, shape, Kp, Vp, 3, edges, O.WEIGHT_F16)
        ys = np.stack([O.dense_layer(x[i:i + 1], t, shape, Ks, Vs, 3 + i, edges, O.WEIGHT_F16)[0] for i in range(T)])
        assert np.array_equal(Kp, Ks) and np.array_equal(Vp, Vs)
        assert np.max(np.abs(yp.astype(np.float64) - ys.astype(np.float64))) <= 2 ** -8 * np.max(np.abs(ys.astype(np.float64)))
        # untouched cache positions stay as they were
        assert np.all(Kp[:, 3 + T:] == 0)


def test_dense_layer_with_zero_weights_is_identity_path():
    """All scales zero => every projection is 0 => y = x (pins the two residual adds), cache row = 0."""
    t, shape = _small_dense()
    tz = {k: ((v[0], np.zeros_like(v[1])) if isinstance(v, tuple) else v) for k, v in t.items()}
    x = W.activations(91, 0, (1, shape.hidden))
    K, V = W.kv_cache(91, 0, shape.n_kv_heads, 8, shape.head_dim, 2)
    y = O.dense_layer(x, tz, shape, K, V, 2)
    assert np.array_equal(y, x)
    assert np.all(K[:, 2] == 0) and np.all(V[:, 2] == 0)


def test_dense_layer_first_token_attention_is_own_value():
    """pos = 0: attention output is the token's own v, so the layer reduces to an expression the
    test assembles from the already-pinned linear/rmsnorm/silu pieces."""
    t, shape = _small_dense()
    x = W.activations(91, 0, (1, shape.hidden)).astype(np.float64)
    K, V = W.kv_cache(91, 0, shape.n_kv_heads, 4, shape.head_dim, 0)
    y = O.dense_layer(x, t, shape, K, V, 0)
    h = O.rmsnorm(x, t["attn_norm"], shape.rms_eps)
    v = O.rn16(O.linear(h, *t["wv"]))  # what the cache holds
    group = shape.n_q_heads // shape.n_kv_heads
    a = np.repeat(v.reshape(shape.n_kv_heads, shape.head_dim), group, axis=0).reshape(1, -1)
    x1 = x + O.linear(a, *t["wo"])
    h2 = O.rmsnorm(x1, t["ffn_norm"], shape.rms_eps)
    d = O.linear(O.silu(O.linear(h2, *t["w_gate"])) * O.linear(h2, *t["w_up"]), *t["w_down"])
    assert np.array_equal(y, (x1 + d).astype(np.float16))
    assert np.array_equal(V[:, 0].reshape(-1), v.reshape(-1).astype(np.float16))


# ---------------------------------------------------------------- routing (a4) and MoE (a5)
def test_topk_brute_force_ties_and_invariances():
    rng = np.random.default_rng(11)
    H, E, k, M = 64, 16, 4, 5
    Wr = rng.normal(0, 0.02, size=(H, E)).astype(np.float16)
    Wr[:, 9] = Wr[:, 2]  # exact tie between experts 2 and 9
    Wr[:, 13] = Wr[:, 2]
    h = rng.normal(size=(M, H)).astype(np.float16)
    ids, gates, logits = O.route_topk(h, Wr, k)
    for m in range(M):
        brute = sorted(range(E), key=lambda e: (-logits[m, e], e))[:k]
        assert ids[m].tolist() == brute
        if 2 in brute and 9 in brute:
            assert brute.index(2) < brute.index(9)
    assert np.allclose(gates.sum(axis=1), 1.0)
    assert np.all(gates[:, :-1] >= gates[:, 1:])
    # gates are the full softmax renormalised over the selected experts
    full = O.softmax(logits)
    sel = np.take_along_axis(full, ids.astype(np.int64), axis=1)
    assert np.allclose(gates, sel / sel.sum(axis=1, keepdims=True), rtol=1e-12)
    # force a tie inside the top-k: make the tied columns dominant
    Wr2 = Wr.copy()
    Wr2[:, [2, 9, 13]] = (h[0] * 0.05).astype(np.float16)[:, None]
    ids2, _, _ = O.route_topk(h[:1], Wr2, k)
    assert ids2[0, :3].tolist() == [2, 9, 13]
    assert O.min_rank_gap(np.array([[5.0, 3.0, 2.5, 0.0]]), 2) == 0.5


def _small_moe(cfg=92, shape=W.MOE_SMALL):
    B = W.moe_block(cfg, 0, shape)
    return {"w_gate": B[W.ROLE_GATE], "w_up": B[W.ROLE_UP], "w_down": B[W.ROLE_DOWN],
            "router": B[W.ROLE_ROUTER], "ffn_norm": B[W.ROLE_FFN_NORM]}, shape


def test_moe_identical_experts_equal_dense_ffn():
    t, shape = _small_moe()
    same = {k: v for k, v in t.items()}
    for name in ("w_gate", "w_up", "w_down"):
        p, s = t[name]
        same[name] = (np.repeat(p[:1], shape.n_experts, axis=0), np.repeat(s[:1], shape.n_experts, axis=0))
    x = W.activations(92, 0, (3, shape.hidden))
    y, ids, gates, _ = O.moe_block(x, same, shape, edges=frozenset())
    h = O.rmsnorm(x, t["ffn_norm"], shape.rms_eps)
    d = O.linear(O.silu(O.linear(h, t["w_gate"][0][0], t["w_gate"][1][0])) * O.linear(h, t["w_up"][0][0], t["w_up"][1][0]),
                 t["w_down"][0][0], t["w_down"][1][0])
    want = x.astype(np.float64) + d  # gates sum to one
    assert np.max(np.abs(y.astype(np.float64) - want)) <= 2 ** -10 * np.max(np.abs(want))


def test_moe_permuting_experts_permutes_ids_and_batch_rows_are_independent():
    t, shape = _small_moe()
    x = W.activations(92, 0, (4, shape.hidden))
    y, ids, gates, _ = O.moe_block(x, t, shape)
    perm = np.random.default_rng(2).permutation(shape.n_experts)  # new index e' holds old expert perm[e']
    tp = dict(t)
    for name in ("w_gate", "w_up", "w_down"):
        tp[name] = (t[name][0][perm], t[name][1][perm])
    tp["router"] = t["router"][:, perm]
    yp, idsp, gatesp, _ = O.moe_block(x, tp, shape)
    assert np.array_equal(perm[idsp], ids) and np.array_equal(gatesp, gates)
    assert np.array_equal(yp, y)
    y1, ids1, _, _ = O.moe_block(x[2:3], t, shape)
    assert np.array_equal(y1[0], y[2]) and np.array_equal(ids1[0], ids[2])


def test_moe_linear_matches_linear_per_slot():
    t, shape = _small_moe()
    x = W.activations(92, 0, (2, shape.hidden))
    ids = np.array([[3, 0], [5, 3]], dtype=np.int32)
    y = O.moe_linear(x, ids, *t["w_gate"])
    for m in range(2):
        for j in range(2):
            e = ids[m, j]
            assert np.array_equal(y[m, j], O.linear(x[m:m + 1], t["w_gate"][0][e], t["w_gate"][1][e], round_out=True)[0])
    xs = W.activations(92, 1, (2, 2, shape.ffn))
    y2 = O.moe_linear(xs, ids, *t["w_down"], x_per_slot=True)
    assert np.array_equal(y2[1, 0], O.linear(xs[1, 0][None], t["w_down"][0][5], t["w_down"][1][5], round_out=True)[0])


def test_embed_and_lm_head_closed_forms():
    """embed: with a power-of-two scale the looked-up row is the integer codes times that scale, for every id incl. repeats;
    a scale whose product needs rounding gives the fp16 nearest to the exact rational.  lm_head: with a unit gain and an
    input of constant magnitude c the normalised row is sign(x) * c / sqrt(c^2 + eps), so the logits are that factor times
    the signed row sums of the codes."""
    from fractions import Fraction
    rng = np.random.default_rng(3)
    V, Hd = 12, 64
    codes = rng.integers(-8, 8, size=(V, Hd)).astype(np.int64)
    nib = np.where(codes < 0, codes + 16, codes).astype(np.uint8)
    packed = (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)  # byte j: code 2j low nibble, 2j+1 high nibble
    scales = np.full((V, Hd // 32), 0.25, dtype=np.float16)
    ids = np.array([5, 0, 11, 5], dtype=np.int32)
    got = O.embed(ids, packed, scales)
    assert got.dtype == np.float16 and np.array_equal(got.astype(np.float64), codes[ids] * 0.25)
    s = np.float16(0.3333)  # code * s is not an fp16 number in general
    scales2 = np.full((V, Hd // 32), s, dtype=np.float16)
    got2 = O.embed(ids, packed, scales2).astype(np.float64)
    sf = Fraction(float(s))
    for m, t in enumerate(ids):
        for k in range(Hd):
            exact = sf * int(codes[t, k])
            cand = np.float16(float(exact))
            assert got2[m, k] == float(cand)  # float(exact) is exact here (15 significant bits): one rounding to fp16
    # lm_head
    c = 0.5
    eps = 1e-2
    x = (c * np.where(rng.random(Hd) < 0.5, -1.0, 1.0)).astype(np.float16)[None, :]
    gain = np.ones(Hd, dtype=np.float16)
    ones = np.ones((V, Hd // 32), dtype=np.float16)
    logits = O.lm_head(x, gain, eps, packed, ones)
    h = np.float64(np.float16(c / np.sqrt(c * c + eps)))  # the normalised magnitude, rounded to fp16 as the contract says
    want = (codes * np.sign(x.astype(np.float64))).sum(axis=1) * h
    assert np.array_equal(np.asarray(logits, dtype=np.float64)[0], O.rn16(want))


def test_linear_w16_exact_rational_and_special_cases():
    """fp16 weights: against exact rational arithmetic on a small case; one-hot activations pick a column; a row of the
    identity returns the activation; rounding of the standalone output happens once."""
    from fractions import Fraction
    rng = np.random.default_rng(9)
    N, K, M = 5, 16, 3
    w = rng.standard_normal((N, K)).astype(np.float16)
    x = rng.standard_normal((M, K)).astype(np.float16)
    got = O.linear_w16(x, w)
    for m in range(M):
        for n in range(N):
            exact = sum(Fraction(float(w[n, k])) * Fraction(float(x[m, k])) for k in range(K))
            assert abs(Fraction(float(got[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 45) + Fraction(1, 2 ** 60)
    e = np.zeros((1, K), dtype=np.float16)
    e[0, 7] = 1
    assert np.array_equal(O.linear_w16(e, w)[0], w[:, 7].astype(np.float64))
    assert np.array_equal(O.linear_w16(x, np.eye(K, dtype=np.float16)), x.astype(np.float64))
    y16 = O.linear_w16(x, w, round_out=True)
    assert np.array_equal(y16, O.rn16(got))


# ---------------------------------------------------------------- the microscaling 4-bit format (Section 5.1)
def test_mxfp4_golden_elements_and_scales():
    section = 0
    for line in open(os.path.join(GOLD, "mxfp4_elements.txt")):
        if line.startswith("# byte"):
            section = 1
        if line.startswith("#") or not line.strip():
            continue
        a, b = line.split()
        if section == 0:
            code = int(a, 2)
            for pos in (0, 1):  # the element in the low and in the high nibble of a byte
                packed = np.zeros((1, 16), dtype=np.uint8)
                packed[0, 3] = code << (4 * pos)
                w = O.dequantize(packed, np.array([[127]], dtype=np.uint8))[0]
                assert w[6 + pos] == float(b) and np.signbit(w[6 + pos]) == b.startswith("-"), line
                assert np.count_nonzero(w) == (1 if float(b) != 0 else 0)
        else:
            packed = np.full((1, 16), 0x22, dtype=np.uint8)  # every element 1.0
            w = O.dequantize(packed, np.array([[int(a)]], dtype=np.uint8))[0]
            assert np.all(w == float(b)), line


def test_mxfp4_integer_form_block_indexing_and_scale_steps():
    # twice the element is an integer: the magnitudes are 0 1 2 3 4 6 8 12 (an independent, all-integer statement)
    twice = [0, 1, 2, 3, 4, 6, 8, 12]
    rng = np.random.default_rng(31)
    packed = rng.integers(0, 256, size=(5, 48), dtype=np.uint8)   # K = 96: three blocks per row
    sb = rng.integers(100, 150, size=(5, 3), dtype=np.uint8)
    w = O.dequantize(packed, sb)
    for n in range(5):
        for k in range(96):
            nib = (int(packed[n, k // 2]) >> (4 * (k & 1))) & 15
            want = Fraction((-1 if nib & 8 else 1) * twice[nib & 7], 2) * Fraction(2) ** (int(sb[n, k // 32]) - 127)
            assert Fraction(float(w[n, k])) == want
    # one step of the scale byte doubles every weight of its block and nothing else
    sb2 = sb.copy()
    sb2[2, 1] += 1
    w2 = O.dequantize(packed, sb2)
    assert np.array_equal(w2[2, 32:64], 2 * w[2, 32:64])
    w2[2, 32:64] = w[2, 32:64]
    assert np.array_equal(w2, w)
    with pytest.raises(AssertionError):
        O.dequantize(packed, np.full((5, 3), 255, dtype=np.uint8))
    # the tensor-core operand mode rounds to fp16 like for the other format; for block exponents from -23 to 13 every weight
    # already is an fp16 value (0.5 * 2^-23 is the smallest subnormal, 6 * 2^13 is below the largest finite), so it changes nothing
    assert np.array_equal(O.dequantize(packed, sb, O.WEIGHT_F16), O.rn16(w))
    for lo, hi in ((104, 141), (104, 105), (140, 141)):
        sb3 = rng.integers(lo, hi, size=(5, 3), dtype=np.uint8)
        w3 = O.dequantize(packed, sb3)
        assert np.array_equal(O.dequantize(packed, sb3, O.WEIGHT_F16), w3) and np.all(np.isfinite(w3.astype(np.float16)))
        assert np.array_equal(w3.astype(np.float16).astype(np.float64), w3)
    assert not np.array_equal(O.rn16(O.dequantize(packed, np.full((5, 3), 103, dtype=np.uint8))), O.dequantize(packed, np.full((5, 3), 103, dtype=np.uint8)))


def test_mxfp4_linear_exact_rational():
    rng = np.random.default_rng(32)
    N, K, M = 6, 64, 3
    packed = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sb = rng.integers(118, 132, size=(N, K // 32), dtype=np.uint8)
    x = rng.standard_normal((M, K)).astype(np.float16)
    y = O.linear(x, packed, sb)
    twice = [0, 1, 2, 3, 4, 6, 8, 12]
    for m in range(M):
        for n in range(N):
            exact = Fraction(0)
            for k in range(K):
                nib = (int(packed[n, k // 2]) >> (4 * (k & 1))) & 15
                wv = Fraction((-1 if nib & 8 else 1) * twice[nib & 7], 2) * Fraction(2) ** (int(sb[n, k // 32]) - 127)
                exact += wv * Fraction(float(x[m, k]))
            assert abs(Fraction(float(y[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 45) + Fraction(1, 2 ** 60)
    # all elements 1.0 and unit scales: row sums of x
    ones = np.full((2, K // 2), 0x22, dtype=np.uint8)
    y1 = O.linear(x, ones, np.full((2, K // 32), 127, dtype=np.uint8))
    assert np.allclose(y1[:, 0], x.astype(np.float64).sum(axis=1), rtol=0, atol=1e-12)
