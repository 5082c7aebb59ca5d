"""CPU oracle for the block-quantized per-tensor forward path and its placement.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, fp64 statement of what
the CUDA library computes.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import it; the product never does.  It shares
no code with the CUDA path and does not import the package.

What it follows
---------------
The paper schedules *tensors*: each weight tensor is one operator executed on
the backend that holds (or receives) it (Section 3, Section 4.3.1); a GPU memory
budget M and a placement b decide which tensors are resident (Section 4.3.2,
the placement objective and Algorithm 1); the others sit in pinned host memory
and are moved into temporary GPU buffers on a transfer stream (Section 4.2.1,
4.2.2), and for MoE operators only the experts the current tokens selected are
moved (Section 4.2.2, Section 4.4.1).  The paper inherits the operator
arithmetic itself from its host framework and never states it; the formulas
below are therefore the workload definition's ("signed 4-bit codes in blocks of
32 along K with one fp16 scale per block, fp32 accumulation, fp16 output",
RMSNorm, rotary embedding, grouped-query attention, SwiGLU, softmax top-k
routing with ties to the lower index), written as their textbook definitions.

Pins (tests/test_oracle_*.py): exact rational arithmetic on tiny shapes,
one-hot / all-ones closed forms, linearity, zero-scale blocks, RoPE identities,
attention special cases, sort-based top-k, 2^n brute force of the placement
objective, prefill == sequential decode.  No function here is "parity unpinned".

Conventions: fp64 everywhere; ``rn16`` (IEEE round-to-nearest-even to binary16,
subnormals kept) is applied only at the edges named in ``edges`` (the numerics
contract the library publishes), at K/V cache writes and at the layer output.
"""
from __future__ import annotations

import numpy as np

BLOCK = 32

# Edges of a decoder layer at which a value may be rounded to fp16 (bit i of the contract mask).
EDGES = ("h", "q", "k", "v", "q_rot", "a", "o", "x1", "h2", "g", "u", "act", "d")
EDGE_BIT = {name: 1 << i for i, name in enumerate(EDGES)}
WEIGHT_EXACT, WEIGHT_F16 = 0, 1


def edges_from_mask(mask: int):
    return frozenset(n for n in EDGES if mask & EDGE_BIT[n])


def rn16(a):
    """Round fp64 values to the nearest fp16 (ties to even, subnormals kept); returned as fp64."""
    with np.errstate(over="ignore"):
        return np.asarray(a, dtype=np.float64).astype(np.float16).astype(np.float64)


def _edge(val, name, edges):
    return rn16(val) if name in edges else val


# --------------------------------------------------------------------------------------
# a1: block dequantization
# --------------------------------------------------------------------------------------
def unpack_codes(packed: np.ndarray) -> np.ndarray:
    """Interchange bytes ``[..., K/2]`` -> signed codes int8 ``[..., K]``.

    Byte j holds code 2j in bits 0..3 and code 2j+1 in bits 4..7, each a
    two's-complement nibble (0..7 -> 0..7, 8..15 -> -8..-1).
    """
    p = np.asarray(packed, dtype=np.uint8)
    lo = (p & 0x0F).astype(np.int8)
    hi = (p >> 4).astype(np.int8)
    lo = np.where(lo >= 8, lo - 16, lo).astype(np.int8)
    hi = np.where(hi >= 8, hi - 16, hi).astype(np.int8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


def dequantize(packed: np.ndarray, scales: np.ndarray, weight_mode: int = WEIGHT_EXACT) -> np.ndarray:
    """w[n,k] = scale[n, k // 32] * code[n,k]  (exact in fp64 and in fp32: 11-bit x 4-bit).

    ``WEIGHT_F16`` rounds that product once to fp16 (what a tensor-core operand holds).
    """
    if np.asarray(scales).dtype == np.uint8:  # shared-exponent bytes: the microscaling 4-bit format
        w = dequantize_mxfp4(packed, scales)
        return rn16(w) if weight_mode == WEIGHT_F16 else w
    codes = unpack_codes(packed).astype(np.float64)
    s = np.asarray(scales, dtype=np.float16).astype(np.float64)
    assert codes.shape[-1] == s.shape[-1] * BLOCK, "one scale per 32 consecutive k"
    w = codes * np.repeat(s, BLOCK, axis=-1)
    return rn16(w) if weight_mode == WEIGHT_F16 else w


def dequantize_mxfp4(packed: np.ndarray, scales_e8m0: np.ndarray) -> np.ndarray:
    """MXFP4, the other 4-bit format the paper evaluates (Section 5.1): blocks of 32 elements along K, each element a
    4-bit float (1 sign, 2 exponent, 1 mantissa bit; exponent bias 1), one shared power-of-two scale per block stored as
    a biased 8-bit exponent.  Written from the definition of the microscaling formats:

      element: s e1 e0 m  ->  (-1)^s * (m / 2            if e = 0   (subnormal)
                                        2^(e-1) * (1 + m/2) otherwise), e = 2 e1 + e0
      scale:   X = 2^(byte - 127), byte 255 = not a number (rejected)
      w[n,k] = X[n, k // 32] * element[n,k]

    Bytes are packed like the other 4-bit format: byte j of a row holds element 2j in bits 0..3 and element 2j+1 in
    bits 4..7.  Every w is a small integer times a power of two, exact in fp64 (and in fp16 for |exponent| small)."""
    p = np.asarray(packed, dtype=np.uint8)
    nib = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    nib[..., 0::2] = p & 0x0F
    nib[..., 1::2] = p >> 4
    sign = np.where(nib & 8, -1.0, 1.0)
    e = ((nib >> 1) & 3).astype(np.int64)
    m = (nib & 1).astype(np.float64)
    mag = np.where(e == 0, m / 2.0, np.ldexp(1.0 + m / 2.0, e - 1))
    sb = np.asarray(scales_e8m0, dtype=np.uint8)
    assert not np.any(sb == 255), "a block scale of 255 encodes NaN"
    assert nib.shape[-1] == sb.shape[-1] * BLOCK, "one scale per 32 consecutive k"
    scale = np.ldexp(1.0, sb.astype(np.int64) - 127)
    return sign * mag * np.repeat(scale, BLOCK, axis=-1)


# --------------------------------------------------------------------------------------
# a2 / a3: the per-tensor operator (GEMV for decode, GEMM for prefill)
# --------------------------------------------------------------------------------------
def linear(x: np.ndarray, packed: np.ndarray, scales: np.ndarray, weight_mode: int = WEIGHT_EXACT,
           round_out: bool = False) -> np.ndarray:
    """y[m,n] = sum_k w[n,k] x[m,k] in fp64; ``round_out`` gives the fp16 output of the standalone op."""
    w = dequantize(packed, scales, weight_mode)
    y = np.asarray(x, dtype=np.float64) @ w.T
    return rn16(y) if round_out else y


def linear_w16(x: np.ndarray, w16: np.ndarray, round_out: bool = False) -> np.ndarray:
    """The per-tensor operator for an unquantized fp16 weight matrix [N][K] (the paper runs one of its models with
    FP16 weights): y[m,n] = sum_k w[n,k] x[m,k] in fp64 over the fp16 values as they are."""
    w = np.asarray(w16, dtype=np.float16).astype(np.float64)
    y = np.asarray(x, dtype=np.float64) @ w.T
    return rn16(y) if round_out else y


def apply_weight(x, w, weight_mode: int = WEIGHT_EXACT) -> np.ndarray:
    """The per-tensor operator for a layer's weight given either as (packed, scales) (block-quantized) or as a
    1-tuple (w16,) holding an unquantized fp16 matrix."""
    if len(w) == 1:
        return linear_w16(x, w[0])
    return linear(x, w[0], w[1], weight_mode)


# --------------------------------------------------------------------------------------
# a6: layer glue
# --------------------------------------------------------------------------------------
def embed(token_ids, packed: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """Embedding lookup in a block-quantized table [vocab][hidden]: row t is the dequantized row rounded
    once to fp16 (the model's residual stream starts as fp16).  Returns fp16 [M, hidden]."""
    w = dequantize(packed, scales, WEIGHT_F16)  # rn16(scale * code) per element
    return np.asarray(w[np.asarray(token_ids, dtype=np.int64)], dtype=np.float16)


def lm_head(x, gain: np.ndarray, eps: float, packed: np.ndarray, scales: np.ndarray, weight_mode: int = WEIGHT_EXACT) -> np.ndarray:
    """Final RMSNorm (rounded to fp16: the contract's edge "h") and the vocabulary projection; logits fp16."""
    h = rn16(rmsnorm(np.asarray(x, dtype=np.float64), gain, eps))
    return linear(h, packed, scales, weight_mode, round_out=True)


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """h_i = x_i g_i / sqrt(mean_j x_j^2 + eps), per row."""
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(gain, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * g / np.sqrt(ms + eps)


def rope(u: np.ndarray, pos, theta: float) -> np.ndarray:
    """Rotary embedding, half-split pairing, on the last axis (head_dim d).

    For i < d/2 the pair (u_i, u_{i+d/2}) is rotated by the angle pos * theta^(-2i/d).
    ``pos`` broadcasts against u's leading axes (scalar, or [T,1] for [T,heads,d]).
    ``theta == 0`` disables the rotation.
    """
    u = np.asarray(u, dtype=np.float64)
    if theta == 0:
        return u.copy()
    d = u.shape[-1]
    half = d // 2
    i = np.arange(half, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta ** (-2.0 * i / d)
    c, s = np.cos(ang), np.sin(ang)
    a, b = u[..., :half], u[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def softmax(s: np.ndarray) -> np.ndarray:
    s = np.asarray(s, dtype=np.float64)
    e = np.exp(s - np.max(s, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def attention_one(q_heads: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray, n_ctx: int) -> np.ndarray:
    """Grouped-query attention of ONE token over cache positions 0..n_ctx-1.

    q_heads [n_q][d]; caches [n_kv][capacity][d].  Query head hq reads kv head hq // (n_q / n_kv).
    Scores are scaled by 1/sqrt(d); softmax is max-subtracted.
    """
    n_q, d = q_heads.shape
    n_kv = k_cache.shape[0]
    group = n_q // n_kv
    out = np.empty((n_q, d), dtype=np.float64)
    for hq in range(n_q):
        kvh = hq // group
        kk = np.asarray(k_cache[kvh, :n_ctx], dtype=np.float64)
        vv = np.asarray(v_cache[kvh, :n_ctx], dtype=np.float64)
        p = softmax(kk @ q_heads[hq] / np.sqrt(d))
        out[hq] = p @ vv
    return out


def silu(z):
    z = np.asarray(z, dtype=np.float64)
    return z / (1.0 + np.exp(-z))


def swiglu_ffn(h2, w_gate, w_up, w_down, edges, weight_mode):
    """d = W_down (silu(W_gate h2) * (W_up h2)) with the contract's roundings."""
    g = _edge(apply_weight(h2, w_gate, weight_mode), "g", edges)
    u = _edge(apply_weight(h2, w_up, weight_mode), "u", edges)
    act = _edge(silu(g) * u, "act", edges)
    return _edge(apply_weight(act, w_down, weight_mode), "d", edges)


def attention_block(x, tensors: dict, shape, k_cache: np.ndarray, v_cache: np.ndarray, pos0: int,
                    edges=frozenset(), weight_mode: int = WEIGHT_EXACT):
    """The attention half of a decoder layer over T = x.shape[0] tokens at positions pos0..pos0+T-1:
    x1 = x + W_o attention(RoPE(W_q h), cache), h = RMSNorm(x).

    The new keys/values are written to the caches (as fp16) first, then the token at position p
    attends to positions 0..p.  ``tensors`` maps 'wq','wk','wv','wo' to (packed, scales) and
    'attn_norm' to an fp16 gain.  The caches (fp16, [n_kv][capacity][d]) are updated in place.
    Returns x1 (fp64 values, rounded to fp16 when 'x1' is an edge).
    """
    x = np.asarray(x, dtype=np.float64)
    T = x.shape[0]
    nq, nkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    h = _edge(rmsnorm(x, tensors["attn_norm"], shape.rms_eps), "h", edges)
    q = _edge(apply_weight(h, tensors["wq"], weight_mode), "q", edges).reshape(T, nq, d)
    k = _edge(apply_weight(h, tensors["wk"], weight_mode), "k", edges).reshape(T, nkv, d)
    v = _edge(apply_weight(h, tensors["wv"], weight_mode), "v", edges).reshape(T, nkv, d)
    pos = (pos0 + np.arange(T, dtype=np.float64)).reshape(T, 1)
    q_rot = _edge(rope(q, pos, shape.rope_theta), "q_rot", edges)
    k_rot = rope(k, pos, shape.rope_theta)
    for t in range(T):
        k_cache[:, pos0 + t, :] = k_rot[t].astype(np.float16)
        v_cache[:, pos0 + t, :] = v[t].astype(np.float16)
    a = np.empty((T, nq * d), dtype=np.float64)
    for t in range(T):
        a[t] = attention_one(q_rot[t], k_cache, v_cache, pos0 + t + 1).reshape(-1)
    a = _edge(a, "a", edges)
    o = _edge(apply_weight(a, tensors["wo"], weight_mode), "o", edges)
    return _edge(x + o, "x1", edges)


def dense_layer(x, tensors: dict, shape, k_cache: np.ndarray, v_cache: np.ndarray, pos0: int,
                edges=frozenset(), weight_mode: int = WEIGHT_EXACT):
    """One dense decoder layer over T = x.shape[0] tokens at positions pos0..pos0+T-1: the attention
    block, then y = x1 + W_down(silu(W_gate h2) * (W_up h2)), h2 = RMSNorm(x1).

    T == 1 is a decode step, T > 1 a prefill chunk; both are the same definition.  ``tensors`` maps
    'wq','wk','wv','wo','w_gate','w_up','w_down' to (packed, scales) and 'attn_norm','ffn_norm' to
    fp16 gains.  The caches are updated in place.  Returns y as fp16.
    """
    x1 = attention_block(x, tensors, shape, k_cache, v_cache, pos0, edges, weight_mode)
    h2 = _edge(rmsnorm(x1, tensors["ffn_norm"], shape.rms_eps), "h2", edges)
    dd = swiglu_ffn(h2, tensors["w_gate"], tensors["w_up"], tensors["w_down"], edges, weight_mode)
    return (x1 + dd).astype(np.float16)


def moe_layer(x, attn_tensors: dict, attn_shape, moe_tensors: dict, moe_shape, k_cache: np.ndarray, v_cache: np.ndarray,
              pos0: int, edges=frozenset(), weight_mode: int = WEIGHT_EXACT):
    """A decoder layer whose FFN is the MoE block: the attention block, then moe_block on x1.
    Returns (y fp16, ids, gates, logits)."""
    x1 = attention_block(x, attn_tensors, attn_shape, k_cache, v_cache, pos0, edges, weight_mode)
    return moe_block(x1, moe_tensors, moe_shape, edges, weight_mode)


# --------------------------------------------------------------------------------------
# a4: router + top-k
# --------------------------------------------------------------------------------------
def route_topk(h: np.ndarray, router_w: np.ndarray, k: int):
    """logits = h W_r (W_r fp16 [hidden][E]); ids = the k largest logits in descending order,
    equal logits -> lower expert index first; gates = softmax over those k logits.

    Returns (ids int32 [M,k], gates fp64 [M,k], logits fp64 [M,E]).
    """
    logits = np.asarray(h, dtype=np.float64) @ np.asarray(router_w, dtype=np.float16).astype(np.float64)
    order = np.argsort(-logits, axis=-1, kind="stable")  # stable: ties keep ascending index
    ids = order[:, :k].astype(np.int32)
    top = np.take_along_axis(logits, ids.astype(np.int64), axis=-1)
    return ids, softmax(top), logits


def min_rank_gap(logits: np.ndarray, k: int) -> float:
    """Smallest gap between adjacent sorted logits among ranks 1..k+1 (degenerate seeds have tiny gaps)."""
    s = -np.sort(-np.asarray(logits, dtype=np.float64), axis=-1)[:, : k + 1]
    return float(np.min(s[:, :-1] - s[:, 1:]))


# --------------------------------------------------------------------------------------
# a5: grouped-expert FFN (the MoE block)
# --------------------------------------------------------------------------------------
def moe_linear(x, ids, packed, scales, x_per_slot: bool = False, weight_mode: int = WEIGHT_EXACT,
               round_out: bool = True):
    """y[m,j,:] = W[ids[m,j]] x[m(,j),:] on a stacked expert tensor (packed [E][N][K/2])."""
    x = np.asarray(x, dtype=np.float64)
    M, k = ids.shape
    n_out = packed.shape[1]
    y = np.empty((M, k, n_out), dtype=np.float64)
    for m in range(M):
        for j in range(k):
            e = int(ids[m, j])
            xv = x[m, j] if x_per_slot else x[m]
            y[m, j] = linear(xv[None, :], packed[e], scales[e], weight_mode)[0]
    return rn16(y) if round_out else y


def moe_block(x, tensors: dict, shape, edges=frozenset({"h2", "act"}), weight_mode: int = WEIGHT_EXACT):
    """MoE FFN block: y = x + sum_j gate_j * FFN_{e_j}(h), h = RMSNorm(x), summed in rank order.

    ``tensors``: 'ffn_norm' gain, 'router' fp16 [hidden][E], 'w_gate','w_up','w_down' stacked (packed, scales).
    Returns (y fp16 [M,hidden], ids, gates, logits).
    """
    x = np.asarray(x, dtype=np.float64)
    M = x.shape[0]
    h = _edge(rmsnorm(x, tensors["ffn_norm"], shape.rms_eps), "h2", edges)
    ids, gates, logits = route_topk(h, tensors["router"], shape.top_k)
    y = np.empty_like(x)
    for m in range(M):
        acc = x[m].copy()
        for j in range(shape.top_k):
            e = int(ids[m, j])
            wg = (tensors["w_gate"][0][e], tensors["w_gate"][1][e])
            wu = (tensors["w_up"][0][e], tensors["w_up"][1][e])
            wd = (tensors["w_down"][0][e], tensors["w_down"][1][e])
            dj = swiglu_ffn(h[m][None, :], wg, wu, wd, edges, weight_mode)[0]
            acc = acc + gates[m, j] * dj
        y[m] = acc
    return y.astype(np.float16), ids, gates, logits


# --------------------------------------------------------------------------------------
# a7: static placement (Algorithm 1 and the placement objective of Section 4.3.2)
# --------------------------------------------------------------------------------------
HOST, GPU = 0, 1
_NEG = -(1 << 62)


def placement_objective(b, r, c) -> int:
    """sum_i r_i [b_i = GPU] - sum_{i>=2} c_i [b_i != b_{i-1}]   (Section 4.3.2)."""
    val = 0
    for i in range(len(b)):
        if b[i] == GPU:
            val += int(r[i])
        if i > 0 and b[i] != b[i - 1]:
            val -= int(c[i])
    return val


def size_units(nbytes, granule: int = 1 << 20):
    """s_i = ceil(bytes_i / G): sizes round up so a unit-feasible placement is byte-feasible."""
    return [-(-int(b) // granule) for b in nbytes]


def budget_units(budget_bytes: int, granule: int = 1 << 20) -> int:
    """M = floor(budget / G)."""
    return int(budget_bytes) // granule


def solve_knapsack_dp(s, r, c, M: int):
    """The dense-model solver of Algorithm 1: knapsack over memory units with a penalty c_i
    whenever tensors i-1 and i get different backends; placement recovered by backtracking.

    State V[i][m][B] = best objective of tensors 1..i using at most m units with b_i = B.
    Ties keep the *same-backend* predecessor; at the end a tie between the two final states
    keeps HOST.  All integers.  Returns (b list of HOST/GPU, objective).
    """
    n = len(s)
    if n == 0:
        return [], 0
    M = max(int(M), 0)
    VH = np.zeros((n, M + 1), dtype=np.int64)
    VG = np.full((n, M + 1), _NEG, dtype=np.int64)
    predH = np.zeros((n, M + 1), dtype=np.int8)  # backend of tensor i-1 on the best path into (i, m, H)
    predG = np.zeros((n, M + 1), dtype=np.int8)
    for i in range(n):
        si, ri, ci = int(s[i]), int(r[i]), int(c[i])
        for m in range(M + 1):
            if i == 0:
                VH[i, m] = 0
                if m >= si:
                    VG[i, m] = ri
                continue
            same, other = VH[i - 1, m], VG[i - 1, m]
            other = other - ci if other > _NEG // 2 else _NEG
            if same >= other:
                VH[i, m], predH[i, m] = same, HOST
            else:
                VH[i, m], predH[i, m] = other, GPU
            if m >= si:
                same, other = VG[i - 1, m - si], VH[i - 1, m - si] - ci
                if same > _NEG // 2 and same >= other:
                    VG[i, m], predG[i, m] = ri + same, GPU
                else:
                    VG[i, m], predG[i, m] = ri + other, HOST
    b = [HOST] * n
    m = M
    cur = HOST if VH[n - 1, M] >= VG[n - 1, M] else GPU
    best = int(max(VH[n - 1, M], VG[n - 1, M]))
    for i in range(n - 1, -1, -1):
        b[i] = cur
        if cur == GPU:
            nxt = predG[i, m]
            m -= int(s[i])
        else:
            nxt = predH[i, m]
        cur = int(nxt)
    return b, best


def static_placement(s, r, c, M: int, is_expert=None):
    """Algorithm 1.  Dense model: the DP over all tensors.  MoE model (some ``is_expert``):
    if the non-expert tensors fit, they all go to the GPU and the DP runs over the expert
    tensors with the remaining budget; otherwise every expert tensor stays on the host and
    the DP runs over the non-expert tensors with the whole budget."""
    n = len(s)
    if is_expert is None or not any(is_expert):
        return solve_knapsack_dp(s, r, c, M)[0]
    exp = [i for i in range(n) if is_expert[i]]
    non = [i for i in range(n) if not is_expert[i]]
    s_non = sum(int(s[i]) for i in non)
    b = [HOST] * n
    if M >= s_non:
        for i in non:
            b[i] = GPU
        sub, rest = exp, M - s_non
    else:
        sub, rest = non, M
    sol, _ = solve_knapsack_dp([s[i] for i in sub], [r[i] for i in sub], [c[i] for i in sub], rest)
    for i, bi in zip(sub, sol):
        b[i] = bi
    return b


# --------------------------------------------------------------------------------------
# a8 / a9: streaming bookkeeping of one call
# --------------------------------------------------------------------------------------
def streamed_dense(tensor_bytes, where, chunk_bytes: int):
    """Tensors of one call in execution order; those placed on the host are streamed whole.
    Returns (bytes_streamed, copies, indices_streamed)."""
    idx = [i for i, w in enumerate(where) if w == HOST]
    nbytes = sum(int(tensor_bytes[i]) for i in idx)
    copies = sum(-(-int(tensor_bytes[i]) // chunk_bytes) for i in idx)
    return nbytes, copies, idx


def streamed_moe(ids: np.ndarray, expert_where, slice_bytes, chunk_bytes: int):
    """Only the experts selected by the current tokens move (Section 4.2.2): the distinct
    host-placed experts over the batch, ascending, each contributing its gate, up and down slice.

    ``expert_where[t][e]`` for t in (gate, up, down); ``slice_bytes[t]`` bytes of one expert slice.
    Returns (bytes_streamed, copies, [(tensor, expert), ...] in issue order: gate_e, up_e for each
    expert, then down_e for each expert).
    """
    sel = sorted(set(int(e) for e in np.asarray(ids).reshape(-1)))
    order = []
    for e in sel:
        for t in (0, 1):
            if expert_where[t][e] == HOST:
                order.append((t, e))
    for e in sel:
        if expert_where[2][e] == HOST:
            order.append((2, e))
    nbytes = sum(int(slice_bytes[t]) for t, _ in order)
    copies = sum(-(-int(slice_bytes[t]) // chunk_bytes) for t, _ in order)
    return nbytes, copies, order


# --------------------------------------------------------------------------------------
# f2: dynamic transfer scheduling (Algorithm 2) and the re-scheduling gate (Algorithm 3)
# --------------------------------------------------------------------------------------
# Tensors are numbered 1..n in execution order as in Section 4.4; the Python lists are 0-based, so
# tensor i is element i-1.  Backends are HOST (the paper's CPU) and GPU.  Readings the text leaves
# open (each is listed with the design's other readings):
#  * j = 0, "the start of the round", is a legal transfer start point with dp[0, CPU] = 0; seg(0, i)
#    then covers tensors 1..i-1 and tensor 1 has no predecessor, hence no switch cost.  Without it
#    the first host tensor of a round could never be promoted.
#  * the switch cost at the boundary of a promoted tensor is the objective's c_i * 1{rb_{i-1} != rb_i}
#    with rb_{i-1} = b_{i-1} (everything between the start point and i runs on its default backend):
#    c_i is charged when b_{i-1} is the host.  (The listing prints the opposite indicator, which
#    would charge a transfer between two GPU operators and none when the activation does cross.)
#  * the start point j of a promoted tensor's transfer is a decision of the plan, as the listing's
#    minimum over j says: the latency T of the problem formulation is evaluated with
#    delta_i = max(w_i - seg(j_i, i), 0) for the chosen j_i.  A plan is admissible when every start
#    point is the round start or a host tensor executed on the host, and nothing between j_i and i
#    is promoted (those tensors run on their default backends: that is what seg adds up).
NO_TRANSFER = -2  # start point of a tensor that is not promoted
ROUND_START = -1  # the transfer starts when the round starts (j = 0 in the paper's numbering)


def seg_window(j: int, i: int, b, t_gpu, t_host, c) -> float:
    """seg(j, i) (Section 4.4.1): compute and activation-transfer time along the DEFAULT path strictly
    between tensors j and i (1-based; j = 0 is the round start): sum over k = j+1 .. i-1 of t_k on
    backend b_k, plus c_k where b_{k-1} != b_k."""
    total = 0.0
    for k in range(j + 1, i):
        total += t_gpu[k - 1] if b[k - 1] == GPU else t_host[k - 1]
        if k >= 2 and b[k - 2] != b[k - 1]:
            total += c[k - 1]
    return total


def transfer_latency(rb, start, b, t_gpu, t_host, c, w) -> float:
    """T(rb) of Section 4.4.1 for a plan: execution times on the runtime backends, switch costs
    between neighbours on different runtime backends, and for every promoted tensor (b_i = HOST,
    rb_i = GPU) the exposed part max(w_i - seg(j_i, i), 0) of its weight transfer, j_i = start[i]
    (0-based tensor index, ROUND_START for the start of the round)."""
    n = len(b)
    total = 0.0
    for i in range(1, n + 1):
        total += t_gpu[i - 1] if rb[i - 1] == GPU else t_host[i - 1]
        if i >= 2 and rb[i - 2] != rb[i - 1]:
            total += c[i - 1]
        if b[i - 1] == HOST and rb[i - 1] == GPU:
            j = 0 if start[i - 1] == ROUND_START else start[i - 1] + 1
            total += max(w[i - 1] - seg_window(j, i, b, t_gpu, t_host, c), 0.0)
    return total


def dynamic_transfer(b, t_gpu, t_host, c, w):
    """Algorithm 2 (Dynamic Transfer Scheduling), in the listing's order: the seg table, then one pass
    over the tensors with two states per tensor (the partial schedule ends on the host / on the GPU).
    A GPU-resident tensor extends either state and can only end on the GPU; a host tensor either
    stays (extends either state, ends on the host) or is promoted: the minimum over legal start
    points j of dp[j, host] + max(w_i, seg[j, i]), plus the switch cost at i and t_i^g.

    Ties keep the earlier candidate in the order the listing enumerates them (same-backend
    predecessor before the other one, smaller j first, host before GPU at the end).
    Returns (T*, rb, start) with rb[i] in {HOST, GPU} and start[i] as transfer_latency takes it.
    """
    n = len(b)
    INF = float("inf")
    seg = [[0.0] * (n + 2) for _ in range(n + 1)]
    for j in range(0, n + 1):
        for i in range(j + 1, n + 1):
            seg[j][i] = seg_window(j, i, b, t_gpu, t_host, c)
    # dp[i][s]: best latency of tensors 1..i with tensor i run on s; back[i][s] = (previous tensor, its state)
    dp = [[INF, INF] for _ in range(n + 1)]
    back = [[None, None] for _ in range(n + 1)]
    dp[0][HOST] = 0.0
    dp[0][GPU] = 0.0
    for i in range(1, n + 1):
        sw = c[i - 1] if i >= 2 else 0.0
        if b[i - 1] == GPU:
            cand = [(dp[i - 1][GPU], (i - 1, GPU)), (dp[i - 1][HOST] + sw, (i - 1, HOST))]
            if i == 1:
                cand = [(0.0, (0, GPU))]
            best = min(cand, key=lambda t: t[0])
            dp[i][GPU] = best[0] + t_gpu[i - 1]
            back[i][GPU] = best[1]
        else:
            cand = [(dp[i - 1][HOST], (i - 1, HOST)), (dp[i - 1][GPU] + sw, (i - 1, GPU))]
            if i == 1:
                cand = [(0.0, (0, HOST))]
            best = min(cand, key=lambda t: t[0])
            dp[i][HOST] = best[0] + t_host[i - 1]
            back[i][HOST] = best[1]
            best_v, best_j = INF, None
            for j in range(0, i):
                if j >= 1 and b[j - 1] != HOST:
                    continue
                v = dp[j][HOST] + max(w[i - 1], seg[j][i])
                if v < best_v:
                    best_v, best_j = v, j
            if best_j is not None:
                at_i = c[i - 1] if (i >= 2 and b[i - 2] == HOST) else 0.0
                dp[i][GPU] = best_v + at_i + t_gpu[i - 1]
                back[i][GPU] = (best_j, HOST)
    end = HOST if dp[n][HOST] <= dp[n][GPU] else GPU
    t_star = dp[n][end]
    rb = list(b)
    start = [NO_TRANSFER] * n
    i, s = n, end
    while i >= 1:
        pj, ps = back[i][s]
        rb[i - 1] = s
        if b[i - 1] == HOST and s == GPU:
            start[i - 1] = ROUND_START if pj == 0 else pj - 1
            # tensors strictly between the start point and i keep their default backends (rb = b already)
        i, s = pj, ps
    return t_star, rb, start


def deviation(m_prev, m_cur) -> float:
    """ComputeDeviation of Algorithm 3 (the paper names it without a formula): the largest relative
    change of any measured quantity, |cur - prev| / prev; a quantity that was 0 and is not any more
    counts as an unbounded change, one that stays 0 as none."""
    d = 0.0
    for p, q in zip(m_prev, m_cur):
        if p == q:
            continue
        d = max(d, abs(q - p) / abs(p) if p != 0 else float("inf"))
    return d


def reschedule(b, rb_prev, m_prev, m_cur, eps: float, tau: float, t_now: float, t_last: float):
    """Algorithm 3 (Load-aware Re-scheduling).  A measurement snapshot is the tuple (t_gpu, t_host, c, w)
    of per-tensor lists.  Keeps the previous assignment while the deviation is below eps or less
    than tau has passed since the last re-scheduling; otherwise runs Algorithm 2 on the current
    snapshot, which becomes the reference, and the clock restarts.
    Returns (rb, reference snapshot, time of last re-scheduling, replanned?)."""
    flat = lambda m: [v for part in m for v in part]
    d = deviation(flat(m_prev), flat(m_cur))
    if d < eps or t_now - t_last < tau:
        return list(rb_prev), m_prev, t_last, False
    t_gpu, t_host, c, w = m_cur
    _, rb, _ = dynamic_transfer(b, t_gpu, t_host, c, w)
    return rb, m_cur, t_now, True
