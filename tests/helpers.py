"""Shared helpers of the GPU parity tests: build a library context from the seeded workloads and compare with the oracle."""
import numpy as np

from paper_2607_10183_b200 import workloads as W

TOL = 2e-3  # max relative error of fp outputs (fp32 accumulation vs the fp64 oracle), as the workload states it


def assert_close(y, ref, tol=TOL, what="", elementwise=True):
    """Max relative error per output row, measured two ways: normwise max|y-r| / max|r| <= tol (always), and mixed
    elementwise |y-r| <= tol (|r| + rms(r)) (a pure elementwise relative error is meaningless next to the zero crossings
    of a dot product).  Single operators and every stage of a layer are held to both (elementwise=True).  The end-to-end
    output of a full-size prefill layer (eleven fp16-rounded stages, two million outputs) is held to the normwise gate and
    to the mixed gate with its violations counted and bounded (elementwise="counted"): a one-ulp difference in the
    rounding of an intermediate (fp32 accumulation and fp64 land on different sides of a rounding boundary for ~1 % of the
    elements) propagates through the later stages, and the maximum of the ratio over millions of outputs is a tail
    statistic of those flips; the stage-wise tests hold every kernel to both gates on the inputs it consumed."""
    y = np.asarray(y, dtype=np.float64).reshape(-1, np.asarray(y).shape[-1])
    r = np.asarray(ref, dtype=np.float64).reshape(y.shape)
    assert np.all(np.isfinite(y)), f"{what}: non-finite output"
    err = np.abs(y - r)
    norm = err.max(axis=1) / np.maximum(np.abs(r).max(axis=1), 1e-30)
    assert norm.max() <= tol, f"{what}: normwise error {norm.max():.3e} > {tol}"
    rms = np.sqrt(np.mean(r * r, axis=1, keepdims=True))
    ratio = err / (tol * (np.abs(r) + rms) + 1e-300)
    if elementwise == "counted":
        # End-to-end output of a layer whose every intermediate is stored as fp16: the mixed gate still holds for all but
        # the few elements downstream of an intermediate that fp32 and fp64 arithmetic rounded to different fp16
        # neighbours.  Those are counted and bounded instead of being let through: at most one element in a thousand may
        # exceed the gate, and none by more than a factor of two.
        over = ratio > 1.0
        assert over.mean() <= 1e-3, f"{what}: {over.mean():.2e} of the elements exceed the mixed elementwise gate"
        assert ratio.max() <= 2.0, f"{what}: mixed elementwise ratio {ratio.max():.3f} > 2"
    elif elementwise:
        assert ratio.max() <= 1.0, f"{what}: mixed elementwise ratio {ratio.max():.3f} > 1"
    return float(norm.max()), float(ratio.max())


def error_measures(y, ref, tol=TOL):
    """The two figures assert_close gates (largest normwise error over the rows, largest mixed elementwise ratio), only
    measured: for results a test reports without holding them to a bound."""
    y = np.asarray(y, dtype=np.float64).reshape(-1, np.asarray(y).shape[-1])
    r = np.asarray(ref, dtype=np.float64).reshape(y.shape)
    err = np.abs(y - r)
    norm = err.max(axis=1) / np.maximum(np.abs(r).max(axis=1), 1e-30)
    rms = np.sqrt(np.mean(r * r, axis=1, keepdims=True))
    return float(norm.max()), float((err / (tol * (np.abs(r) + rms) + 1e-300)).max())


def bits_equal_mod_zero_sign(a, b):
    """Bitwise equality after mapping -0 to +0."""
    a = np.asarray(a)
    b = np.asarray(b)
    a = np.where(a == 0, np.zeros_like(a), a)
    b = np.where(b == 0, np.zeros_like(b), b)
    ia = a.view(np.uint32 if a.dtype == np.float32 else np.uint16)
    ib = b.view(np.uint32 if b.dtype == np.float32 else np.uint16)
    return np.array_equal(ia, ib)


ROLE_NAME = {W.ROLE_Q: "wq", W.ROLE_K: "wk", W.ROLE_V: "wv", W.ROLE_O: "wo", W.ROLE_GATE: "w_gate", W.ROLE_UP: "w_up",
             W.ROLE_DOWN: "w_down"}
DENSE_ROLES = (W.ROLE_Q, W.ROLE_K, W.ROLE_V, W.ROLE_O, W.ROLE_GATE, W.ROLE_UP, W.ROLE_DOWN)


def oracle_dense_tensors(L):
    t = {ROLE_NAME[r]: L[r] for r in DENSE_ROLES}
    t["attn_norm"], t["ffn_norm"] = L[W.ROLE_ATTN_NORM], L[W.ROLE_FFN_NORM]
    return t


def oracle_moe_tensors(B):
    return {"w_gate": B[W.ROLE_GATE], "w_up": B[W.ROLE_UP], "w_down": B[W.ROLE_DOWN], "router": B[W.ROLE_ROUTER],
            "ffn_norm": B[W.ROLE_FFN_NORM]}


def register_dense_layer(ctx, L, layer_idx, kv_capacity):
    """Registers one dense layer's tensors in execution order; returns (layer descriptor, {role: id}).  A matrix given
    as (packed, scales) is block-quantized, one given as (w16,) is an unquantized fp16 matrix."""
    from paper_2607_10183_b200 import binding as B
    shape = L["shape"]
    ids = {}

    def reg(r):
        if len(L[r]) == 1:
            return ctx.register_w16(L[r][0], layer=layer_idx, role=r)
        return ctx.register_q4(*L[r], layer=layer_idx, role=r)

    ids["attn_norm"] = ctx.register_f16(L[W.ROLE_ATTN_NORM], layer_idx, W.ROLE_ATTN_NORM)
    for r in (W.ROLE_Q, W.ROLE_K, W.ROLE_V, W.ROLE_O):
        ids[ROLE_NAME[r]] = reg(r)
    ids["ffn_norm"] = ctx.register_f16(L[W.ROLE_FFN_NORM], layer_idx, W.ROLE_FFN_NORM)
    for r in (W.ROLE_GATE, W.ROLE_UP, W.ROLE_DOWN):
        ids[ROLE_NAME[r]] = reg(r)
    desc = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                        head_dim=shape.head_dim, kv_capacity=kv_capacity, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, **ids)
    return desc, ids


def register_moe_block(ctx, Bk, layer_idx=0):
    from paper_2607_10183_b200 import binding as B
    shape = Bk["shape"]
    ids = {}
    ids["ffn_norm"] = ctx.register_f16(Bk[W.ROLE_FFN_NORM], layer_idx, W.ROLE_FFN_NORM)
    ids["router"] = ctx.register_f16(Bk[W.ROLE_ROUTER], layer_idx, W.ROLE_ROUTER)
    for r in (W.ROLE_GATE, W.ROLE_UP, W.ROLE_DOWN):
        ids[ROLE_NAME[r]] = ctx.register_q4(*Bk[r], layer=layer_idx, role=r)
    desc = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, n_experts=shape.n_experts, top_k=shape.top_k, rms_eps=shape.rms_eps, **ids)
    return desc, ids


def dense_layer_bytes(shape):
    return sum(W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes())


def to_dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()
