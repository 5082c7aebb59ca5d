"""GPU parity of the prefill path (dequantize-fused tensor-core GEMM, causal attention, layer) against the CPU oracle."""
import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu
MB = 1 << 20


@pytest.fixture(scope="module")
def B():
    from paper_2607_10183_b200 import binding
    return binding


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def gemm_ctx(B, N, K, T, where, extra=0):
    nb = W.q4_bytes(N, K)
    ws = 8 * T * N * 4 + 2 * MB
    arena = ws + 2 * (nb + 256) + nb + MB + extra
    ctx = B.Context(arena, workspace_bytes=ws, ring_slots=2, slot_bytes=nb, chunk_bytes=MB)
    return ctx


@pytest.mark.parametrize("N,K,T", [(128, 64, 16), (128, 256, 9), (136, 320, 127), (256, 512, 128), (384, 1024, 129), (130, 96, 300),
                                   (512, 2048, 512), (256, 4096, 600), (1024, 14336, 33)])
def test_linear_gemm_matches_oracle(B, torch, N, K, T):
    """M > 8 takes the tensor-core GEMM: fp16 operands (weights rounded once), fp32 accumulation, fp16 output.
    Shapes cover ragged feature tiles, ragged token tiles, split-K and K that is not a multiple of the 64-wide stage."""
    packed, scales = W.q4_packed(99, 0, W.ROLE_Q, N, K)
    x = W.activations(99, 0, (T, K))
    want16 = O.linear(x, packed, scales, O.WEIGHT_F16, round_out=True)
    want_exact = O.linear(x, packed, scales, O.WEIGHT_EXACT, round_out=True)
    outs = []
    for where in (B.ATS_GPU, B.ATS_HOST):
        ctx = gemm_ctx(B, N, K, T, where)
        tid = ctx.register_q4(packed, scales)
        ctx.set_placement([(tid, -1, where)])
        y = torch.full((T, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.linear(tid, H.to_dev(x), y, T)
        ctx.sync()
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want16, what=f"gemm {N}x{K} T={T} vs fp16-weight oracle")
        H.assert_close(outs[-1], want_exact, what=f"gemm {N}x{K} T={T} vs exact-weight oracle")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


def test_gemm_rows_equal_gemv_within_tolerance_and_one_hot(B, torch):
    """Row m of the GEMM agrees with the GEMV of row m; one-hot activations return the fp16-rounded weight column."""
    N, K, T = 256, 512, 64
    packed, scales = W.q4_packed(99, 1, W.ROLE_Q, N, K)
    ctx = gemm_ctx(B, N, K, T, 1)
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    x = W.activations(99, 1, (T, K))
    yg = torch.empty((T, N), dtype=torch.float16, device="cuda")
    ctx.linear(tid, H.to_dev(x), yg, T)
    yv = torch.empty((4, N), dtype=torch.float16, device="cuda")
    ctx.linear(tid, H.to_dev(x[10:14]), yv, 4)
    ctx.sync()
    H.assert_close(yg.cpu().numpy()[10:14], yv.cpu().numpy().astype(np.float64), what="gemm row vs gemv")
    eye = np.zeros((T, K), dtype=np.float16)
    ks = [0, 1, 7, 8, 31, 32, 63, 64, 65, 255, 256, 511]
    for i, k in enumerate(ks):
        eye[i, k] = 1
    ctx.linear(tid, H.to_dev(eye), yg, T)
    ctx.sync()
    w16 = O.dequantize(packed, scales, O.WEIGHT_F16).astype(np.float16)
    got = yg.cpu().numpy()
    for i, k in enumerate(ks):
        assert H.bits_equal_mod_zero_sign(got[i], w16[:, k]), k
    assert not got[len(ks):].any()
    ctx.close()


def prefill_ctx(B, shape, cap, T, placement, ring_slots=2):
    L = None
    slot = max(W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes())
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, wq=0, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, kv_capacity=cap)
    ws = B.workspace_bytes(probe, T) + MB
    arena = ws + ring_slots * (slot + 256) + H.dense_layer_bytes(shape) + MB
    return B.Context(arena, workspace_bytes=ws, ring_slots=ring_slots, slot_bytes=slot, chunk_bytes=4 * MB)


def run_prefill(B, torch, shape, cfg, pos0, T, cap, placement):
    L = W.dense_layer(cfg, 0, shape)
    ctx = prefill_ctx(B, shape, cap, T, placement)
    desc, ids = H.register_dense_layer(ctx, L, 0, cap)
    ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
    kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos0)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    x = W.activations(cfg, 0, (T, shape.hidden))
    y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.reset_stats()
    ctx.layer_prefill(desc, H.to_dev(x), y, kd, vd, pos0, T)
    ctx.sync()
    out = (y.cpu().numpy(), kd.cpu().numpy(), vd.cpu().numpy(), ctx.stats(), ctx.numerics(B.ATS_MODE_PREFILL), L, x, kc, vc)
    ctx.close()
    return out


ALL_GPU = {n: 1 for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")}


@pytest.mark.parametrize("shape_name,pos0,T,cap", [("small", 0, 7, 16), ("small", 5, 40, 64), ("small", 0, 130, 130), ("full", 0, 512, 512)])
def test_dense_layer_prefill_matches_oracle(B, torch, shape_name, pos0, T, cap):
    shape = W.DENSE_SMALL if shape_name == "small" else W.DENSE_FULL
    cfg = 96 if shape_name == "small" else 3
    y, kg, vg, st, (edges, wmode), L, x, kc, vc = run_prefill(B, torch, shape, cfg, pos0, T, cap, ALL_GPU)
    assert wmode == O.WEIGHT_F16 and edges == frozenset(O.EDGES)
    want = O.dense_layer(x, H.oracle_dense_tensors(L), shape, kc, vc, pos0, edges, wmode)
    H.assert_close(y, want, what="prefill layer output", elementwise=True if shape_name == "small" else "counted")
    for got, ref in ((kg, kc), (vg, vc)):
        a = got[:, pos0:pos0 + T].astype(np.float64)
        b = ref[:, pos0:pos0 + T].astype(np.float64)
        assert np.array_equal(got[:, :pos0], ref[:, :pos0]) and np.array_equal(got[:, pos0 + T:], ref[:, pos0 + T:])
        # written rows: fp16 values of an fp16 GEMM output, so at most a few ulps off the oracle's
        assert np.max(np.abs(a - b)) <= 4e-3 * np.max(np.abs(b))


def test_prefill_placement_invariance(B, torch):
    shape, cfg = W.DENSE_SMALL, 96
    base = run_prefill(B, torch, shape, cfg, 3, 40, 64, ALL_GPU)
    hyb = run_prefill(B, torch, shape, cfg, 3, 40, 64, {**ALL_GPU, "wk": 0, "wo": 0, "w_gate": 0, "w_up": 0})
    assert np.array_equal(base[0].view(np.uint16), hyb[0].view(np.uint16))
    assert np.array_equal(base[1], hyb[1]) and np.array_equal(base[2], hyb[2])
    nbytes = {n: W.q4_bytes(r, k) for (role, r, k), n in zip(shape.tensor_shapes(), ALL_GPU)}
    assert hyb[3].streamed_bytes == sum(nbytes[n] for n in ("wk", "wo", "w_gate", "w_up"))


def test_prefill_then_decode_continues_the_cache(B, torch):
    """A prefill of T tokens followed by a decode step equals (within tolerance) the oracle doing the same, which pins
    that both calls agree on cache layout and positions."""
    shape, cfg, T, cap = W.DENSE_SMALL, 96, 24, 32
    L = W.dense_layer(cfg, 0, shape)
    ctx = prefill_ctx(B, shape, cap, T, ALL_GPU)
    desc, ids = H.register_dense_layer(ctx, L, 0, cap)
    ctx.set_placement([(ids[n], -1, 1) for n in ALL_GPU])
    kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, 0)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    x = W.activations(cfg, 0, (T, shape.hidden))
    y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.layer_prefill(desc, H.to_dev(x), y, kd, vd, 0, T)
    x1 = W.activations(cfg, 0, (1, shape.hidden), step=7)
    y1 = torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.layer_decode(desc, H.to_dev(x1), y1, kd, vd, T, 1)
    ctx.sync()
    t = H.oracle_dense_tensors(L)
    O.dense_layer(x, t, shape, kc, vc, 0, frozenset(O.EDGES), O.WEIGHT_F16)
    e, w = ctx.numerics(B.ATS_MODE_DECODE)
    want = O.dense_layer(x1, t, shape, kc, vc, T, e, w)
    H.assert_close(y1.cpu().numpy(), want, what="decode after prefill")
    ctx.close()


def test_model_loop_chunked_prefill_then_decode_three_layers(B, torch):
    """The whole-model loop on a small stack: a 40-token prompt prefilled in chunks of 16, 16 and 8 through three layers
    with distinct weights (later chunks attend to the cache the earlier ones wrote), then two decode steps through the
    same layers.  Every layer call is held against the oracle run on exactly what the library was given (its input rows
    and its cache state before the call), so rounding differences do not compound from layer to layer."""
    shape, cfg, cap, n_layers = W.DENSE_SMALL, 98, 48, 3
    layers = [W.dense_layer(cfg, l, shape) for l in range(n_layers)]
    ctx = make_stack_ctx(B, shape, cap, 16, n_layers)
    descs, place = [], []
    for l, Lw in enumerate(layers):
        desc, ids = H.register_dense_layer(ctx, Lw, l, cap)
        descs.append(desc)
        place += [(ids[n], -1, 1) for n in ALL_GPU]
    ctx.set_placement(place)
    caches = [tuple(H.to_dev(c) for c in W.kv_cache(cfg, l, shape.n_kv_heads, cap, shape.head_dim, 0)) for l in range(n_layers)]
    e_pre, w_pre = ctx.numerics(B.ATS_MODE_PREFILL)
    e_dec, w_dec = ctx.numerics(B.ATS_MODE_DECODE)

    def run_layer(l, x_host, pos, T, prefill):
        kc0, vc0 = caches[l][0].cpu().numpy().copy(), caches[l][1].cpu().numpy().copy()
        y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
        if prefill:
            ctx.layer_prefill(descs[l], H.to_dev(x_host), y, caches[l][0], caches[l][1], pos, T)
        else:
            ctx.layer_decode(descs[l], H.to_dev(x_host), y, caches[l][0], caches[l][1], pos, T)
        ctx.sync()
        got = y.cpu().numpy()
        want = O.dense_layer(x_host, H.oracle_dense_tensors(layers[l]), shape, kc0, vc0, pos,
                             e_pre if prefill else e_dec, w_pre if prefill else w_dec)
        H.assert_close(got, want, what=f"layer {l} pos {pos} T {T} {'prefill' if prefill else 'decode'}")
        # the oracle appended the rows the library did (fp16 values of rounded projections: a few ulps apart at most),
        # and neither touched any other row
        for dev_c, ref_c in ((caches[l][0], kc0), (caches[l][1], vc0)):
            got_c = dev_c.cpu().numpy()
            a, b = got_c[:, pos:pos + T].astype(np.float64), ref_c[:, pos:pos + T].astype(np.float64)
            assert np.max(np.abs(a - b)) <= 4e-3 * np.max(np.abs(b))
            assert np.array_equal(got_c[:, :pos], ref_c[:, :pos]) and np.array_equal(got_c[:, pos + T:], ref_c[:, pos + T:])
        return got

    pos = 0
    for c, T in enumerate((16, 16, 8)):
        x = W.activations(cfg, 0, (T, shape.hidden), step=c)
        for l in range(n_layers):
            x = run_layer(l, x, pos, T, True)
        pos += T
    for s in range(2):
        x = W.activations(cfg, 1, (1, shape.hidden), step=s)
        for l in range(n_layers):
            x = run_layer(l, x, pos, 1, False)
        pos += 1
    ctx.close()


def make_stack_ctx(B, shape, cap, T, n_layers):
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, wq=0, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, kv_capacity=cap)
    ws = max(B.workspace_bytes(probe, T), B.workspace_bytes(probe, 1)) + MB
    arena = ws + n_layers * (H.dense_layer_bytes(shape) + 32 * 256 + 8 * shape.hidden) + MB
    return B.Context(arena, workspace_bytes=ws)


@pytest.mark.parametrize("gain_std", [W.DENSE_GAIN_STD, 1.0])
def test_prefill_layer_stage_by_stage_full_size(B, torch, gain_std):
    """Config 3 (512 tokens through the full-size layer), every kernel on its own: each stage's output is compared with the
    oracle's definition of that stage applied to the inputs the stage actually consumed, under both error gates.  Once with
    the norm gains the other full-size tests use and once with gains ~N(0, 1), which make every intermediate four times
    larger; the end-to-end error of the layer is reported, not gated, in this test."""
    shape, cfg, T, cap = W.DENSE_FULL, 3, 512, 512
    L = W.dense_layer(cfg, 0, shape, gain_std)
    t = H.oracle_dense_tensors(L)
    ctx = prefill_ctx(B, shape, cap, T, ALL_GPU)
    desc, ids = H.register_dense_layer(ctx, L, 0, cap)
    ctx.set_placement([(ids[n], -1, 1) for n in ALL_GPU])
    kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, 0)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    x = W.activations(cfg, 0, (T, shape.hidden))
    y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.layer_prefill(desc, H.to_dev(x), y, kd, vd, 0, T)
    ctx.sync()
    g = {n: ctx.debug_prefill_buffer(desc, T, i).astype(np.float64)
         for i, n in enumerate(("h", "qkv", "q_rot", "a", "o", "x1", "h2", "gu", "act", "d"))}
    yg, kg, vg = y.cpu().numpy(), kd.cpu().numpy(), vd.cpu().numpy()
    e_pre, w_pre = ctx.numerics(B.ATS_MODE_PREFILL)
    ctx.close()
    nq, nkv, d, ffn = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn
    qd, kvd = nq * d, nkv * d
    F16 = O.WEIGHT_F16
    H.assert_close(g["h"], O.rn16(O.rmsnorm(x, t["attn_norm"], shape.rms_eps)), what="h")
    for name, lo, hi in (("wq", 0, qd), ("wk", qd, qd + kvd), ("wv", qd + kvd, qd + 2 * kvd)):
        H.assert_close(g["qkv"][:, lo:hi], O.linear(g["h"], *t[name], F16, round_out=True), what=name)
    pos = np.arange(T, dtype=np.float64).reshape(T, 1)
    H.assert_close(g["q_rot"], O.rn16(O.rope(g["qkv"][:, :qd].reshape(T, nq, d), pos, shape.rope_theta)).reshape(T, -1), what="q_rot")
    k_rot = O.rn16(O.rope(g["qkv"][:, qd:qd + kvd].reshape(T, nkv, d), pos, shape.rope_theta))
    H.assert_close(kg.transpose(1, 0, 2).reshape(T, -1), k_rot.reshape(T, -1), what="k cache")
    assert np.array_equal(vg.transpose(1, 0, 2).reshape(T, -1).astype(np.float64), g["qkv"][:, qd + kvd:])
    a = np.stack([O.attention_one(g["q_rot"][i].reshape(nq, d), kg, vg, i + 1).reshape(-1) for i in range(T)])
    H.assert_close(g["a"], O.rn16(a), what="attention")
    H.assert_close(g["o"], O.linear(g["a"], *t["wo"], F16, round_out=True), what="wo")
    assert np.array_equal(g["x1"], O.rn16(x.astype(np.float64) + g["o"]))
    H.assert_close(g["h2"], O.rn16(O.rmsnorm(g["x1"], t["ffn_norm"], shape.rms_eps)), what="h2")
    H.assert_close(g["gu"][:, :ffn], O.linear(g["h2"], *t["w_gate"], F16, round_out=True), what="w_gate")
    H.assert_close(g["gu"][:, ffn:], O.linear(g["h2"], *t["w_up"], F16, round_out=True), what="w_up")
    H.assert_close(g["act"], O.rn16(O.silu(g["gu"][:, :ffn]) * g["gu"][:, ffn:]), what="swiglu")
    H.assert_close(g["d"], O.linear(g["act"], *t["w_down"], F16, round_out=True), what="w_down")
    assert np.array_equal(yg.astype(np.float64), O.rn16(g["x1"] + g["d"]))
    kc2, vc2 = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, 0)
    want = O.dense_layer(x, t, shape, kc2, vc2, 0, e_pre, w_pre)
    end_to_end = H.error_measures(yg, want)
    assert np.all(np.isfinite(yg.astype(np.float64)))
    print(f"prefill layer, gains ~N(0, {gain_std}): end-to-end normwise error {end_to_end[0]:.2e}, mixed elementwise ratio {end_to_end[1]:.2f}")


# ------------------------------------------------------------------------------------------------- MoE prefill
def run_moe_prefill(B, torch, shape, cfg, T, host_experts, extra_ws=0):
    """The routed FFN block over T tokens in one ats_layer_prefill call (no attention)."""
    Bk = W.moe_block(cfg, 0, shape)
    sl = W.q4_bytes(shape.ffn, shape.hidden)
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, n_experts=shape.n_experts, top_k=shape.top_k, w_gate=0, w_up=0, w_down=0)
    ws = B.workspace_bytes(probe, T) + MB + extra_ws  # room beyond the layer's buffers: where selected host experts are staged
    ctx = B.Context(ws + 8 * (sl + 256) + 3 * shape.n_experts * (sl + 256) + MB, workspace_bytes=ws, ring_slots=8, slot_bytes=sl,
                    chunk_bytes=MB)
    desc, ids = H.register_moe_block(ctx, Bk)
    ctx.set_placement([(ids[n], e, B.ATS_HOST if e in host_experts else B.ATS_GPU) for n in ("w_gate", "w_up", "w_down")
                       for e in range(shape.n_experts)])
    x = W.activations(cfg, 0, (T, shape.hidden))
    y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.reset_stats()
    ctx.layer_prefill(desc, H.to_dev(x), y, None, None, 0, T)
    ctx.sync()
    out = (Bk, x, y.cpu().numpy(), ctx.stats(), ctx.numerics(B.ATS_MODE_PREFILL))
    ctx.close()
    return out


@pytest.mark.parametrize("T", [1, 37, 150])
def test_moe_prefill_block_matches_oracle_small(B, torch, T):
    """Every token of the chunk against the oracle's routed FFN under the prefill contract (fp16 GEMM outputs, fp16-rounded
    weights); 16 experts, top-4: expert row counts from 0 to well over one 128-row tile at T = 150 (ragged tails)."""
    shape, cfg = W.MOE_SMALL, 97
    Bk, x, y, st, (edges, wmode) = run_moe_prefill(B, torch, shape, cfg, T, set())
    want, ids_ref, gates_ref, logits = O.moe_block(x, H.oracle_moe_tensors(Bk), shape, edges, wmode)
    # a token whose k-th and (k+1)-th logits nearly tie may legitimately route differently in fp32: leave it out
    clear = np.array([O.min_rank_gap(logits[t:t + 1], shape.top_k) > 1e-4 for t in range(T)])
    assert clear.sum() >= T - 2
    H.assert_close(y[clear], want[clear], what="moe prefill block")
    assert st.host_syncs == 1 and st.streamed_bytes == 0
    # host-placed experts are read in place through the mapped pinned store: same bits
    odd = {e for e in range(shape.n_experts) if e % 2}
    _, _, y_h, st_h, _ = run_moe_prefill(B, torch, shape, cfg, T, odd)
    assert np.array_equal(y.view(np.uint16), y_h.view(np.uint16))
    _, _, y_all, _, _ = run_moe_prefill(B, torch, shape, cfg, T, set(range(shape.n_experts)))
    assert np.array_equal(y.view(np.uint16), y_all.view(np.uint16))


def test_moe_prefill_block_full_size_sampled_tokens(B, torch):
    """Config-4 shapes (hidden 2048, 128 experts x 768, top-8), 512 tokens: sampled tokens against the oracle, and the
    single-token decode path on the same tokens (a different kernel family, same contract up to the fp16 edges)."""
    shape, cfg, T = W.MOE_FULL, 4, 512
    Bk, x, y, st, (edges, wmode) = run_moe_prefill(B, torch, shape, cfg, T, set())
    assert np.all(np.isfinite(y.astype(np.float64)))
    sample = [0, 1, 127, 128, 300, 511]
    want, _, _, logits = O.moe_block(x[sample], H.oracle_moe_tensors(Bk), shape, edges, wmode)
    assert O.min_rank_gap(logits, shape.top_k) > 1e-4
    H.assert_close(y[sample], want, what="moe prefill block, sampled tokens")
    odd = {e for e in range(shape.n_experts) if e % 2}
    _, _, y_h, st_h, _ = run_moe_prefill(B, torch, shape, cfg, T, odd)  # no room to stage: slices read in place
    assert np.array_equal(y.view(np.uint16), y_h.view(np.uint16)) and st_h.streamed_bytes == 0
    sl = W.q4_bytes(shape.ffn, shape.hidden)
    _, _, y_s, st_s, _ = run_moe_prefill(B, torch, shape, cfg, T, odd, extra_ws=3 * (shape.n_experts // 2) * (sl + 256) + MB)
    assert np.array_equal(y.view(np.uint16), y_s.view(np.uint16))  # staged by the copy kernel
    assert 0 < st_s.streamed_bytes <= 3 * (shape.n_experts // 2) * (sl + 256) and st_s.copies == 0


@pytest.mark.parametrize("host_experts", [(), (1, 3, 4, 7)])
def test_moe_layer_with_attention_prefill_matches_oracle(B, torch, host_experts):
    """A decoder layer whose FFN is the MoE block, over a chunk of tokens: causal attention with cache append, then the
    routed experts on x1 (fp16 residual stream, as in the dense prefill contract)."""
    dshape = W.DENSE_SMALL
    mshape = W.MoEShape(hidden=dshape.hidden, n_experts=8, ffn=64, top_k=2)
    cfg, cap, pos0, T = 94, 64, 5, 41
    Lw = W.dense_layer(cfg, 0, dshape)
    Bk = W.moe_block(cfg, 0, mshape)
    sl = W.q4_bytes(mshape.ffn, mshape.hidden)
    attn_bytes = sum(W.q4_bytes(n, k) for r, n, k in dshape.tensor_shapes() if r in (W.ROLE_Q, W.ROLE_K, W.ROLE_V, W.ROLE_O))
    probe = B.layer_desc(hidden=dshape.hidden, ffn=mshape.ffn, wq=0, n_q_heads=dshape.n_q_heads, n_kv_heads=dshape.n_kv_heads,
                         head_dim=dshape.head_dim, kv_capacity=cap, n_experts=mshape.n_experts, top_k=mshape.top_k)
    ws = B.workspace_bytes(probe, T) + MB
    ctx = B.Context(ws + 6 * (sl + 256) + attn_bytes + 3 * mshape.n_experts * (sl + 256) + MB, workspace_bytes=ws, ring_slots=6,
                    slot_bytes=sl, chunk_bytes=MB)
    ids = {"attn_norm": ctx.register_f16(Lw[W.ROLE_ATTN_NORM], 0, W.ROLE_ATTN_NORM)}
    for r, n in ((W.ROLE_Q, "wq"), (W.ROLE_K, "wk"), (W.ROLE_V, "wv"), (W.ROLE_O, "wo")):
        ids[n] = ctx.register_q4(*Lw[r], layer=0, role=r)
    ids["ffn_norm"] = ctx.register_f16(Bk[W.ROLE_FFN_NORM], 0, W.ROLE_FFN_NORM)
    ids["router"] = ctx.register_f16(Bk[W.ROLE_ROUTER], 0, W.ROLE_ROUTER)
    for r, n in ((W.ROLE_GATE, "w_gate"), (W.ROLE_UP, "w_up"), (W.ROLE_DOWN, "w_down")):
        ids[n] = ctx.register_q4(*Bk[r], layer=0, role=r)
    desc = B.layer_desc(hidden=dshape.hidden, ffn=mshape.ffn, n_q_heads=dshape.n_q_heads, n_kv_heads=dshape.n_kv_heads,
                        head_dim=dshape.head_dim, kv_capacity=cap, rms_eps=dshape.rms_eps, rope_theta=dshape.rope_theta,
                        n_experts=mshape.n_experts, top_k=mshape.top_k, **ids)
    place = [(ids[n], -1, 1) for n in ("wq", "wk", "wv", "wo")]
    place += [(ids[n], e, 0 if e in host_experts else 1) for n in ("w_gate", "w_up", "w_down") for e in range(mshape.n_experts)]
    ctx.set_placement(place)
    kc, vc = W.kv_cache(cfg, 0, dshape.n_kv_heads, cap, dshape.head_dim, pos0)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL)
    x = W.activations(cfg, 0, (T, dshape.hidden))
    y = torch.empty((T, dshape.hidden), dtype=torch.float16, device="cuda")
    ctx.layer_prefill(desc, H.to_dev(x), y, kd, vd, pos0, T)
    ctx.sync()
    want, _, _, logits = O.moe_layer(x, H.oracle_dense_tensors(Lw), dshape, H.oracle_moe_tensors(Bk), mshape, kc, vc, pos0, edges, wmode)
    clear = np.array([O.min_rank_gap(logits[t:t + 1], mshape.top_k) > 1e-4 for t in range(T)])
    assert clear.sum() >= T - 2
    H.assert_close(y.cpu().numpy()[clear], want[clear], what="attention + MoE layer, prefill")
    kg = kd.cpu().numpy()
    assert np.max(np.abs(kg[:, pos0:pos0 + T].astype(np.float64) - kc[:, pos0:pos0 + T].astype(np.float64))) <= 4e-3 * np.max(np.abs(kc))
    ctx.close()


@pytest.mark.parametrize("N,K,T", [(128, 64, 16), (136, 320, 127), (384, 1024, 129), (130, 96, 300), (1024, 4096, 512), (4096, 1024, 9)])
def test_linear_w16_gemm_matches_oracle(B, torch, N, K, T):
    """More than 8 rows against an unquantized fp16 weight matrix: the tcgen05 GEMM with the weight tile loaded by TMA
    instead of dequantized; ragged N, K, T, split-K shapes; resident and streamed give the same bits."""
    rng = np.random.default_rng(N * 7 + K * 3 + T)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float16)
    x = W.activations(96, 0, (T, K))
    want = O.linear_w16(x, w, round_out=True)
    nb = N * K * 2
    slot = -(-nb // 256) * 256
    outs = []
    for where in (B.ATS_GPU, B.ATS_HOST):
        ws = 9 * T * N * 4 + 2 * MB
        ctx = B.Context(ws + 2 * (slot + 256) + slot + MB, workspace_bytes=ws, ring_slots=2, slot_bytes=slot, chunk_bytes=MB)
        tid = ctx.register_w16(w)
        ctx.set_placement([(tid, -1, where)])
        y = torch.full((T, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.linear(tid, H.to_dev(x), y, T)
        ctx.sync()
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"w16 gemm {N}x{K} T={T}")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


@pytest.mark.parametrize("pos0,T,cap", [(0, 9, 16), (5, 150, 160)])
def test_dense_layer_fp16_weights_prefill_matches_oracle(B, torch, pos0, T, cap):
    """The prefill chunk of a dense layer with unquantized fp16 matrices (one GEMM per matrix, the residual of the
    O projection in its epilogue) against the oracle; streamed matrices give the same bits as resident ones."""
    shape, cfg = W.DENSE_SMALL, 93
    L = W.dense_layer_w16(cfg, 0, shape)
    nbytes = sum(n * k * 2 for _, n, k in shape.tensor_shapes())
    slot = max(n * k * 2 for _, n, k in shape.tensor_shapes())
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, wq=0, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, kv_capacity=cap)
    ws = B.workspace_bytes(probe, T) + MB
    x = W.activations(cfg, 0, (T, shape.hidden))
    outs = []
    for placement in (ALL_GPU, dict(ALL_GPU, wk=0, wo=0, w_gate=0, w_down=0)):
        ctx = B.Context(ws + 2 * (slot + 256) + nbytes + MB, workspace_bytes=ws, ring_slots=2, slot_bytes=slot, chunk_bytes=MB)
        desc, ids = H.register_dense_layer(ctx, L, 0, cap)
        ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
        edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL)
        kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos0)
        kd, vd = H.to_dev(kc), H.to_dev(vc)
        y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.layer_prefill(desc, H.to_dev(x), y, kd, vd, pos0, T)
        ctx.sync()
        want = O.dense_layer(x, H.oracle_dense_tensors(L), shape, kc, vc, pos0, edges, wmode)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what="fp16-weight prefill layer")
        got_k = kd.cpu().numpy()
        assert np.array_equal(got_k[:, :pos0], kc[:, :pos0]) and np.array_equal(got_k[:, pos0 + T:], kc[:, pos0 + T:])
        a, b = got_k[:, pos0:pos0 + T].astype(np.float64), kc[:, pos0:pos0 + T].astype(np.float64)
        assert np.max(np.abs(a - b)) <= 4e-3 * np.max(np.abs(b))
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


@pytest.mark.parametrize("N,K,T", [(14336, 256, 512), (14400, 200, 700), (7200, 4096, 1100)])
def test_linear_w16_gemm_as_cta_pair_matches_oracle(B, torch, N, K, T):
    """fp16-weight GEMMs with enough tiles run as pairs of CTAs on two SMs (tcgen05 cta_group::2: 512 tokens x 256 features
    per pair, each CTA loading half of the weight rows).  Against the oracle, incl. ragged N, K and T (rows past the
    matrix and k past K read as zeros, stores guarded), and against the single-CTA kernel selected by flag."""
    rng = np.random.default_rng(N + K + T)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float16)
    x = W.activations(96, 2, (T, K))
    want = O.linear_w16(x, w, round_out=True)
    outs = []
    for flags in (0, B.ATS_FLAG_NO_GEMM_PAIR):
        ws = 9 * T * N * 4 + 2 * MB
        ctx = B.Context(ws + N * K * 2 + 4 * MB, workspace_bytes=ws, flags=flags)
        tid = ctx.register_w16(w)
        ctx.set_placement([(tid, -1, B.ATS_GPU)])
        y = torch.full((T, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.linear(tid, H.to_dev(x), y, T)
        ctx.sync()
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"w16 gemm {N}x{K} T={T} flags={flags}")
        ctx.close()
    # same products, fp32 accumulation in both; the single-CTA kernel may split K, so not necessarily the same bits
    H.assert_close(outs[0], outs[1].astype(np.float64), what="pair against single-CTA kernel")


@pytest.mark.parametrize("fmt,N,K,T", [("q4", 4000, 8192, 2000), ("mxfp4", 4000, 8192, 2000), ("q4", 4096, 14336, 1024), ("mxfp4", 3900, 14336, 1000)])
def test_linear_gemm_4bit_as_cta_pair_matches_oracle(B, torch, fmt, N, K, T):
    """The dequantizing GEMM as a pair of CTAs (long reductions): every CTA dequantizes half of the pair's 256 weight rows
    into its own shared memory, the leader issues the M = 256 instructions; with few tiles K is split over blockIdx.z
    and a second launch sums the fp32 partials (the 1024-token cases).  Sampled tokens against the oracle (all features), the
    whole output against the single-CTA kernel selected by flag; ragged N and T."""
    packed, scales = (W.q4_packed if fmt == "q4" else W.mxfp4_packed)(90, 0, W.ROLE_DOWN, N, K)
    x = W.activations(90, 0, (T, K))
    outs = []
    for flags in (0, B.ATS_FLAG_NO_GEMM_PAIR):
        ws = 9 * T * N * 4 + 2 * MB
        ctx = B.Context(ws + W.q4_bytes(N, K) + 4 * MB, workspace_bytes=ws, flags=flags)
        tid = ctx.register_q4(packed, scales)
        ctx.set_placement([(tid, -1, B.ATS_GPU)])
        edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL)
        y = torch.full((T, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.linear(tid, H.to_dev(x), y, T)
        ctx.sync()
        outs.append(y.cpu().numpy())
        ctx.close()
    rows = np.array([r for r in (0, 1, 127, 128, 255, 256, 499, 511, 512, 777, 1023, 1024, 1535, 1536, 1999) if r < T])
    want = O.linear(x[rows], packed, scales, wmode, round_out=True)
    H.assert_close(outs[0][rows], want, what=f"{fmt} pair gemm, sampled tokens")
    H.assert_close(outs[1][rows], want, what=f"{fmt} single-CTA gemm, sampled tokens")
    H.assert_close(outs[0], outs[1].astype(np.float64), what="pair against single-CTA kernel")
