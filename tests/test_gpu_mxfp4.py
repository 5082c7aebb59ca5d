"""GPU parity of the microscaling 4-bit weight format (MXFP4, the paper's other 4-bit format) against the CPU oracle:
dequantized values bit for bit, the per-tensor operator as GEMV and as tensor-core GEMM, dense layers (decode and
prefill), the routed-expert block, and the placement / streaming invariance every format must have."""
import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu
MB = 1 << 20
ALL_GPU = {n: 1 for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")}


@pytest.fixture(scope="module")
def B():
    from paper_2607_10183_b200 import binding
    return binding


@pytest.fixture(scope="module")
def torch():
    import torch
    return torch


def ctx_for(B, resident, ws=8 * MB, ring_slots=2, slot=0, chunk=MB, flags=0):
    if slot == 0:
        ring_slots = 0
    arena = ws + ring_slots * (slot + 256) + resident + 64 * 1024
    return B.Context(arena, workspace_bytes=ws, ring_slots=ring_slots, slot_bytes=slot, chunk_bytes=chunk, flags=flags)


def test_dequant_every_element_pair_times_every_accepted_scale(B, torch):
    """All 256 byte values (every pair of element encodings) under each of the 37 accepted block exponents, as fp32 and as
    fp16: bit-exact (every such weight is an fp16 value), resident and streamed; rejected scale bytes give statuses."""
    sbytes = np.arange(104, 141, dtype=np.uint8)
    N = sbytes.size * 16
    packed = np.tile(np.arange(256, dtype=np.uint8).reshape(16, 16), (sbytes.size, 1))  # K = 32: one block per row
    scales = np.repeat(sbytes, 16).reshape(N, 1)
    want = O.dequantize(packed, scales)
    assert np.array_equal(want.astype(np.float16).astype(np.float64), want)
    nbytes = W.q4_bytes(N, 32)
    for where in (B.ATS_GPU, B.ATS_HOST):
        ctx = ctx_for(B, nbytes, slot=nbytes)
        tid = ctx.register_mxfp4(packed, scales)
        assert ctx.slice_bytes(tid) == nbytes  # the slice layout and size of the other 4-bit format
        ctx.set_placement([(tid, -1, where)])
        o32 = torch.empty((N, 32), dtype=torch.float32, device="cuda")
        o16 = torch.empty((N, 32), dtype=torch.float16, device="cuda")
        ctx.dequantize(tid, 0, o32, B.ATS_OUT_F32)
        ctx.dequantize(tid, 0, o16, B.ATS_OUT_F16)
        ctx.sync()
        assert H.bits_equal_mod_zero_sign(o32.cpu().numpy(), want.astype(np.float32))
        assert H.bits_equal_mod_zero_sign(o16.cpu().numpy(), want.astype(np.float16))
        ctx.close()
    ctx = ctx_for(B, MB)
    for byte, code in ((255, B.ATS_ERR_INVALID), (103, B.ATS_ERR_UNSUPPORTED), (141, B.ATS_ERR_UNSUPPORTED), (0, B.ATS_ERR_UNSUPPORTED)):
        bad = np.full((4, 2), 127, dtype=np.uint8)
        bad[3, 1] = byte
        with pytest.raises(B.AtsError) as e:
            ctx.register_mxfp4(np.zeros((4, 32), dtype=np.uint8), bad)
        assert e.value.code == code
    ctx.close()


@pytest.mark.parametrize("N,K,M", [(8, 32, 1), (37, 96, 3), (130, 1024, 8), (4096, 4096, 1), (256, 14336, 2), (300, 4096, 20), (1024, 1024, 129), (2048, 768, 1), (64, 256, 1)])
def test_linear_matches_oracle_gemv_and_gemm(B, torch, N, K, M):
    """Up to 8 rows: the generic GEMV (fp32 accumulation of exact products); more: the tcgen05 GEMM with the weight tile
    dequantized in the kernel (weights exact in fp16).  Streamed through the ring = resident, bit for bit."""
    packed, sb = W.mxfp4_packed(91, 0, W.ROLE_Q, N, K)
    x = W.activations(91, 0, (M, K))
    want = O.linear(x, packed, sb, round_out=True)
    nb = W.q4_bytes(N, K)
    slot = -(-nb // 256) * 256
    outs = []
    for where in (B.ATS_GPU, B.ATS_HOST):
        ws = 9 * M * N * 4 + 2 * MB
        ctx = ctx_for(B, slot, ws=ws, slot=slot, chunk=256 * 1024)
        tid = ctx.register_q4(packed, sb)  # uint8 scale bytes select the microscaling format
        ctx.set_placement([(tid, -1, where)])
        y = torch.full((M, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.reset_stats()
        ctx.linear(tid, H.to_dev(x), y, M)
        ctx.sync()
        st = ctx.stats()
        assert st.streamed_bytes == (nb if where == B.ATS_HOST else 0)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"mxfp4 linear {N}x{K} M={M}")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


def test_linear_closed_forms(B, torch):
    """Every element 1.0 with unit scales gives row sums of x; a one-hot x picks a column of the weight matrix."""
    N, K = 64, 256
    ctx = ctx_for(B, 2 * W.q4_bytes(N, K) + MB)
    ones = ctx.register_mxfp4(np.full((N, K // 2), 0x22, dtype=np.uint8), np.full((N, K // 32), 127, dtype=np.uint8))
    packed, sb = W.mxfp4_packed(91, 1, W.ROLE_Q, N, K)
    rnd = ctx.register_mxfp4(packed, sb)
    ctx.set_placement([(ones, -1, 1), (rnd, -1, 1)])
    x = W.activations(91, 1, (1, K))
    y = torch.empty((1, N), dtype=torch.float16, device="cuda")
    ctx.linear(ones, H.to_dev(x), y, 1)
    ctx.sync()
    assert np.allclose(y.cpu().numpy().astype(np.float64), x.astype(np.float64).sum(), rtol=2e-3)
    w = O.dequantize(packed, sb)
    for k in (0, 1, 31, 32, 77, 255):
        e = np.zeros((1, K), dtype=np.float16)
        e[0, k] = 1.0
        ctx.linear(rnd, H.to_dev(e), y, 1)
        ctx.sync()
        assert np.array_equal(y.cpu().numpy()[0].astype(np.float64), w[:, k])  # exact: every weight is an fp16 value
    ctx.close()


def test_embed_rows_bit_exact(B, torch):
    V, Hd = 300, 256
    packed, sb = W.mxfp4_packed(91, 2, W.ROLE_Q, V, Hd)
    ctx = ctx_for(B, W.q4_bytes(V, Hd) + MB)
    tid = ctx.register_mxfp4(packed, sb)
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    ids = np.array([0, 299, 17, 17, 123], dtype=np.int32)
    out = torch.empty((ids.size, Hd), dtype=torch.float16, device="cuda")
    ctx.embed(tid, H.to_dev(ids), out, ids.size)
    ctx.sync()
    assert H.bits_equal_mod_zero_sign(out.cpu().numpy(), O.embed(ids, packed, sb).astype(np.float16))
    ctx.close()


@pytest.mark.parametrize("M", [1, 4])
def test_dense_layer_decode_matches_oracle(B, torch, M):
    """A dense layer whose seven matrices are MXFP4: the decode step with attention (M = 1) and the FFN-only step over M
    rows; streamed matrices give the same bits; a layer mixing the two 4-bit formats is refused."""
    shape, cfg, pos, cap = W.DENSE_SMALL, 91, 37, 64
    L = W.dense_layer_mxfp4(cfg, 0, shape)
    t = H.oracle_dense_tensors(L)
    by_name = {H.ROLE_NAME[r]: W.q4_bytes(n, k) for r, n, k in shape.tensor_shapes()}
    slot = max(by_name.values())
    x = W.activations(cfg, 0, (M, shape.hidden))
    outs = []
    for placement in (ALL_GPU, dict(ALL_GPU, wk=0, wo=0, w_gate=0, w_down=0)):
        ctx = ctx_for(B, sum(by_name.values()) + 16 * 256 + 4 * shape.hidden * 2, slot=slot, chunk=64 * 1024)
        desc, ids = H.register_dense_layer(ctx, L, 0, cap)
        ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
        edges, wmode = ctx.numerics(B.ATS_MODE_DECODE)
        kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)
        kd, vd = H.to_dev(kc), H.to_dev(vc)
        y = torch.empty((M, shape.hidden), dtype=torch.float16, device="cuda")
        if M == 1:
            ctx.layer_decode(desc, H.to_dev(x), y, kd, vd, pos, 1)
            want = O.dense_layer(x, t, shape, kc, vc, pos, edges, wmode)
        else:
            ffn_ids = {n: ids[n] for n in ("ffn_norm", "w_gate", "w_up", "w_down")}
            ffn_desc = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, rms_eps=shape.rms_eps, **ffn_ids)
            ctx.layer_decode(ffn_desc, H.to_dev(x), y, None, None, 0, M)
            h2 = O._edge(O.rmsnorm(x, t["ffn_norm"], shape.rms_eps), "h2", edges)
            want = (x.astype(np.float64) + O.swiglu_ffn(h2, t["w_gate"], t["w_up"], t["w_down"], edges, wmode)).astype(np.float16)
        ctx.sync()
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"mxfp4 decode layer M={M}")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    mixed = dict(L)
    mixed[W.ROLE_O] = W.q4_packed(cfg, 0, W.ROLE_O, shape.hidden, shape.n_q_heads * shape.head_dim)
    ctx = ctx_for(B, sum(by_name.values()) + MB)
    desc, ids = H.register_dense_layer(ctx, mixed, 0, cap)
    ctx.set_placement([(ids[n], -1, 1) for n in ALL_GPU])
    kd = H.to_dev(W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)[0])
    with pytest.raises(B.AtsError) as e:
        ctx.layer_decode(desc, H.to_dev(x[:1]), torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda"), kd, kd.clone(), pos, 1)
    assert e.value.code == B.ATS_ERR_INVALID
    ctx.close()


@pytest.mark.parametrize("pos0,T,cap", [(0, 9, 16), (5, 150, 160)])
def test_dense_layer_prefill_matches_oracle(B, torch, pos0, T, cap):
    shape, cfg = W.DENSE_SMALL, 91
    L = W.dense_layer_mxfp4(cfg, 1, shape)
    nbytes = H.dense_layer_bytes(shape)
    slot = max(W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes())
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, wq=0, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, kv_capacity=cap)
    ws = B.workspace_bytes(probe, T) + MB
    x = W.activations(cfg, 1, (T, shape.hidden))
    outs = []
    for placement in (ALL_GPU, dict(ALL_GPU, wq=0, wv=0, w_up=0, w_down=0)):
        ctx = ctx_for(B, nbytes + MB, ws=ws, slot=slot)
        desc, ids = H.register_dense_layer(ctx, L, 0, cap)
        ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
        edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL)
        kc, vc = W.kv_cache(cfg, 1, shape.n_kv_heads, cap, shape.head_dim, pos0)
        kd, vd = H.to_dev(kc), H.to_dev(vc)
        y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.layer_prefill(desc, H.to_dev(x), y, kd, vd, pos0, T)
        ctx.sync()
        want = O.dense_layer(x, H.oracle_dense_tensors(L), shape, kc, vc, pos0, edges, wmode)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what="mxfp4 prefill layer")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


def moe_ctx(B, shape, T, ring_slots=8, flags=0):
    sl = W.q4_bytes(shape.ffn, shape.hidden)
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, n_experts=shape.n_experts, top_k=shape.top_k, w_gate=0, w_up=0, w_down=0)
    ws = B.workspace_bytes(probe, T) + MB
    return B.Context(ws + ring_slots * (sl + 256) + 3 * shape.n_experts * (sl + 256) + MB, workspace_bytes=ws, ring_slots=ring_slots,
                     slot_bytes=sl, chunk_bytes=MB, flags=flags)


@pytest.mark.parametrize("M", [1, 5])
def test_moe_block_decode_matches_oracle(B, torch, M):
    """Routed experts in MXFP4: ids bit-exact, output within tolerance, host-placed odd experts streamed = resident bitwise."""
    shape, cfg = W.MOE_SMALL, 91
    Bk = W.moe_block_mxfp4(cfg, 0, shape)
    x = W.activations(cfg, 0, (M, shape.hidden))
    want, ids_ref, gates_ref, logits = O.moe_block(x, H.oracle_moe_tensors(Bk), shape)
    assert O.min_rank_gap(logits, shape.top_k) > 1e-4
    outs = []
    for host in (set(), {e for e in range(shape.n_experts) if e % 2}):
        ctx = moe_ctx(B, shape, 32)
        desc, ids = H.register_moe_block(ctx, Bk)
        ctx.set_placement([(ids[n], e, B.ATS_HOST if e in host else B.ATS_GPU) for n in ("w_gate", "w_up", "w_down")
                           for e in range(shape.n_experts)])
        y = torch.empty((M, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.reset_stats()
        ctx.layer_decode(desc, H.to_dev(x), y, None, None, 0, M)
        ctx.sync()
        st = ctx.stats()
        assert (st.streamed_bytes > 0) == bool(host)
        got_ids = ctx.debug_decode_buffer(desc, M, 8, np.int32).reshape(M, -1)[:, :shape.top_k]
        assert np.array_equal(got_ids, ids_ref)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"mxfp4 moe block M={M}")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


@pytest.mark.parametrize("T", [37, 150])
def test_moe_block_prefill_matches_oracle(B, torch, T):
    shape, cfg = W.MOE_SMALL, 91
    Bk = W.moe_block_mxfp4(cfg, 0, shape)
    x = W.activations(cfg, 0, (T, shape.hidden))
    outs = []
    for host in (set(), {e for e in range(shape.n_experts) if e % 2}):
        ctx = moe_ctx(B, shape, T)
        desc, ids = H.register_moe_block(ctx, Bk)
        ctx.set_placement([(ids[n], e, B.ATS_HOST if e in host else B.ATS_GPU) for n in ("w_gate", "w_up", "w_down")
                           for e in range(shape.n_experts)])
        edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL)
        y = torch.empty((T, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.layer_prefill(desc, H.to_dev(x), y, None, None, 0, T)
        ctx.sync()
        outs.append(y.cpu().numpy())
        ctx.close()
    want, ids_ref, gates_ref, logits = O.moe_block(x, H.oracle_moe_tensors(Bk), shape, edges, wmode)
    clear = np.array([O.min_rank_gap(logits[t:t + 1], shape.top_k) > 1e-4 for t in range(T)])
    assert clear.sum() >= T - 2
    H.assert_close(outs[0][clear], want[clear], what="mxfp4 moe prefill block")
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


@pytest.mark.parametrize("M", [1, 12])
def test_lm_head_matches_oracle(B, torch, M):
    """Final norm + vocabulary projection with an MXFP4 head: a norm launch, then the generic GEMV or the GEMM; without
    scratch the call is refused (this format has no one-launch form)."""
    V, Hd, eps = 1000, 448, 1e-5
    packed, sb = W.mxfp4_packed(91, 3, W.ROLE_Q, V, Hd)
    gain = W.activations(91, 3, (Hd,)).astype(np.float16)
    x = W.activations(91, 4, (M, Hd))
    ctx = ctx_for(B, W.q4_bytes(V, Hd) + 64 * 1024, ws=16 * MB)
    nid, hid = ctx.register_f16(gain), ctx.register_mxfp4(packed, sb)
    ctx.set_placement([(hid, -1, B.ATS_GPU)])
    logits = torch.empty((M, V), dtype=torch.float16, device="cuda")
    scratch = torch.empty((M, Hd), dtype=torch.float16, device="cuda")
    ctx.lm_head(nid, hid, eps, H.to_dev(x), logits, M, scratch)
    ctx.sync()
    edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL if M > 8 else B.ATS_MODE_DECODE)
    H.assert_close(logits.cpu().numpy(), O.lm_head(x, gain, eps, packed, sb, wmode), what=f"mxfp4 lm head M={M}")
    if M == 1:
        with pytest.raises(B.AtsError) as e:
            ctx.lm_head(nid, hid, eps, H.to_dev(x), logits, 1, None)
        assert e.value.code == B.ATS_ERR_INVALID
    ctx.close()


def test_dense_layer_decode_full_size_on_the_streaming_kernel(B, torch):
    """Config-2 shapes with MXFP4 matrices: every GEMV of the step runs on the streaming single-token kernel (norm prologue,
    fused QKV, residual epilogues, fused gate/up + SwiGLU) in its microscaling mode; output against the oracle, and the
    same bits with the FFN matrices streamed from the host."""
    shape, cfg, pos, cap = W.DENSE_FULL, 91, 300, 301
    L = W.dense_layer_mxfp4(cfg, 0, shape)
    t = H.oracle_dense_tensors(L)
    by_name = {H.ROLE_NAME[r]: W.q4_bytes(n, k) for r, n, k in shape.tensor_shapes()}
    slot = max(by_name.values())
    x = W.activations(cfg, 0, (1, shape.hidden))
    outs = []
    for placement in (ALL_GPU, dict(ALL_GPU, w_gate=0, w_up=0, w_down=0)):
        ctx = ctx_for(B, sum(by_name.values()) + 16 * 256 + 4 * shape.hidden * 2, slot=slot, chunk=4 * MB)
        desc, ids = H.register_dense_layer(ctx, L, 0, cap)
        ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
        edges, wmode = ctx.numerics(B.ATS_MODE_DECODE)
        kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)
        kd, vd = H.to_dev(kc), H.to_dev(vc)
        y = torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.reset_stats()
        ctx.layer_decode(desc, H.to_dev(x), y, kd, vd, pos, 1)
        ctx.sync()
        assert ctx.stats().kernel_launches == 5  # four streaming GEMVs and the attention kernel: no separate norm launch
        outs.append(y.cpu().numpy())
        if placement is ALL_GPU:
            want = O.dense_layer(x, t, shape, kc, vc, pos, edges, wmode)
            H.assert_close(outs[-1], want, what="mxfp4 decode layer, full size")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


@pytest.mark.parametrize("M", [1, 8])
def test_moe_block_decode_full_size_on_the_streaming_kernel(B, torch, M):
    """Config-4 shapes (hidden 2048, 128 experts x 768, top-8) with MXFP4 experts: the grouped-expert streaming kernel in its
    microscaling mode, resident and with the odd experts on the host; ids bit-exact, output against the oracle."""
    shape, cfg = W.MOE_FULL, 91
    Bk = W.moe_block_mxfp4(cfg, 0, shape)
    x = W.activations(cfg, 0, (M, shape.hidden))
    want, ids_ref, gates_ref, logits = O.moe_block(x, H.oracle_moe_tensors(Bk), shape)
    assert O.min_rank_gap(logits, shape.top_k) > 1e-4
    outs = []
    odd = {e for e in range(shape.n_experts) if e % 2}
    # resident; odd experts on the host through the ring; the same read in place by the kernel (batch 1) / gathered by the
    # copy kernel (batch 8) without the host round trip
    for host, flags in ((set(), 0), (odd, B.ATS_FLAG_MOE_RING_ONLY), (odd, 0)):
        ctx = moe_ctx(B, shape, 32, ring_slots=16, flags=flags)
        desc, ids = H.register_moe_block(ctx, Bk)
        ctx.set_placement([(ids[n], e, B.ATS_HOST if e in host else B.ATS_GPU) for n in ("w_gate", "w_up", "w_down")
                           for e in range(shape.n_experts)])
        y = torch.empty((M, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.layer_decode(desc, H.to_dev(x), y, None, None, 0, M)
        ctx.sync()
        got_ids = ctx.debug_decode_buffer(desc, M, 8, np.int32).reshape(M, -1)[:, :shape.top_k]
        assert np.array_equal(got_ids, ids_ref)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"mxfp4 moe block full size M={M}")
        if host and not flags and M == 1:
            assert ctx.stats().host_syncs == 0
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    assert np.array_equal(outs[0].view(np.uint16), outs[2].view(np.uint16))
