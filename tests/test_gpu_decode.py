"""GPU parity of the decode path against the CPU oracle, through the C ABI.

Integer / byte work (dequantized values, routing ids, placement and streaming bookkeeping) must be bit-exact;
floating-point outputs must be within 2e-3 (see helpers.assert_close)."""
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


def make_ctx(B, resident_bytes, ws=8 * MB, ring_slots=2, slot_bytes=0, chunk_bytes=MB, flags=0):
    if slot_bytes == 0:
        ring_slots = 0
    arena = ws + ring_slots * (slot_bytes + 256) + resident_bytes + 64 * 1024
    return B.Context(arena, workspace_bytes=ws, ring_slots=ring_slots, slot_bytes=slot_bytes, chunk_bytes=chunk_bytes, flags=flags)


# ------------------------------------------------------------------------------------------------- a1 dequantization
def test_dequant_exhaustive_codes_times_all_finite_scales(B, torch):
    """16 codes x every finite fp16 scale bit pattern, fp32 (exact) and fp16 (one rounding), resident and streamed."""
    bits = np.arange(65536, dtype=np.uint32)
    bits = bits[(bits & 0x7C00) != 0x7C00].astype(np.uint16)  # drop Inf / NaN
    N = bits.size
    scales = bits.view(np.float16).reshape(N, 1)
    codes = np.tile(np.arange(-8, 8, dtype=np.int8), (N, 2))  # K = 32: each row one block holding all 16 codes twice
    packed = W.codes_to_packed(codes)
    want32 = O.dequantize(packed, scales).astype(np.float32)
    with np.errstate(over="ignore"):
        want16 = O.dequantize(packed, scales, O.WEIGHT_F16).astype(np.float16)
    nbytes = W.q4_bytes(N, 32)
    for where in (B.ATS_GPU, B.ATS_HOST):
        ctx = make_ctx(B, nbytes, slot_bytes=nbytes)
        tid = ctx.register_q4(packed, scales)
        ctx.set_placement([(tid, -1, where)])
        o32 = torch.empty((N, 32), dtype=torch.float32, device="cuda")
        o16 = torch.empty((N, 32), dtype=torch.float16, device="cuda")
        ctx.dequantize(tid, 0, o32, B.ATS_OUT_F32)
        ctx.dequantize(tid, 0, o16, B.ATS_OUT_F16)
        ctx.sync()
        assert H.bits_equal_mod_zero_sign(o32.cpu().numpy(), want32)
        assert H.bits_equal_mod_zero_sign(o16.cpu().numpy(), want16)
        assert not np.isnan(o16.cpu().numpy().astype(np.float32)).any()
        ctx.close()


def test_dequant_random_tensor_and_expert_slices(B, torch):
    packed, scales = W.q4_packed(94, 0, W.ROLE_GATE, 24, 160, n_experts=3)
    scales[1, 3, 2] = 0  # a zero-scale block
    scales[2, 5, 1] = -scales[2, 5, 1]  # negative scales are legal
    ctx = make_ctx(B, 3 * (W.q4_bytes(24, 160) + 256), slot_bytes=W.q4_bytes(24, 160))
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, 0, B.ATS_GPU), (tid, 1, B.ATS_HOST), (tid, 2, B.ATS_GPU)])
    for e in range(3):
        out = torch.empty((24, 160), dtype=torch.float32, device="cuda")
        ctx.dequantize(tid, e, out, B.ATS_OUT_F32)
        ctx.sync()
        assert H.bits_equal_mod_zero_sign(out.cpu().numpy(), O.dequantize(packed[e], scales[e]).astype(np.float32))
    assert ctx.get_placement(tid, 1) == B.ATS_HOST and ctx.get_placement(tid, 2) == B.ATS_GPU
    ctx.close()


# ------------------------------------------------------------------------------------------------- a2 GEMV
# (64, 256), (2048, 768), (96, 1024): single rows of at most 1024 elements take the streaming kernel's wide tiles (32 rows,
# four producer warps); (2048, 768) is the down projection of a config-4 expert
@pytest.mark.parametrize("N,K,M", [(1, 32, 1), (3, 64, 2), (17, 96, 3), (130, 1056, 8), (257, 4096, 1), (64, 14336, 5),
                                   (4096, 4096, 1), (64, 256, 1), (2048, 768, 1), (96, 1024, 1)])
def test_linear_gemv_matches_oracle(B, torch, N, K, M):
    cfg = 1 if (N, K, M) == (4096, 4096, 1) else 95
    packed, scales = W.q4_packed(cfg, 0, W.ROLE_Q, N, K)
    x = W.activations(cfg, 0, (M, K))
    want = O.linear(x, packed, scales, round_out=True)
    outs = []
    for where in (B.ATS_GPU, B.ATS_HOST):
        ctx = make_ctx(B, W.q4_bytes(N, K), slot_bytes=W.q4_bytes(N, K), chunk_bytes=64 * 1024)
        tid = ctx.register_q4(packed, scales)
        ctx.set_placement([(tid, -1, where)])
        y = torch.full((M, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.linear(tid, H.to_dev(x), y, M)
        ctx.sync()
        st = ctx.stats()
        if where == B.ATS_HOST:
            assert st.streamed_bytes == W.q4_bytes(N, K) and st.copies == -(-W.q4_bytes(N, K) // (64 * 1024))
        else:
            assert st.streamed_bytes == 0 and st.resident_bytes == W.q4_bytes(N, K)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"gemv {N}x{K} M={M}")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))  # placement never changes the math


def test_streaming_gemv_activation_extremes(B, torch):
    """The single-token kernel carries each 32-element activation block as 16-bit fixed point scaled by the block's largest
    exponent.  Blocks that stress that form: all zeros, fp16 subnormals only, one element at the top of the fp16 range
    among tiny ones (the tiny ones fall below the block's resolution: their contribution is below the gate by
    construction), alternating signs at full scale, and a one-hot (which must return the weight column exactly)."""
    N, K = 512, 2048  # a shape the streaming kernel takes (K a multiple of 256, rows a multiple of 16)
    packed, scales = W.q4_packed(95, 0, W.ROLE_Q, N, K)
    scales = (scales.astype(np.float32) * 1e-3).astype(np.float16)  # keeps the full-scale cases inside fp16 on output
    rng = np.random.default_rng(11)
    cases = {}
    cases["zeros"] = np.zeros(K, dtype=np.float16)
    cases["subnormal"] = (rng.integers(-1023, 1024, size=K).astype(np.float64) * 2.0 ** -24).astype(np.float16)
    x = (rng.standard_normal(K) * 1e-4).astype(np.float16)
    x[::32] = np.float16(60000.0) * np.where(rng.random(K // 32) < 0.5, -1, 1).astype(np.float16)
    cases["outlier_per_block"] = x
    cases["full_scale_alternating"] = (np.float16(65504.0) * np.where(np.arange(K) % 2, -1, 1)).astype(np.float16)
    x = np.zeros(K, dtype=np.float16)
    x[777] = np.float16(1.0)
    cases["one_hot"] = x
    x = rng.standard_normal(K).astype(np.float16)
    x[rng.random(K) < 0.5] = 0  # half the elements exactly zero, some blocks mostly empty
    cases["sparse"] = x
    ctx = make_ctx(B, W.q4_bytes(N, K))
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    for name, xv in cases.items():
        y = torch.full((1, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.linear(tid, H.to_dev(xv[None, :]), y, 1)
        ctx.sync()
        got = y.cpu().numpy()
        want = O.linear(xv[None, :].astype(np.float64), packed, scales, round_out=True)
        assert np.all(np.isfinite(want.astype(np.float64))), name
        if name == "zeros":
            assert np.all(got == 0), name
        elif name == "one_hot":
            assert np.array_equal(got.view(np.uint16), np.asarray(want, dtype=np.float16).view(np.uint16)), name
        elif name == "subnormal":
            # outputs are far below fp16's normal range: compare absolutely, at the resolution of the fp16 output
            assert np.max(np.abs(got.astype(np.float64) - want.astype(np.float64))) <= 2.0 ** -24, name
        else:
            H.assert_close(got, want, what=f"gemv, activations: {name}")
    ctx.close()


@pytest.mark.parametrize("where", ["gpu", "host"])
def test_embed_rows_bit_exact(B, torch, where):
    """Embedding lookup = the dequantized rows rounded once to fp16, bit for bit; a host-placed table is read in place."""
    V, Hd = 1000, 512
    packed, scales = W.q4_packed(95, 0, W.ROLE_Q, V, Hd)
    ctx = make_ctx(B, W.q4_bytes(V, Hd), slot_bytes=W.q4_bytes(V, Hd))
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, -1, B.ATS_GPU if where == "gpu" else B.ATS_HOST)])
    ids = np.array([0, 999, 17, 17, 512, 3], dtype=np.int32)
    out = torch.full((len(ids), Hd), 7.0, dtype=torch.float16, device="cuda")
    ctx.reset_stats()
    ctx.embed(tid, H.to_dev(ids), out, len(ids))
    ctx.sync()
    want = O.embed(ids, packed, scales)
    assert np.array_equal(out.cpu().numpy().view(np.uint16), want.view(np.uint16))
    assert ctx.stats().streamed_bytes == 0  # never streamed whole
    # an id outside the table: a row of zeros, and the next sync reports it
    bad = np.array([5, V], dtype=np.int32)
    out2 = torch.full((2, Hd), 7.0, dtype=torch.float16, device="cuda")
    ctx.embed(tid, H.to_dev(bad), out2, 2)
    with pytest.raises(B.AtsError):
        ctx.sync()
    assert np.all(out2.cpu().numpy()[1] == 0)
    ctx.close()


@pytest.mark.parametrize("V,Hd,M", [(4096, 1024, 1), (1000, 448, 1), (2048, 512, 5), (640, 256, 12)])
def test_lm_head_matches_oracle(B, torch, V, Hd, M):
    """Final norm + vocabulary projection: one launch of the streaming GEMV for a single row where its shapes allow, a norm
    launch and the GEMV / GEMM otherwise."""
    packed, scales = W.q4_packed(95, 1, W.ROLE_Q, V, Hd)
    gain = W.activations(95, 3, (Hd,)).astype(np.float16)
    x = W.activations(95, 0, (M, Hd))
    eps = 1e-5
    ctx = make_ctx(B, W.q4_bytes(V, Hd) + 64 * 1024, ws=16 * MB)
    nid = ctx.register_f16(gain)
    hid = ctx.register_q4(packed, scales)
    ctx.set_placement([(hid, -1, B.ATS_GPU)])
    logits = torch.empty((M, V), dtype=torch.float16, device="cuda")
    scratch = torch.empty((M, Hd), dtype=torch.float16, device="cuda")
    ctx.lm_head(nid, hid, eps, H.to_dev(x), logits, M, scratch)
    ctx.sync()
    edges, wmode = ctx.numerics(B.ATS_MODE_PREFILL if M > 8 else B.ATS_MODE_DECODE)
    want = O.lm_head(x, gain, eps, packed, scales, wmode)
    H.assert_close(logits.cpu().numpy(), want, what=f"lm head {V}x{Hd} M={M}")
    if (V, Hd, M) == (4096, 1024, 1):  # the one-launch form needs no scratch
        logits2 = torch.empty_like(logits)
        ctx.reset_stats()
        ctx.lm_head(nid, hid, eps, H.to_dev(x), logits2, 1, None)
        ctx.sync()
        assert ctx.stats().kernel_launches == 1
        assert np.array_equal(logits.cpu().numpy().view(np.uint16), logits2.cpu().numpy().view(np.uint16))
    ctx.close()


@pytest.mark.parametrize("M", [1, 4, 20])
def test_lm_head_fp16_weights_matches_oracle(B, torch, M):
    """The vocabulary projection as an unquantized fp16 matrix (the FP16 model's head): norm launch, then GEMV or GEMM."""
    V, Hd, eps = 1000, 448, 1e-5
    w = W.w16_matrix(95, 2, W.ROLE_Q, V, Hd)
    gain = W.activations(95, 3, (Hd,)).astype(np.float16)
    x = W.activations(95, 0, (M, Hd))
    ctx = make_ctx(B, V * Hd * 2 + 64 * 1024, ws=16 * MB)
    nid, hid = ctx.register_f16(gain), ctx.register_w16(w)
    ctx.set_placement([(hid, -1, B.ATS_GPU)])
    logits = torch.empty((M, V), dtype=torch.float16, device="cuda")
    scratch = torch.empty((M, Hd), dtype=torch.float16, device="cuda")
    ctx.lm_head(nid, hid, eps, H.to_dev(x), logits, M, scratch)
    ctx.sync()
    want = O.linear_w16(O.rn16(O.rmsnorm(x, gain, eps)), w, round_out=True)
    H.assert_close(logits.cpu().numpy(), want, what=f"fp16 lm head M={M}")
    if M == 1:  # this format has no one-launch form: without scratch the call is refused
        with pytest.raises(B.AtsError) as e:
            ctx.lm_head(nid, hid, eps, H.to_dev(x), logits, 1, None)
        assert e.value.code == B.ATS_ERR_INVALID
    ctx.close()


@pytest.mark.parametrize("N,K,M", [(1, 8, 1), (7, 72, 3), (130, 1000, 8), (257, 4096, 1), (4096, 4096, 1), (64, 14336, 5)])
def test_linear_w16_gemv_matches_oracle(B, torch, N, K, M):
    """An unquantized fp16 weight matrix: resident and streamed through the ring give the same bits; both match the oracle."""
    rng = np.random.default_rng(N * 131 + K)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float16)
    x = W.activations(95, 0, (M, K))
    want = O.linear_w16(x, w, round_out=True)
    outs = []
    nb = N * K * 2
    slot = -(-nb // 256) * 256
    for where in (B.ATS_GPU, B.ATS_HOST):
        ctx = make_ctx(B, slot, slot_bytes=slot, chunk_bytes=64 * 1024)
        tid = ctx.register_w16(w)
        ctx.set_placement([(tid, -1, where)])
        y = torch.full((M, N), 7.0, dtype=torch.float16, device="cuda")
        ctx.reset_stats()
        ctx.linear(tid, H.to_dev(x), y, M)
        ctx.sync()
        st = ctx.stats()
        if where == B.ATS_HOST:
            assert st.streamed_bytes == nb and st.copies == -(-nb // (64 * 1024))
        else:
            assert st.streamed_bytes == 0 and st.resident_bytes == nb
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"w16 gemv {N}x{K} M={M}")
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))


def test_plan_placement_over_mixed_formats(B, torch):
    """Algorithm 1 sees quantized and fp16 weight tensors alike (sizes in granules, values = bytes): the library's vector
    equals the oracle's on the same numbers, and the placed tensors compute the same bits as an all-resident run."""
    rng = np.random.default_rng(21)
    shapes = [("q4", 512, 1024), ("w16", 256, 512), ("q4", 1024, 512), ("w16", 512, 512), ("q4", 256, 256)]
    G = 64 * 1024
    data, nbytes = [], []
    for kind, N, K in shapes:
        if kind == "q4":
            data.append(W.q4_packed(95, len(data), W.ROLE_Q, N, K))
            nbytes.append(W.q4_bytes(N, K))
        else:
            data.append((rng.standard_normal((N, K)) * 0.05).astype(np.float16))
            nbytes.append(N * K * 2)
    budget = int(0.55 * sum(nbytes))
    slot = max(-(-b // 256) * 256 for b in nbytes)
    outs = {}
    for mode in ("all", "plan"):
        ctx = make_ctx(B, sum(nbytes) + 4096 * len(nbytes), ring_slots=2, slot_bytes=slot, chunk_bytes=64 * 1024)
        ids = [ctx.register_q4(*d) if k[0] == "q4" else ctx.register_w16(d) for k, d in zip(shapes, data)]
        if mode == "all":
            ctx.set_placement([(t, -1, B.ATS_GPU) for t in ids])
        else:
            got = ctx.plan_placement(budget, len(ids), G)
            want = O.static_placement(O.size_units(nbytes, G), nbytes, [0] * len(ids), O.budget_units(budget, G))
            assert list(got) == list(want) and 0 < sum(got) < len(ids)
        ys = []
        for t, (kind, N, K) in zip(ids, shapes):
            x = W.activations(95, 1, (1, K))
            y = torch.empty((1, N), dtype=torch.float16, device="cuda")
            ctx.linear(t, H.to_dev(x), y, 1)
            ctx.sync()
            ys.append(y.cpu().numpy())
        outs[mode] = ys
        ctx.close()
    for a, b in zip(outs["all"], outs["plan"]):
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))


def test_profile_tensor_feeds_measured_values_into_algorithm_1(B, torch):
    """Empirical performance density (Section 4.3.1): operator times measured resident and host-placed, turned into the
    residency benefit r_i of each tensor and handed to Algorithm 1; the resulting placement is the oracle's on the same
    integers.  The measuring call leaves the placement (or the unplaced state) and the results of later calls as they were."""
    shapes = [(4096, 4096), (1024, 1024), (8192, 4096), (2048, 2048)]
    data = [W.q4_packed(92, i, W.ROLE_Q, n, k) for i, (n, k) in enumerate(shapes)]
    nbytes = [W.q4_bytes(n, k) for n, k in shapes]
    slot = max(nbytes)
    ctx = make_ctx(B, sum(nbytes) + 64 * 1024, ring_slots=2, slot_bytes=slot, chunk_bytes=4 * MB)
    ids = [ctx.register_q4(*d) for d in data]
    xs = [H.to_dev(W.activations(92, i, (1, k))) for i, (n, k) in enumerate(shapes)]
    ys = [torch.empty((1, n), dtype=torch.float16, device="cuda") for n, k in shapes]
    # before any placement: measuring works and leaves the context unplaced
    t_res0, t_host0 = ctx.profile_tensor(ids[1], xs[1], ys[1], 1, iters=5)
    assert t_res0 > 0 and t_host0 > 0
    with pytest.raises(B.AtsError) as e:
        ctx.linear(ids[1], xs[1], ys[1], 1)
    assert e.value.code == B.ATS_ERR_STATE
    place = [(ids[0], -1, B.ATS_GPU), (ids[1], -1, B.ATS_HOST), (ids[2], -1, B.ATS_HOST), (ids[3], -1, B.ATS_GPU)]
    ctx.set_placement(place)
    before = []
    for t, x, y in zip(ids, xs, ys):
        ctx.linear(t, x, y, 1)
        ctx.sync()
        before.append(y.cpu().numpy().copy())
    t_res, t_host = zip(*[ctx.profile_tensor(t, x, y, 1, iters=10) for t, x, y in zip(ids, xs, ys)])
    # a streamed tensor costs its PCIe time, far above its HBM time; more bytes cost more
    for i in (0, 2, 3):
        assert t_host[i] > 3 * t_res[i], (i, t_res, t_host)
    assert t_host[2] > t_host[0] > t_host[3] > t_host[1]
    # the placement in force is back, and so are the bits
    assert [ctx.get_placement(t) for t in ids] == [w for _, _, w in place]
    for t, x, y, ref in zip(ids, xs, ys, before):
        y.zero_()
        ctx.linear(t, x, y, 1)
        ctx.sync()
        assert np.array_equal(y.cpu().numpy().view(np.uint16), ref.view(np.uint16))
    # r_i in nanoseconds saved per call by residency, c_i = 0; budget: 70 % of the bytes at 1 MiB granularity
    r = [max(0, int(round(1e3 * (h - g)))) for g, h in zip(t_res, t_host)]
    for t, v in zip(ids, r):
        ctx.set_tensor_value(t, v, 0)
    budget = int(0.7 * sum(nbytes))
    got = ctx.plan_placement(budget, len(ids))
    s_units = O.size_units(nbytes)
    want = O.static_placement(s_units, r, [0] * len(ids), O.budget_units(budget))
    assert list(got) == list(want)
    # density k = t / s: what the tensors' times say per byte (the figure the paper sorts tensors by)
    k_res = [g / b for g, b in zip(t_res, nbytes)]
    assert all(v > 0 for v in k_res)
    ctx.close()


def test_linear_closed_forms_on_gpu(B, torch):
    """One-hot activations return a weight column exactly; all-ones with unit scales return integer row sums."""
    N, K = 40, 256
    rng = np.random.default_rng(5)
    codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    scales = np.abs(rng.normal(0, 0.02, size=(N, K // 32))).astype(np.float16)
    ctx = make_ctx(B, 2 * W.q4_bytes(N, K) + 512)
    t1 = ctx.register_q4(W.codes_to_packed(codes), scales)
    t2 = ctx.register_q4(W.codes_to_packed(codes), np.ones_like(scales))
    ctx.set_placement([(t1, -1, B.ATS_GPU), (t2, -1, B.ATS_GPU)])
    y = torch.empty((1, N), dtype=torch.float16, device="cuda")
    for k in (0, 1, 7, 8, 31, 32, 255):
        x = np.zeros((1, K), dtype=np.float16)
        x[0, k] = 1
        ctx.linear(t1, H.to_dev(x), y, 1)
        ctx.sync()
        want = (scales[:, k // 32].astype(np.float64) * codes[:, k]).astype(np.float16)
        assert H.bits_equal_mod_zero_sign(y.cpu().numpy()[0], want), k
    ctx.linear(t2, H.to_dev(np.ones((1, K), dtype=np.float16)), y, 1)
    ctx.sync()
    assert np.array_equal(y.cpu().numpy()[0].astype(np.int64), codes.astype(np.int64).sum(axis=1))
    ctx.close()


# ------------------------------------------------------------------------------------------------- dense layer decode
def run_dense_decode(B, torch, shape, cfg, pos, cap, placement, ring_slots=2, flags=0, steps=1, chunk=MB, host_io=False,
                     debug=None):
    """Returns (list of y per step, final K cache, final V cache, stats) for one layer.  host_io: drive the step through
    ats_layer_decode_host from host buffers instead of device buffers ("registered": pinned buffers registered with the
    library, True: pinned but unregistered, "pageable": ordinary memory).  debug: a dict that receives the last step's
    normalised operand h (fp16) and the fp32 [q | k | v] projections as the library computed them."""
    L = W.dense_layer(cfg, 0, shape)
    slot = max(W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes())
    ctx = make_ctx(B, H.dense_layer_bytes(shape) + 16 * 256 + 4 * shape.hidden * 2, ring_slots=ring_slots, slot_bytes=slot,
                   chunk_bytes=chunk, flags=flags)
    desc, ids = H.register_dense_layer(ctx, L, 0, cap)
    assert ctx.cfg.workspace_bytes >= B.workspace_bytes(desc, 1)
    ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
    kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    ys = []
    ctx.reset_stats()
    for s in range(steps):
        x = W.activations(cfg, 0, (1, shape.hidden), step=s)
        if host_io == "pageable":  # ordinary host memory: the result comes back by a copy
            xh = np.ascontiguousarray(x)
            yh = np.zeros((1, shape.hidden), dtype=np.float16)
            ctx.layer_decode_host(desc, xh, yh, kd, vd, pos + s, 1)
            ys.append(yh.copy())
            continue
        if host_io:  # pinned memory; registered: no copy engine, the layer's last kernel writes the result into it
            xh = torch.from_numpy(x).pin_memory()
            yh = torch.zeros((1, shape.hidden), dtype=torch.float16).pin_memory()
            if host_io == "registered":
                ctx.register_host_buffer(xh)
                ctx.register_host_buffer(yh)
            ctx.layer_decode_host(desc, xh, yh, kd, vd, pos + s, 1)  # returns with yh valid: no sync here
            ys.append(yh.numpy().copy())
            if host_io == "registered":
                ctx.unregister_host_buffer(xh)
                ctx.unregister_host_buffer(yh)
            continue
        y = torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.layer_decode(desc, H.to_dev(x), y, kd, vd, pos + s, 1)
        ctx.sync()
        ys.append(y.cpu().numpy())
        if debug is not None:
            debug["h"] = ctx.debug_decode_buffer(desc, 1, 0, np.float16).copy()
            debug["qkv"] = ctx.debug_decode_buffer(desc, 1, 1, np.float32).copy()
    st = ctx.stats()
    out = (ys, kd.cpu().numpy(), vd.cpu().numpy(), st, ctx.numerics(B.ATS_MODE_DECODE))
    ctx.close()
    return out


ALL_GPU = {n: 1 for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")}


def fixed_point_gemv_bound(h, w):
    """Largest error the single-token GEMV may make on y = w h given ITS OWN operand h (fp16 values) and the exact weights
    w [N][K]: every activation is rounded to the 16-bit fixed-point grid of its block of 32, whose step is 2^(E - 29) for
    the fp16 exponent field E of the block's largest magnitude (so each activation moves by at most half a step), block dot
    products are exact, and one fp32 multiply-add per block plus the fp32 scale product accumulate the blocks."""
    h = np.asarray(h, dtype=np.float64).reshape(-1)
    n, k = w.shape
    m = np.abs(h.reshape(-1, 32)).max(axis=1)
    e_field = np.maximum(np.floor(np.log2(np.maximum(m, 2.0 ** -24))) + 15, 1)
    half_step = 2.0 ** (e_field - 30)
    quant = np.abs(w).reshape(n, -1, 32).sum(axis=2) @ half_step
    fp32 = (k // 32 + 3) * 2.0 ** -24 * (np.abs(w) @ np.abs(h))
    return quant + fp32


# positions around the attention kernel's tiling: 64 or 128 positions per CTA (contexts up to / beyond 1024), the final
# merge reads 16 splits per round trip (context 2101 at 128 per CTA needs a second one)
@pytest.mark.parametrize("shape_name,pos,cap", [("small", 0, 8), ("small", 37, 64), ("small", 63, 64), ("small", 64, 80),
                                                ("small", 200, 300), ("small", 1023, 1024), ("small", 1100, 1101),
                                                ("small", 2100, 2200), ("full", 1024, 1025)])
def test_dense_layer_decode_matches_oracle(B, torch, shape_name, pos, cap):
    shape = W.DENSE_SMALL if shape_name == "small" else W.DENSE_FULL
    cfg = 96 if shape_name == "small" else 2
    dbg = {}
    ys, kg, vg, st, (edges, wmode) = run_dense_decode(B, torch, shape, cfg, pos, cap, ALL_GPU, debug=dbg)
    L = W.dense_layer(cfg, 0, shape)
    kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)
    x = W.activations(cfg, 0, (1, shape.hidden), step=0)
    want = O.dense_layer(x, H.oracle_dense_tensors(L), shape, kc, vc, pos, edges, wmode)
    H.assert_close(ys[0], want, what="decode layer output")
    # The projections and the cache rows, held to a bound derived from the inputs instead of a fitted constant: the exact
    # product of the exact weights with the operand h the library itself formed (so that a flipped fp16 rounding of h
    # does not enter), against the library's fp32 [q | k | v]; then the rows written at `pos`: the fp16 rounding of the
    # rotated key / the value, so one fp16 ulp on top of the projection's bound (a rotation mixes two elements with
    # |cos|, |sin| <= 1, and the fp32 rotation itself adds a relative 2^-22).  Everything else in the caches is untouched.
    h_gpu = dbg["h"].astype(np.float64).reshape(-1)
    qd, kvd, d = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim, shape.head_dim
    qkv_gpu = dbg["qkv"].astype(np.float64).reshape(-1)
    proj, bound = {}, {}
    for name, role, lo, n in (("q", W.ROLE_Q, 0, qd), ("k", W.ROLE_K, qd, kvd), ("v", W.ROLE_V, qd + kvd, kvd)):
        w = O.dequantize(*L[role])
        proj[name], bound[name] = w @ h_gpu, fixed_point_gemv_bound(h_gpu, w)
        err = np.abs(qkv_gpu[lo:lo + n] - proj[name])
        assert np.all(err <= bound[name]), (name, float((err / bound[name]).max()))
        # how tight the bound is on this data: errors of random sign stay well inside the worst case
        assert err.max() <= 0.5 * bound[name].max()
    k_rot = O.rope(proj["k"].reshape(shape.n_kv_heads, d), pos, shape.rope_theta)
    bk = bound["k"].reshape(shape.n_kv_heads, d)
    bk_rot = bk + np.roll(bk, d // 2, axis=1) + 2.0 ** -21 * np.abs(k_rot)
    for got, ref, ref_new, b in ((kg, kc, k_rot, bk_rot), (vg, vc, proj["v"].reshape(shape.n_kv_heads, d), bound["v"].reshape(shape.n_kv_heads, d))):
        assert np.array_equal(np.delete(got, pos, axis=1), np.delete(ref, pos, axis=1))
        a = got[:, pos].astype(np.float64)
        ulp = np.spacing(np.abs(ref_new).astype(np.float16)).astype(np.float64)
        assert np.all(np.abs(a - ref_new) <= ulp + b)
    assert st.streamed_bytes == 0 and st.resident_bytes == H.dense_layer_bytes(shape)


@pytest.mark.parametrize("gain_std", [W.DENSE_GAIN_STD, 1.0])
def test_decode_layer_stage_by_stage_full_size(B, torch, gain_std):
    """Config 2 (one token at position 1024 through the full-size layer), every kernel on its own: each stage's output is
    compared with the oracle's definition of that stage applied to the inputs the stage actually consumed (read back from
    the library's workspace), under both error gates; the GEMV stages also under the bound derived from their operand.
    Once with the norm gains the other full-size tests use and once with gains ~N(0, 1); the end-to-end error of the layer
    is reported, not gated, in this test."""
    shape, cfg, pos, cap = W.DENSE_FULL, 2, 1024, 1025
    L = W.dense_layer(cfg, 0, shape, gain_std)
    t = H.oracle_dense_tensors(L)
    ws = B.workspace_bytes(B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, wq=0, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                                        head_dim=shape.head_dim, kv_capacity=cap), 1) + MB
    ctx = B.Context(ws + H.dense_layer_bytes(shape) + 32 * 256 + 8 * shape.hidden + MB, workspace_bytes=ws)
    desc, ids = H.register_dense_layer(ctx, L, 0, cap)
    ctx.set_placement([(ids[n], -1, B.ATS_GPU) for n in ALL_GPU])
    kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    x = W.activations(cfg, 0, (1, shape.hidden), step=0)
    y = torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.layer_decode(desc, H.to_dev(x), y, kd, vd, pos, 1)
    ctx.sync()
    g = {n: ctx.debug_decode_buffer(desc, 1, i, dt).astype(np.float64).reshape(1, -1)
         for i, (n, dt) in enumerate((("h", np.float16), ("qkv", np.float32), ("q_rot", np.float32), ("a", np.float16), ("x1", np.float32),
                                      ("h2", np.float16), ("act", np.float16)))}
    yg, kg, vg = y.cpu().numpy(), kd.cpu().numpy(), vd.cpu().numpy()
    edges, wmode = ctx.numerics(B.ATS_MODE_DECODE)
    ctx.close()
    nq, nkv, d, ffn, hid = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn, shape.hidden
    qd, kvd = nq * d, nkv * d
    x64 = x.astype(np.float64)

    def gemv_stage(got, operand, name, what):
        """A single-token GEMV stage against the exact product with ITS operand: both gates and the derived bound."""
        w = O.dequantize(*t[name])
        ref = (w @ operand.reshape(-1)).reshape(1, -1)
        H.assert_close(got, ref, what=what)
        assert np.all(np.abs(got - ref).reshape(-1) <= fixed_point_gemv_bound(operand, w)), what
        return ref

    H.assert_close(g["h"], O.rn16(O.rmsnorm(x64, t["attn_norm"], shape.rms_eps)), what="h")
    for name, lo, hi in (("wq", 0, qd), ("wk", qd, qd + kvd), ("wv", qd + kvd, qd + 2 * kvd)):
        gemv_stage(g["qkv"][:, lo:hi], g["h"], name, name)
    H.assert_close(g["q_rot"], O.rope(g["qkv"][:, :qd].reshape(1, nq, d), np.array([[float(pos)]]), shape.rope_theta).reshape(1, -1), what="q_rot")
    # the row appended at `pos`: the fp16 rounding of the rotated key / of the value the library itself computed
    k_new = O.rope(g["qkv"][:, qd:qd + kvd].reshape(1, nkv, d), np.array([[float(pos)]]), shape.rope_theta).reshape(nkv, d)
    ulp = lambda r: np.spacing(np.abs(r).astype(np.float16)).astype(np.float64)
    assert np.all(np.abs(kg[:, pos].astype(np.float64) - k_new) <= ulp(k_new))  # fp32 rotation vs fp64: at most the neighbouring fp16
    assert np.array_equal(vg[:, pos], g["qkv"][:, qd + kvd:].reshape(nkv, d).astype(np.float32).astype(np.float16))
    assert np.array_equal(np.delete(kg, pos, axis=1), np.delete(kc, pos, axis=1)) and np.array_equal(np.delete(vg, pos, axis=1), np.delete(vc, pos, axis=1))
    a = O.attention_one(g["q_rot"].reshape(nq, d), kg, vg, pos + 1).reshape(1, -1)
    H.assert_close(g["a"], O.rn16(a), what="attention")
    o = gemv_stage(g["x1"] - x64, g["a"], "wo", "wo (x1 - x)")
    H.assert_close(g["x1"], x64 + o, what="x1")
    H.assert_close(g["h2"], O.rn16(O.rmsnorm(g["x1"], t["ffn_norm"], shape.rms_eps)), what="h2")
    gate = O.dequantize(*t["w_gate"]) @ g["h2"].reshape(-1)
    up = O.dequantize(*t["w_up"]) @ g["h2"].reshape(-1)
    H.assert_close(g["act"], O.rn16(O.silu(gate) * up).reshape(1, -1), what="swiglu(gate, up)")
    dn = O.dequantize(*t["w_down"]) @ g["act"].reshape(-1)
    H.assert_close(yg, O.rn16(g["x1"] + dn.reshape(1, -1)), what="x1 + w_down act")
    kc2, vc2 = kc.copy(), vc.copy()
    want = O.dense_layer(x, t, shape, kc2, vc2, pos, edges, wmode)
    end_to_end = H.error_measures(yg, want)
    assert np.all(np.isfinite(yg.astype(np.float64)))
    print(f"decode layer, gains ~N(0, {gain_std}): end-to-end normwise error {end_to_end[0]:.2e}, mixed elementwise ratio {end_to_end[1]:.2f}")


@pytest.mark.parametrize("M", [1, 3])
def test_dense_layer_fp16_weights_decode_matches_oracle(B, torch, M):
    """A dense layer whose seven matrices are unquantized fp16 (the FP16 model of Section 5.1): the decode step with
    attention (M = 1) and the FFN-only step over M rows against the oracle; streaming four of the matrices through the
    ring gives the same bits as the resident run; a layer that mixes formats is refused."""
    shape, cfg, pos, cap = W.DENSE_SMALL, 94, 37, 64
    L = W.dense_layer_w16(cfg, 0, shape)
    by_name = {H.ROLE_NAME[r]: n * k * 2 for r, n, k in shape.tensor_shapes()}
    nbytes, slot = sum(by_name.values()), max(by_name.values())
    hybrid = dict(ALL_GPU, wq=0, wo=0, w_up=0, w_down=0)
    x = W.activations(cfg, 0, (M, shape.hidden))
    t = H.oracle_dense_tensors(L)
    outs = []
    for placement in (ALL_GPU, hybrid):
        ctx = make_ctx(B, nbytes + 16 * 256 + 4 * shape.hidden * 2, ring_slots=2, slot_bytes=slot, chunk_bytes=64 * 1024)
        desc, ids = H.register_dense_layer(ctx, L, 0, cap)
        ctx.set_placement([(ids[n], -1, w) for n, w in placement.items()])
        edges, wmode = ctx.numerics(B.ATS_MODE_DECODE)
        kc, vc = W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)
        kd, vd = H.to_dev(kc), H.to_dev(vc)
        y = torch.empty((M, shape.hidden), dtype=torch.float16, device="cuda")
        ctx.reset_stats()
        if M == 1:
            ctx.layer_decode(desc, H.to_dev(x), y, kd, vd, pos, 1)
            want = O.dense_layer(x, t, shape, kc, vc, pos, edges, wmode)  # appends position `pos` to kc, vc
            used = list(ALL_GPU)
        else:  # FFN only: the same tensors without the attention half
            ffn_ids = {n: ids[n] for n in ("ffn_norm", "w_gate", "w_up", "w_down")}
            ffn_desc = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, rms_eps=shape.rms_eps, **ffn_ids)
            ctx.layer_decode(ffn_desc, H.to_dev(x), y, None, None, 0, M)
            h2 = O._edge(O.rmsnorm(x, t["ffn_norm"], shape.rms_eps), "h2", edges)
            want = (x.astype(np.float64) + O.swiglu_ffn(h2, t["w_gate"], t["w_up"], t["w_down"], edges, wmode)).astype(np.float16)
            used = ["w_gate", "w_up", "w_down"]
        ctx.sync()
        assert ctx.stats().streamed_bytes == sum(by_name[n] for n in used if placement[n] == 0)
        outs.append(y.cpu().numpy())
        H.assert_close(outs[-1], want, what=f"fp16-weight decode layer, M={M}")
        if M == 1:
            got_k = kd.cpu().numpy()
            assert np.array_equal(np.delete(got_k, pos, axis=1), np.delete(kc, pos, axis=1))
            a, b = got_k[:, pos].astype(np.float64), kc[:, pos].astype(np.float64)
            # fp16-weight GEMV: exact products summed in fp32, no fixed-point operand
            assert np.all(np.abs(a - b) <= np.spacing(np.abs(kc[:, pos])).astype(np.float64) + 2e-5 * np.abs(b).max())
        ctx.close()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    # one quantized matrix among fp16 ones: a status, not a launch
    mixed = dict(L)
    mixed[W.ROLE_DOWN] = W.q4_packed(cfg, 0, W.ROLE_DOWN, shape.hidden, shape.ffn)
    ctx = make_ctx(B, nbytes + MB)
    desc, ids = H.register_dense_layer(ctx, mixed, 0, cap)
    ctx.set_placement([(ids[n], -1, 1) for n in ALL_GPU])
    y = torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda")
    kd = H.to_dev(W.kv_cache(cfg, 0, shape.n_kv_heads, cap, shape.head_dim, pos)[0])
    with pytest.raises(B.AtsError) as e:
        ctx.layer_decode(desc, H.to_dev(x[:1]), y, kd, kd.clone(), pos, 1)
    assert e.value.code == B.ATS_ERR_INVALID
    ctx.close()


def test_host_driven_decode_equals_device_driven(B, torch):
    """ats_layer_decode_host (H2D, step, D2H, wait) returns bit for bit what ats_layer_decode leaves on the device, with
    resident and with streamed tensors, over consecutive steps that extend the same caches."""
    shape, cfg, pos, cap = W.DENSE_SMALL, 96, 20, 40
    for placement in (ALL_GPU, {**ALL_GPU, "wk": 0, "w_up": 0, "w_down": 0}):
        dev = run_dense_decode(B, torch, shape, cfg, pos, cap, placement, steps=3)
        for mode in ("registered", True, "pageable"):
            host = run_dense_decode(B, torch, shape, cfg, pos, cap, placement, steps=3, host_io=mode)
            for a, b in zip(dev[0], host[0]):
                assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
            assert np.array_equal(dev[1], host[1]) and np.array_equal(dev[2], host[2])


def test_placement_invariance_and_bookkeeping_small(B, torch):
    """A hybrid run equals the all-resident run bit for bit (placement moves bytes, never changes math), for every ring
    size down to one slot and with freed slots poisoned; streamed bytes / copies follow the oracle's bookkeeping."""
    shape, cfg, pos, cap = W.DENSE_SMALL, 96, 20, 40
    base = run_dense_decode(B, torch, shape, cfg, pos, cap, ALL_GPU, steps=3)
    again = run_dense_decode(B, torch, shape, cfg, pos, cap, ALL_GPU, steps=3)
    for a, b in zip(base[0], again[0]):
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))  # run-to-run deterministic
    names = list(ALL_GPU)
    nbytes = [W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes()]
    rng = np.random.default_rng(0)
    cases = [({n: 0 for n in names}, 2), ({n: 0 for n in names}, 3), ({n: 0 for n in names}, 7)]
    cases += [({n: int(rng.integers(0, 2)) for n in names}, int(rng.integers(2, 5))) for _ in range(4)]
    cases += [({**ALL_GPU, "wq": 0, "wo": 0, "w_down": 0}, 1)]  # one slot is enough when no operator needs two at once
    for placement, slots in cases:
        chunk = 4096
        got = run_dense_decode(B, torch, shape, cfg, pos, cap, placement, ring_slots=slots, flags=B.ATS_FLAG_POISON_SLOTS,
                               steps=3, chunk=chunk)
        for a, b in zip(base[0], got[0]):
            assert np.array_equal(a.view(np.uint16), b.view(np.uint16)), (placement, slots)
        assert np.array_equal(base[1], got[1]) and np.array_equal(base[2], got[2])
        where = [placement[n] for n in names]
        want_bytes, want_copies, _ = O.streamed_dense(nbytes, where, chunk)
        st = got[3]
        assert st.streamed_bytes == 3 * want_bytes and st.copies == 3 * want_copies
        assert st.resident_bytes == sum(b for b, w in zip(nbytes, where) if w == 1)
        assert st.n_streamed == 3 * where.count(0)


def test_stack_under_planned_budget_full_size(B, torch):
    """Config-5 shape: a stack of full-size layers under a 60 % byte budget placed by ats_plan_placement (Algorithm 1).
    Decode steps through the stack equal the all-resident run bit for bit; the bytes and copies that moved are the
    oracle's bookkeeping for the planned placement; the planned placement equals the oracle's DP on the same records."""
    shape, cfg, n_layers, cap, pos = W.DENSE_FULL, 5, 2, 48, 32
    layer_bytes = H.dense_layer_bytes(shape)
    slot = max(W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes())
    chunk = 8 * MB
    nbytes = [W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes()]

    def run(budget_frac):
        ctx = make_ctx(B, n_layers * (layer_bytes + 16 * 256) + 8 * shape.hidden * 2, ws=16 * MB, ring_slots=4, slot_bytes=slot,
                       chunk_bytes=chunk)
        descs, q4 = [], []
        for l in range(n_layers):
            desc, ids = H.register_dense_layer(ctx, W.dense_layer(cfg, l, shape), l, cap)
            descs.append(desc)
            q4 += [ids[n] for n in ALL_GPU]
        if budget_frac is None:
            ctx.set_placement([(i, -1, 1) for i in q4])
            where = np.ones(len(q4), dtype=np.uint8)
        else:
            where = ctx.plan_placement(int(budget_frac * n_layers * layer_bytes), len(q4))
        caches = [tuple(H.to_dev(c) for c in W.kv_cache(cfg, l, shape.n_kv_heads, cap, shape.head_dim, pos)) for l in range(n_layers)]
        ctx.reset_stats()
        outs = []
        for s in range(2):
            a = H.to_dev(W.activations(cfg, 0, (1, shape.hidden), step=s))
            b = torch.empty_like(a)
            for l in range(n_layers):
                ctx.layer_decode(descs[l], a, b, caches[l][0], caches[l][1], pos + s, 1)
                a, b = b, a
            ctx.sync()
            outs.append(a.cpu().numpy().copy())
        st = ctx.stats()
        ctx.close()
        return outs, where, st

    res, _, st_res = run(None)
    hyb, where, st = run(0.60)
    assert 0 < int(where.sum()) < len(where)
    budget = int(0.60 * n_layers * layer_bytes)
    want_where = O.static_placement(O.size_units(nbytes * n_layers), nbytes * n_layers, [0] * (7 * n_layers), O.budget_units(budget))
    assert list(where) == list(want_where)  # Algorithm 1 on the same records (value = byte size, no switch cost)
    for a, b in zip(res, hyb):
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    assert st_res.streamed_bytes == 0
    per_step_bytes, per_step_copies, _ = O.streamed_dense(nbytes * n_layers, [int(w) for w in where], chunk)
    assert st.streamed_bytes == 2 * per_step_bytes and st.copies == 2 * per_step_copies
    assert st.resident_bytes == sum(b for b, w in zip(nbytes * n_layers, where) if w)
    assert st.resident_bytes <= int(0.60 * n_layers * layer_bytes)


def test_gate_up_both_streamed_needs_two_slots(B, torch):
    shape = W.DENSE_SMALL
    with pytest.raises(B.AtsError) as e:
        run_dense_decode(B, torch, shape, 96, 3, 8, {**ALL_GPU, "w_gate": 0, "w_up": 0}, ring_slots=1)
    assert e.value.code == B.ATS_ERR_BUDGET


# ------------------------------------------------------------------------------------------------- a4 routing, a5 MoE
# (hidden, experts, k): the cluster kernel with the selection by counting ranks (up to 256 experts, incl. exactly 256), the
# cluster kernel with the warp argmax (more experts), the one-CTA kernel (shapes the cluster form does not take), and the
# largest router the library accepts
@pytest.mark.parametrize("Hd,E,k", [(128, 48, 6), (128, 256, 8), (128, 264, 8), (100, 50, 6), (256, 1024, 32)])
def test_route_topk_bit_exact_with_ties(B, torch, Hd, E, k):
    rng = np.random.default_rng(11)
    M = 9
    Wr = rng.normal(0, 0.02, size=(Hd, E)).astype(np.float16)
    Wr[:, 9] = Wr[:, 2]
    Wr[:, 40] = Wr[:, 2]  # exact ties: equal columns give bitwise equal logits in any summation order
    h = rng.normal(size=(M, Hd)).astype(np.float16)
    h[0] = (Wr[:, 2].astype(np.float32) * 50).astype(np.float16)  # token 0 ranks the tied experts first
    ids_ref, gates_ref, logits = O.route_topk(h, Wr, k)
    assert ids_ref[0, :3].tolist() == [2, 9, 40]
    ctx = make_ctx(B, MB)
    rid = ctx.register_f16(Wr)
    ctx.set_placement([])
    ids = torch.empty((M, k), dtype=torch.int32, device="cuda")
    gates = torch.empty((M, k), dtype=torch.float32, device="cuda")
    ctx.route_topk(rid, H.to_dev(h), M, k, ids, gates)
    ctx.sync()
    assert np.array_equal(ids.cpu().numpy(), ids_ref)
    assert np.max(np.abs(gates.cpu().numpy() - gates_ref)) <= 1e-6
    ctx.close()


def run_moe(B, torch, shape, cfg, M, host_experts, ring_slots=8, chunk=MB, flags=0, ws=4 * MB):
    Bk = W.moe_block(cfg, 0, shape)
    sl = W.q4_bytes(shape.ffn, shape.hidden)
    ctx = make_ctx(B, 3 * shape.n_experts * (sl + 256) + MB, ws=ws, ring_slots=ring_slots, slot_bytes=sl, chunk_bytes=chunk, flags=flags)
    desc, ids = H.register_moe_block(ctx, Bk)
    ent = []
    for name in ("w_gate", "w_up", "w_down"):
        for e in range(shape.n_experts):
            ent.append((ids[name], e, B.ATS_HOST if e in host_experts else B.ATS_GPU))
    ctx.set_placement(ent)
    x = W.activations(cfg, 0, (M, shape.hidden))
    y = torch.empty((M, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.reset_stats()
    ctx.layer_decode(desc, H.to_dev(x), y, None, None, 0, M)
    ctx.sync()
    st = ctx.stats()
    out = y.cpu().numpy()
    ctx.close()
    return Bk, x, out, st


@pytest.mark.parametrize("shape_name,M", [("small", 1), ("small", 5), ("full", 1), ("full", 8)])
def test_moe_block_matches_oracle_and_streams_only_selected_experts(B, torch, shape_name, M):
    shape = W.MOE_SMALL if shape_name == "small" else W.MOE_FULL
    cfg = 97 if shape_name == "small" else 4
    odd = {e for e in range(shape.n_experts) if e % 2}
    chunk = 256 * 1024
    Bk, x, y_res, st_res = run_moe(B, torch, shape, cfg, M, set())
    _, _, y_hyb, st_hyb = run_moe(B, torch, shape, cfg, M, odd, chunk=chunk, flags=B.ATS_FLAG_POISON_SLOTS | B.ATS_FLAG_MOE_RING_ONLY)
    t = H.oracle_moe_tensors(Bk)
    want, ids_ref, gates_ref, logits = O.moe_block(x, t, shape)
    assert O.min_rank_gap(logits, shape.top_k) > 1e-4, "degenerate seed: near-tie among the routed experts"
    H.assert_close(y_res, want, what="moe block")
    assert np.array_equal(y_res.view(np.uint16), y_hyb.view(np.uint16))  # placement invariance
    assert st_res.streamed_bytes == 0 and st_res.host_syncs == 0
    sl = [W.q4_bytes(shape.ffn, shape.hidden)] * 3
    where = [[0 if e in odd else 1 for e in range(shape.n_experts)]] * 3
    nb, copies, order = O.streamed_moe(ids_ref, where, sl, chunk)
    assert st_hyb.streamed_bytes == nb and st_hyb.copies == copies and st_hyb.n_streamed == len(order)
    assert st_hyb.host_syncs == 1
    got_order = [(st_hyb.streamed_ids[i], st_hyb.streamed_experts[i]) for i in range(min(st_hyb.n_streamed, B.ATS_STATS_LIST))]
    # tensor ids are registration order: ffn_norm 0, router 1, gate 2, up 3, down 4
    assert got_order == [(2 + t_, e) for t_, e in order][:len(got_order)]


@pytest.mark.parametrize("M", [1, 8])
def test_moe_device_gather_equals_resident_without_host_round_trip(B, torch, M):
    """The default path for host-placed experts (no ATS_FLAG_MOE_RING_ONLY): the grouped-expert kernels read the selected
    host-placed experts straight from the mapped pinned store, addressed through the per-tensor slice table by the ids on the device.  Same bits as the all-resident
    run, no host synchronisation, nothing through the staging ring."""
    shape, cfg = W.MOE_FULL, 4
    odd = {e for e in range(shape.n_experts) if e % 2}
    _, _, y_res, _ = run_moe(B, torch, shape, cfg, M, set())
    _, _, y_dg, st = run_moe(B, torch, shape, cfg, M, odd)
    assert np.array_equal(y_res.view(np.uint16), y_dg.view(np.uint16))
    # every expert on the host
    _, _, y_all, st_all = run_moe(B, torch, shape, cfg, M, set(range(shape.n_experts)))
    assert np.array_equal(y_res.view(np.uint16), y_all.view(np.uint16))
    if M == 1:  # the gather path: nothing through the ring, no ids on the host
        assert st.host_syncs == 0 and st.streamed_bytes == 0 and st.copies == 0
        assert st_all.host_syncs == 0 and st_all.streamed_bytes == 0
    else:       # several tokens, no room in the workspace: the ring path (every distinct expert moves once)
        assert st.host_syncs == 1 and st.streamed_bytes > 0 and st.copies > 0
        # with room beyond the call's buffers the copy kernel gathers the distinct selected experts in one launch
        sl = W.q4_bytes(shape.ffn, shape.hidden)
        _, _, y_st, st_st = run_moe(B, torch, shape, cfg, M, odd, ws=4 * MB + 3 * 64 * (sl + 256))
        assert np.array_equal(y_res.view(np.uint16), y_st.view(np.uint16))
        # same distinct experts as the ring run moved (slices of this shape need no padding), no DMA copies
        assert st_st.host_syncs == 1 and st_st.copies == 0 and st_st.streamed_bytes == st.streamed_bytes


@pytest.mark.parametrize("host_experts", [(), (1, 3, 4, 7)])
def test_moe_layer_with_attention_matches_oracle(B, torch, host_experts):
    """A decoder layer whose FFN is the MoE block (attention, then router + routed experts on x1): the residual stream
    reaches the MoE half in fp32, the experts may sit on the host.  Two consecutive decode steps extend the caches."""
    dshape = W.DENSE_SMALL
    mshape = W.MoEShape(hidden=dshape.hidden, n_experts=8, ffn=64, top_k=2)
    cfg, cap, pos = 94, 24, 9
    Lw = W.dense_layer(cfg, 0, dshape)
    Bk = W.moe_block(cfg, 0, mshape)
    sl = W.q4_bytes(mshape.ffn, mshape.hidden)
    attn_bytes = sum(W.q4_bytes(n, k) for r, n, k in dshape.tensor_shapes() if r in (W.ROLE_Q, W.ROLE_K, W.ROLE_V, W.ROLE_O))
    ctx = make_ctx(B, attn_bytes + 3 * mshape.n_experts * (sl + 256) + MB, ring_slots=6, slot_bytes=sl, chunk_bytes=MB)
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
    kc, vc = W.kv_cache(cfg, 0, dshape.n_kv_heads, cap, dshape.head_dim, pos)
    kd, vd = H.to_dev(kc), H.to_dev(vc)
    edges, wmode = ctx.numerics(B.ATS_MODE_DECODE)
    at = H.oracle_dense_tensors(Lw)
    mt = H.oracle_moe_tensors(Bk)
    for s in range(2):
        x = W.activations(cfg, 0, (1, dshape.hidden), step=s)
        y = torch.empty((1, dshape.hidden), dtype=torch.float16, device="cuda")
        ctx.layer_decode(desc, H.to_dev(x), y, kd, vd, pos + s, 1)
        ctx.sync()
        want, ids_ref, _, logits = O.moe_layer(x, at, dshape, mt, mshape, kc, vc, pos + s, edges, wmode)
        assert O.min_rank_gap(logits, mshape.top_k) > 1e-4, "degenerate seed: near-tie among the routed experts"
        H.assert_close(y.cpu().numpy(), want, what=f"attention + MoE layer, step {s}")
        assert np.array_equal(ctx.debug_decode_buffer(desc, 1, 8, np.int32).reshape(1, -1)[:, :mshape.top_k], ids_ref)
    ctx.close()


def test_moe_small_ring_forces_waves(B, torch):
    shape = W.MOE_SMALL
    everything = set(range(shape.n_experts))
    Bk, x, y_res, _ = run_moe(B, torch, shape, 97, 5, set())
    for slots in (2, 3, 5):
        _, _, y, st = run_moe(B, torch, shape, 97, 5, everything, ring_slots=slots, flags=B.ATS_FLAG_POISON_SLOTS | B.ATS_FLAG_MOE_RING_ONLY)
        assert np.array_equal(y.view(np.uint16), y_res.view(np.uint16)), slots
        assert st.ring_reuses > 0


def test_route_and_moe_linear_standalone(B, torch):
    shape = W.MOE_SMALL
    Bk = W.moe_block(97, 0, shape)
    sl = W.q4_bytes(shape.ffn, shape.hidden)
    ctx = make_ctx(B, 3 * shape.n_experts * (sl + 256) + MB, ring_slots=4, slot_bytes=sl)
    desc, ids = H.register_moe_block(ctx, Bk)
    ctx.set_placement([(ids["w_gate"], -1, B.ATS_GPU), (ids["w_up"], -1, B.ATS_GPU)] +
                      [(ids["w_down"], e, e % 2) for e in range(shape.n_experts)])
    M, k = 3, shape.top_k
    h = W.activations(97, 3, (M, shape.hidden))
    idt = np.array([[1, 4, 7, 2], [0, 15, 3, 8], [7, 7, 6, 5]], dtype=np.int32)
    y = torch.empty((M, k, shape.ffn), dtype=torch.float16, device="cuda")
    ctx.moe_linear(ids["w_gate"], H.to_dev(h), H.to_dev(idt), y, M, k, 0)
    ctx.sync()
    H.assert_close(y.cpu().numpy().reshape(M * k, -1), O.moe_linear(h, idt, *Bk[W.ROLE_GATE]).reshape(M * k, -1))
    xs = W.activations(97, 4, (M, k, shape.ffn))
    y2 = torch.empty((M, k, shape.hidden), dtype=torch.float16, device="cuda")
    ctx.moe_linear(ids["w_down"], H.to_dev(xs), H.to_dev(idt), y2, M, k, 1)
    ctx.sync()
    H.assert_close(y2.cpu().numpy().reshape(M * k, -1), O.moe_linear(xs, idt, *Bk[W.ROLE_DOWN], x_per_slot=True).reshape(M * k, -1))
    ctx.close()


# ------------------------------------------------------------------------------------------------- errors (host-made)
def test_errors_are_statuses_and_context_stays_usable(B, torch):
    ctx = make_ctx(B, 4 * MB, ring_slots=1, slot_bytes=1024)
    packed, scales = W.q4_packed(98, 0, 0, 8, 64)
    import ctypes as C
    d = B.ats_tensor_desc(B.ATS_FMT_Q4B32, 1, 8, 40, 0, 0, -1, 0)
    out = C.c_int32()
    assert B.ats_register_tensor(ctx.h, C.byref(d), packed.ctypes.data, scales.ctypes.data, C.byref(out)) == B.ATS_ERR_SHAPE
    bad = scales.copy()
    bad[0, 0] = np.inf
    with pytest.raises(B.AtsError) as e:
        ctx.register_q4(packed, bad)
    assert e.value.code == B.ATS_ERR_INVALID
    tid = ctx.register_q4(packed, scales)
    y = torch.empty((1, 8), dtype=torch.float16, device="cuda")
    x = H.to_dev(W.activations(98, 0, (1, 64)))
    with pytest.raises(B.AtsError) as e:
        ctx.linear(tid, x, y, 1)  # no placement yet
    assert e.value.code == B.ATS_ERR_STATE
    with pytest.raises(B.AtsError) as e:
        ctx.set_placement([(tid + 5, -1, 1)])
    assert e.value.code == B.ATS_ERR_INVALID
    big = ctx.register_q4(*W.q4_packed(98, 1, 0, 64, 64))
    with pytest.raises(B.AtsError) as e:
        ctx.set_placement([(tid, -1, 1), (big, -1, 0)])  # host slice larger than a ring slot
    assert e.value.code == B.ATS_ERR_BUDGET
    ctx.set_placement([(tid, -1, 0), (big, -1, 1)])
    ctx.linear(tid, x, y, 1)
    ctx.sync(timeout_ms=5000)
    H.assert_close(y.cpu().numpy(), O.linear(W.activations(98, 0, (1, 64)), packed, scales, round_out=True))
    # injected copy failure: status, then the context reports itself poisoned
    B.ats_debug_fail_copies(ctx.h, 1)
    with pytest.raises(B.AtsError) as e:
        ctx.linear(tid, x, y, 1)
    assert e.value.code == B.ATS_ERR_CUDA
    with pytest.raises(B.AtsError):
        ctx.linear(tid, x, y, 1)
    ctx.close()
    # arena too small for the resident set
    ctx = make_ctx(B, 0, ring_slots=0, ws=0)
    tid = ctx.register_q4(*W.q4_packed(98, 2, 0, 1024, 1024))
    with pytest.raises(B.AtsError) as e:
        ctx.set_placement([(tid, -1, 1)])
    assert e.value.code == B.ATS_ERR_BUDGET
    ctx.close()


# ------------------------------------------------------------------------------------------------- failure paths
def test_empty_calls_and_longest_rows(B, torch):
    """Degenerate and maximal sizes: calls over zero rows / tokens succeed and write nothing; the longest row the streaming
    kernel takes (16384 elements) and the next longer one (which the generic kernel takes) both match the oracle."""
    N, K = 64, 256
    packed, scales = W.q4_packed(94, 0, W.ROLE_Q, N, K)
    ctx = make_ctx(B, 4 * MB)
    tid = ctx.register_q4(packed, scales)
    rid = ctx.register_f16(np.zeros((K, 8), dtype=np.float16))
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    x = torch.zeros((1, K), dtype=torch.float16, device="cuda")
    y = torch.full((1, N), 7.0, dtype=torch.float16, device="cuda")
    ids = torch.full((1, 2), -5, dtype=torch.int32, device="cuda")
    gates = torch.full((1, 2), 3.0, dtype=torch.float32, device="cuda")
    ctx.linear(tid, x, y, 0)
    ctx.route_topk(rid, x, 0, 2, ids, gates)
    ctx.sync()
    assert (y.cpu().numpy() == 7.0).all() and (ids.cpu().numpy() == -5).all() and (gates.cpu().numpy() == 3.0).all()
    ctx.close()
    shape = W.DENSE_SMALL
    L = W.dense_layer(96, 0, shape)
    ctx = make_ctx(B, H.dense_layer_bytes(shape) + 64 * 1024, ws=8 * MB)
    desc, lids = H.register_dense_layer(ctx, L, 0, 16)
    ctx.set_placement([(lids[n], -1, B.ATS_GPU) for n in ALL_GPU])
    kd = torch.zeros((shape.n_kv_heads, 16, shape.head_dim), dtype=torch.float16, device="cuda")
    vd = torch.zeros_like(kd)
    xa = torch.zeros((1, shape.hidden), dtype=torch.float16, device="cuda")
    ya = torch.full((1, shape.hidden), 7.0, dtype=torch.float16, device="cuda")
    ctx.layer_decode(desc, xa, ya, kd, vd, 0, 0)
    ctx.layer_prefill(desc, xa, ya, kd, vd, 0, 0)
    ctx.sync()
    assert (ya.cpu().numpy() == 7.0).all() and not kd.cpu().numpy().any() and not vd.cpu().numpy().any()
    ctx.close()
    for K2 in (16384, 16384 + 256):
        N2 = 32
        p2, s2 = W.q4_packed(94, 1, W.ROLE_Q, N2, K2)
        x2 = W.activations(94, 1, (1, K2))
        ctx = make_ctx(B, W.q4_bytes(N2, K2) + 64 * 1024)
        t2 = ctx.register_q4(p2, s2)
        ctx.set_placement([(t2, -1, B.ATS_GPU)])
        y2 = torch.empty((1, N2), dtype=torch.float16, device="cuda")
        ctx.linear(t2, H.to_dev(x2), y2, 1)
        ctx.sync()
        H.assert_close(y2.cpu().numpy(), O.linear(x2, p2, s2, round_out=True), what=f"gemv over rows of {K2} elements")
        ctx.close()


def test_gemv_non_finite_activation_gives_non_finite_output(B, torch):
    """An Inf or a NaN among the activations must not turn into a finite output: the streaming kernel's fixed-point operand
    cannot carry it, so the block's term becomes NaN (the plain definition gives Inf or NaN in every row here, since every
    output sums over every k)."""
    N, K = 64, 512
    packed, scales = W.q4_packed(93, 0, W.ROLE_Q, N, K)
    ctx = make_ctx(B, W.q4_bytes(N, K) + 512)
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    y = torch.empty((1, N), dtype=torch.float16, device="cuda")
    for bad_k, bad in ((5, np.inf), (300, -np.inf), (77, np.nan)):
        x = W.activations(93, 0, (1, K))
        x[0, bad_k] = bad
        with np.errstate(invalid="ignore", over="ignore"):
            want = O.linear(x, packed, scales)
        assert not np.isfinite(want).any()
        ctx.linear(tid, H.to_dev(x), y, 1)
        ctx.sync()
        assert not np.isfinite(y.cpu().numpy().astype(np.float32)).any(), (bad_k, bad)
    # finite again afterwards
    x = W.activations(93, 0, (1, K))
    ctx.linear(tid, H.to_dev(x), y, 1)
    ctx.sync()
    H.assert_close(y.cpu().numpy(), O.linear(x, packed, scales), what="gemv after non-finite inputs")
    ctx.close()


def test_router_ids_stay_in_range_for_a_nan_row(B, torch):
    """A row of NaN activations gives NaN logits, which compare false with everything: the ids must still name experts
    (they index weight slices downstream) and the row's gates are NaN; the other rows are unaffected."""
    rng = np.random.default_rng(12)
    Hd, E, k, M = 128, 48, 6, 3
    Wr = rng.normal(0, 0.02, size=(Hd, E)).astype(np.float16)
    h = rng.normal(size=(M, Hd)).astype(np.float16)
    h[1, :] = np.nan
    ctx = make_ctx(B, 64 * 1024)
    rid = ctx.register_f16(Wr)
    ctx.set_placement([])
    ids = torch.full((M, k), -7, dtype=torch.int32, device="cuda")
    gates = torch.zeros((M, k), dtype=torch.float32, device="cuda")
    ctx.route_topk(rid, H.to_dev(h), M, k, ids, gates)
    ctx.sync()
    got_ids, got_gates = ids.cpu().numpy(), gates.cpu().numpy()
    assert got_ids.min() >= 0 and got_ids.max() < E
    assert len(set(got_ids[1].tolist())) == k and np.isnan(got_gates[1]).all()
    ids_ref, gates_ref, _ = O.route_topk(h[[0, 2]], Wr, k)
    assert np.array_equal(got_ids[[0, 2]], ids_ref) and np.allclose(got_gates[[0, 2]], gates_ref, atol=1e-6)
    ctx.close()


def test_moe_linear_rejects_ids_out_of_range(B, torch):
    """ids are caller data.  Host-placed slices: checked on the host before anything runs.  All slices resident: only the
    kernel sees them; it computes with expert 0 in place of the bad id (no wild address) and raises the status word, so
    the next ats_sync reports ATS_ERR_INVALID."""
    shape = W.MOE_SMALL
    Bk = W.moe_block(95, 0, shape)
    sl = W.q4_bytes(shape.ffn, shape.hidden)
    x = W.activations(95, 0, (1, shape.hidden))
    for where, code_at in ((B.ATS_HOST, "call"), (B.ATS_GPU, "sync")):
        ctx = make_ctx(B, shape.n_experts * (sl + 256) + 64 * 1024, ring_slots=4, slot_bytes=sl, chunk_bytes=sl)
        tid = ctx.register_q4(*Bk[W.ROLE_GATE])
        ctx.set_placement([(tid, -1, where)])
        ids = torch.tensor([[1, shape.n_experts + 5, 2, -3]], dtype=torch.int32, device="cuda")
        y = torch.zeros((1, 4, shape.ffn), dtype=torch.float16, device="cuda")
        with pytest.raises(B.AtsError) as e:
            ctx.moe_linear(tid, H.to_dev(x), ids, y, 1, 4)
            assert code_at == "sync"
            ctx.sync()
        assert e.value.code == B.ATS_ERR_INVALID
        if code_at == "sync":
            # the slots with valid ids were computed; the bad ones ran on expert 0
            got = y.cpu().numpy()
            want = O.moe_linear(x, np.array([[1, 0, 2, 0]]), *Bk[W.ROLE_GATE])
            H.assert_close(got.reshape(4, -1), want.reshape(4, -1), what="moe_linear with clamped ids")
        ctx.close()


def test_bounded_wait_expiry_is_reported_and_leaves_other_contexts_usable(B, torch):
    """The failure path of the streaming GEMV, made to run without anything faulting or hanging: the test hook shortens
    the kernel's wait limit to about two milliseconds and makes the producer leave out the copies of tile 0, so the
    consumers of that tile wait in vain, give up, raise the status word and return; the other CTAs finish their rows.
    ats_sync then returns ATS_ERR_TIMEOUT and the context refuses further work; a fresh context computes correctly."""
    N, K = 64, 2048  # four tiles of 16 rows (rows longer than 1024 take 16-row tiles), one per CTA
    packed, scales = W.q4_packed(93, 1, W.ROLE_Q, N, K)
    x = W.activations(93, 1, (1, K))
    want = O.linear(x, packed, scales)
    ctx = make_ctx(B, W.q4_bytes(N, K) + 512)
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    y = torch.zeros((1, N), dtype=torch.float16, device="cuda")
    ctx.linear(tid, H.to_dev(x), y, 1)
    ctx.sync()
    H.assert_close(y.cpu().numpy(), want, what="gemv before the injected expiry")
    ctx.debug_gemv_wait(4_000_000, withhold_tile=0)
    y.zero_()
    ctx.linear(tid, H.to_dev(x), y, 1)
    with pytest.raises(B.AtsError) as e:
        ctx.sync(timeout_ms=5000)
    assert e.value.code == B.ATS_ERR_TIMEOUT and "bounded wait" in str(e.value)
    got = y.cpu().numpy()
    assert not got[0, :16].any()  # tile 0 never arrived: its rows were not written
    H.assert_close(got[:, 16:], want[:, 16:], what="rows of the tiles that did arrive")
    with pytest.raises(B.AtsError) as e:
        ctx.linear(tid, H.to_dev(x), y, 1)
    assert e.value.code == B.ATS_ERR_CUDA  # poisoned
    ctx.close()
    ctx2 = make_ctx(B, W.q4_bytes(N, K) + 512)
    t2 = ctx2.register_q4(packed, scales)
    ctx2.set_placement([(t2, -1, B.ATS_GPU)])
    y2 = torch.zeros((1, N), dtype=torch.float16, device="cuda")
    ctx2.linear(t2, H.to_dev(x), y2, 1)
    ctx2.sync()
    H.assert_close(y2.cpu().numpy(), want, what="gemv on a fresh context after the expiry")
    ctx2.close()
