"""Config 5 at its stated size: a 32-layer dense stack (3.93 GB of 4-bit weights) under a 60 % byte budget placed by the
library (Algorithm 1, Section 4.3.2), the other tensors in pinned host memory and streamed through the staging ring by the
transfer stream while the compute stream runs the operators (Sections 4.2.1, 4.2.2): a 512-token prefill, then 128 decode
steps (positions 512 .. 639).

Checked: the placement vector against the oracle's dynamic program; the bytes and copies that crossed PCIe per pass
against the oracle's bookkeeping; the hybrid run against the all-resident run bit for bit at every decode step, on the
prefill output and on every cache; and single layers against the oracle, each recomputed from exactly what the library
was given (its input rows and its cache before the call), at the first and last decode step and in the prefill, so that
rounding differences do not compound over 32 layers (end-to-end drift is not gated)."""
import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu
MB = 1 << 20

N_LAYERS, CAP, T_PREFILL, N_STEPS, CFG = 32, 640, 512, 128, 5
NAMES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
# (layer, decode step) pairs and prefill layers that are held to the oracle
DECODE_POINTS = ((0, 0), (31, 0), (17, 64), (0, 127), (31, 127))
PREFILL_LAYERS = (0, 31)


def x_step(shape, step):
    """The token fed to layer 0 at a decode step: a fresh seeded row per step (no token feedback without an LM head)."""
    return W.activations(CFG, 0, (1, shape.hidden), step=step)


def run_stack(B, torch, shape, layers, hybrid, budget, chunk, capture):
    """Prefill then decode through the stack.  Returns a dict of outputs; with `capture`, also the inputs, the cache
    before the call and the output of the sampled layer calls."""
    layer_bytes = H.dense_layer_bytes(shape)
    slot = max(W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes())
    probe = B.layer_desc(hidden=shape.hidden, ffn=shape.ffn, wq=0, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, kv_capacity=CAP)
    ws = max(B.workspace_bytes(probe, T_PREFILL), B.workspace_bytes(probe, 1)) + MB
    ring_slots = 8 if hybrid else 0
    resident = (budget if hybrid else N_LAYERS * layer_bytes) + N_LAYERS * (16 * 256 + 4 * shape.hidden) + 4 * MB
    ctx = B.Context(ws + ring_slots * (slot + 256) + resident, workspace_bytes=ws, ring_slots=ring_slots, slot_bytes=slot,
                    chunk_bytes=chunk)
    descs, q4 = [], []
    for l, Lw in enumerate(layers):
        desc, ids = H.register_dense_layer(ctx, Lw, l, CAP)
        descs.append(desc)
        q4 += [ids[n] for n in NAMES]
    out = {}
    if hybrid:
        out["where"] = ctx.plan_placement(budget, len(q4))
    else:
        ctx.set_placement([(i, -1, B.ATS_GPU) for i in q4])
    out["resident_bytes"] = int(ctx.stats().resident_bytes)
    caches = [(torch.zeros((shape.n_kv_heads, CAP, shape.head_dim), dtype=torch.float16, device="cuda"),
               torch.zeros((shape.n_kv_heads, CAP, shape.head_dim), dtype=torch.float16, device="cuda")) for _ in range(N_LAYERS)]
    cap = {}

    # ---- prefill: 512 tokens at positions 0..511 through every layer
    ctx.reset_stats()
    xa = H.to_dev(W.activations(CFG, 0, (T_PREFILL, shape.hidden), step=10_000))
    xb = torch.empty_like(xa)
    torch.cuda.synchronize()
    for l in range(N_LAYERS):
        if capture and l in PREFILL_LAYERS:
            ctx.sync()
            cap[("prefill", l, "x")] = xa.cpu().numpy().copy()
        ctx.layer_prefill(descs[l], xa, xb, caches[l][0], caches[l][1], 0, T_PREFILL)
        if capture and l in PREFILL_LAYERS:
            ctx.sync()
            cap[("prefill", l, "y")] = xb.cpu().numpy().copy()
            cap[("prefill", l, "k")] = caches[l][0].cpu().numpy().copy()
            cap[("prefill", l, "v")] = caches[l][1].cpu().numpy().copy()
        xa, xb = xb, xa
    ctx.sync()
    st = ctx.stats()
    out["prefill_y"] = xa.cpu().numpy().copy()
    out["prefill_streamed"] = (int(st.streamed_bytes), int(st.copies), int(st.n_streamed))

    # ---- 128 decode steps at positions 512..639
    ctx.reset_stats()
    # Every buffer a step touches is written by the library's own stream only: the inputs of all steps are on the device
    # before the first step, the layers ping-pong between two scratch rows, and the last layer of step s writes row s of
    # `ys`.  Nothing synchronises inside a step, and the host only waits every 16 steps, so the transfer stream runs as
    # far ahead of the compute stream as the ring lets it.
    xs = H.to_dev(np.concatenate([x_step(shape, s) for s in range(N_STEPS)], axis=0))
    ys = torch.zeros((N_STEPS, shape.hidden), dtype=torch.float16, device="cuda")
    da = torch.empty((1, shape.hidden), dtype=torch.float16, device="cuda")
    db = torch.empty_like(da)
    torch.cuda.synchronize()
    for s in range(N_STEPS):
        pos = T_PREFILL + s
        src = xs[s:s + 1]
        for l in range(N_LAYERS):
            dst = ys[s:s + 1] if l == N_LAYERS - 1 else (db if src is da else da)
            point = capture and (l, s) in DECODE_POINTS
            if point:
                ctx.sync()
                cap[("decode", l, s, "x")] = src.cpu().numpy().copy()
                cap[("decode", l, s, "k")] = caches[l][0].cpu().numpy().copy()
                cap[("decode", l, s, "v")] = caches[l][1].cpu().numpy().copy()
            ctx.layer_decode(descs[l], src, dst, caches[l][0], caches[l][1], pos, 1)
            if point:
                ctx.sync()
                cap[("decode", l, s, "y")] = dst.cpu().numpy().copy()
            src = dst
        if s % 16 == 15:
            ctx.sync()  # keeps the host from running unboundedly far ahead of the device
    ctx.sync()
    st = ctx.stats()
    out["decode_ys"] = [ys[s:s + 1].cpu().numpy() for s in range(N_STEPS)]
    out["decode_streamed"] = (int(st.streamed_bytes), int(st.copies), int(st.n_streamed))
    out["caches"] = [(k.cpu().numpy(), v.cpu().numpy()) for k, v in caches]
    out["numerics"] = (ctx.numerics(B.ATS_MODE_DECODE), ctx.numerics(B.ATS_MODE_PREFILL))
    out["capture"] = cap
    ctx.close()
    del caches
    torch.cuda.empty_cache()
    return out


def test_config5_full_stack_hybrid_prefill_then_128_decode_steps():
    import torch
    from paper_2607_10183_b200 import binding as B
    shape = W.DENSE_FULL
    layers = [W.dense_layer(CFG, l, shape) for l in range(N_LAYERS)]
    nbytes = [W.q4_bytes(n, k) for _, n, k in shape.tensor_shapes()] * N_LAYERS
    total = sum(nbytes)
    assert total == 3_925_868_544 and len(nbytes) == 224
    budget = (60 * total) // 100  # floor(0.60 * total): "60 %" is read as bytes of the memory budget M
    chunk = 8 * MB

    # ---- what the oracle says the placement and the traffic must be
    want_where = O.static_placement(O.size_units(nbytes), nbytes, [0] * len(nbytes), O.budget_units(budget))
    pass_bytes, pass_copies, pass_order = O.streamed_dense(nbytes, [int(w) for w in want_where], chunk)
    want_resident = sum(b for b, w in zip(nbytes, want_where) if w)
    assert 0.55 * total < want_resident <= budget

    res = run_stack(B, torch, shape, layers, False, budget, chunk, capture=False)
    hyb = run_stack(B, torch, shape, layers, True, budget, chunk, capture=True)

    # ---- placement and bookkeeping: bit-exact
    assert list(hyb["where"]) == list(want_where)
    assert hyb["resident_bytes"] == want_resident and res["resident_bytes"] == total
    assert res["prefill_streamed"][0] == 0 and res["decode_streamed"][0] == 0
    n_host = len(nbytes) - int(np.sum(want_where))
    assert hyb["prefill_streamed"] == (pass_bytes, pass_copies, n_host)  # one pass over the host-placed tensors
    assert hyb["decode_streamed"] == (N_STEPS * pass_bytes, N_STEPS * pass_copies, N_STEPS * n_host)

    # ---- placement invariance: the same bits wherever the tensors live
    assert np.array_equal(res["prefill_y"].view(np.uint16), hyb["prefill_y"].view(np.uint16))
    for s in range(N_STEPS):
        assert np.array_equal(res["decode_ys"][s].view(np.uint16), hyb["decode_ys"][s].view(np.uint16)), s
    for l in range(N_LAYERS):
        assert np.array_equal(res["caches"][l][0], hyb["caches"][l][0]) and np.array_equal(res["caches"][l][1], hyb["caches"][l][1]), l
    assert all(np.isfinite(y.astype(np.float32)).all() for y in hyb["decode_ys"])

    # ---- single layers against the oracle, from what the library was given
    (e_dec, w_dec), (e_pre, w_pre) = hyb["numerics"]
    cap = hyb["capture"]
    drift = {}
    for l, s in DECODE_POINTS:
        pos = T_PREFILL + s
        kc, vc = cap[("decode", l, s, "k")].copy(), cap[("decode", l, s, "v")].copy()
        want = O.dense_layer(cap[("decode", l, s, "x")], H.oracle_dense_tensors(layers[l]), shape, kc, vc, pos, e_dec, w_dec)
        drift[(l, s)] = H.assert_close(cap[("decode", l, s, "y")], want, what=f"decode layer {l} step {s}")
    for l in PREFILL_LAYERS:
        kc = np.zeros((shape.n_kv_heads, CAP, shape.head_dim), dtype=np.float16)
        vc = np.zeros_like(kc)
        want = O.dense_layer(cap[("prefill", l, "x")], H.oracle_dense_tensors(layers[l]), shape, kc, vc, 0, e_pre, w_pre)
        H.assert_close(cap[("prefill", l, "y")], want, what=f"prefill layer {l}", elementwise="counted")
        for got, ref in ((cap[("prefill", l, "k")], kc), (cap[("prefill", l, "v")], vc)):
            a, b = got[:, :T_PREFILL].astype(np.float64), ref[:, :T_PREFILL].astype(np.float64)
            assert np.max(np.abs(a - b)) <= 4e-3 * np.max(np.abs(b))  # fp16 outputs of an fp16-operand GEMM: a few ulps
            assert not got[:, T_PREFILL:].any()
