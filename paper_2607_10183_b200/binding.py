"""Thin ctypes binding of libats.so: argument marshalling only, every step runs in the CUDA library.

The module-level ``ats_*`` functions mirror include/ats.h one to one.  ``Context`` is a small convenience
wrapper that owns the arena (a torch uint8 tensor), the two streams and the ``ats_ctx`` handle.
Importing this module fails loudly when the library has not been built; there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ATS_LIB_PATH") or os.path.join(HERE, "libats.so")  # ATS_LIB_PATH: another build of the same library

ATS_OK = 0
ATS_ERR_INVALID, ATS_ERR_SHAPE, ATS_ERR_NOMEM, ATS_ERR_BUDGET = -1, -2, -3, -4
ATS_ERR_STATE, ATS_ERR_CUDA, ATS_ERR_TIMEOUT, ATS_ERR_UNSUPPORTED = -5, -6, -7, -8
ATS_HOST, ATS_GPU = 0, 1
ATS_FMT_Q4B32, ATS_FMT_F16, ATS_FMT_W16, ATS_FMT_MXFP4 = 0, 1, 2, 3
ATS_OUT_F32, ATS_OUT_F16 = 0, 1
ATS_MODE_DECODE, ATS_MODE_PREFILL = 0, 1
ATS_FLAG_POISON_SLOTS, ATS_FLAG_SKIP_SCALE_CHECK, ATS_FLAG_TIME_KERNELS, ATS_FLAG_NO_PDL, ATS_FLAG_MOE_RING_ONLY = 1, 2, 4, 8, 16
ATS_FLAG_NO_GEMM_PAIR = 32
ATS_LAYER_NO_TOPK_RENORM = 1
ATS_STATS_LIST = 512
EDGES = ("h", "q", "k", "v", "q_rot", "a", "o", "x1", "h2", "g", "u", "act", "d")

EXPORTS = (
    "ats_init", "ats_destroy", "ats_last_error", "ats_register_tensor", "ats_tensor_slice_bytes", "ats_set_placement",
    "ats_plan_placement", "ats_get_placement", "ats_linear", "ats_linear_static_scratch", "ats_route_topk", "ats_moe_linear", "ats_layer_decode", "ats_layer_decode_host", "ats_embed", "ats_lm_head",
    "ats_layer_prefill", "ats_workspace_bytes", "ats_dequantize", "ats_get_numerics", "ats_get_stats", "ats_set_flags", "ats_reset_stats",
    "ats_sync", "ats_measure_h2d", "ats_measure_hbm_read", "ats_debug_fail_copies", "ats_debug_gemv_wait", "ats_debug_skip_stages", "ats_register_host_buffer", "ats_unregister_host_buffer", "ats_debug_decode_buffer", "ats_debug_prefill_buffer", "ats_host_solve_placement", "ats_host_repack_q4",
    "ats_host_unpack_q4", "ats_host_group_pairs", "ats_host_dynamic_transfer", "ats_host_transfer_latency", "ats_host_deviation",
    "ats_host_reschedule", "ats_profile_tensor", "ats_set_tensor_value",
)


class ats_config(C.Structure):
    _fields_ = [("arena", C.c_void_p), ("arena_bytes", C.c_uint64), ("compute_stream", C.c_void_p),
                ("transfer_stream", C.c_void_p), ("ring_slots", C.c_uint32), ("slot_bytes", C.c_uint64),
                ("chunk_bytes", C.c_uint64), ("workspace_bytes", C.c_uint64), ("device", C.c_int32), ("flags", C.c_uint32)]


class ats_tensor_desc(C.Structure):
    _fields_ = [("fmt", C.c_uint32), ("n_experts", C.c_uint32), ("n_out", C.c_uint32), ("k_in", C.c_uint32),
                ("layer", C.c_uint32), ("role", C.c_uint32), ("value", C.c_int64), ("switch_cost", C.c_int64)]


class ats_layer_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down", "router")] + \
               [(n, C.c_uint32) for n in ("hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "n_experts", "top_k", "kv_capacity")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("flags", C.c_uint32)]


class ats_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("resident_bytes", "aux_bytes", "host_store_bytes", "streamed_bytes", "copies",
                                          "kernel_launches", "ring_reuses", "host_syncs")] + \
               [("timed_launches", C.c_uint64 * 3), ("timed_work", C.c_uint64 * 3), ("timed_ms", C.c_double * 3),
                ("n_streamed", C.c_uint32), ("reserved", C.c_uint32),
                ("streamed_ids", C.c_int32 * ATS_STATS_LIST), ("streamed_experts", C.c_int32 * ATS_STATS_LIST)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_10183_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, u32, i32, u64 = C.c_void_p, C.c_uint32, C.c_int32, C.c_uint64
    P = C.POINTER
    sig = {
        "ats_init": (i32, [P(ats_config), P(vp)]),
        "ats_destroy": (i32, [vp]),
        "ats_last_error": (C.c_char_p, [vp]),
        "ats_register_tensor": (i32, [vp, P(ats_tensor_desc), vp, vp, P(i32)]),
        "ats_tensor_slice_bytes": (i32, [vp, i32, P(u64)]),
        "ats_set_placement": (i32, [vp, vp, vp, vp, u32]),
        "ats_plan_placement": (i32, [vp, u64, u32, vp, u32]),
        "ats_get_placement": (i32, [vp, i32, i32, P(C.c_uint8)]),
        "ats_linear": (i32, [vp, i32, vp, vp, u32]),
        "ats_linear_static_scratch": (i32, [vp, i32, vp, vp, u32]),
        "ats_route_topk": (i32, [vp, i32, vp, u32, u32, vp, vp]),
        "ats_moe_linear": (i32, [vp, i32, vp, vp, vp, u32, u32, u32]),
        "ats_layer_decode": (i32, [vp, P(ats_layer_desc), vp, vp, vp, vp, u32, u32]),
        "ats_layer_decode_host": (i32, [vp, P(ats_layer_desc), vp, vp, vp, vp, u32, u32]),
        "ats_embed": (i32, [vp, i32, vp, u32, vp]),
        "ats_lm_head": (i32, [vp, i32, i32, C.c_float, vp, vp, u32, vp]),
        "ats_layer_prefill": (i32, [vp, P(ats_layer_desc), vp, vp, vp, vp, u32, u32]),
        "ats_workspace_bytes": (u64, [P(ats_layer_desc), u32]),
        "ats_dequantize": (i32, [vp, i32, i32, vp, u32]),
        "ats_get_numerics": (i32, [vp, u32, P(u32), P(u32)]),
        "ats_get_stats": (i32, [vp, P(ats_stats)]),
        "ats_reset_stats": (i32, [vp]),
        "ats_set_flags": (i32, [vp, u32]),
        "ats_sync": (i32, [vp, u32]),
        "ats_measure_h2d": (i32, [vp, u64, u32, P(C.c_double)]),
        "ats_measure_hbm_read": (i32, [vp, u64, u32, P(C.c_double)]),
        "ats_debug_fail_copies": (i32, [vp, u32]),
        "ats_debug_gemv_wait": (i32, [vp, u64, i32]),
        "ats_debug_skip_stages": (i32, [vp, u32]),
        "ats_register_host_buffer": (i32, [vp, vp, u64]),
        "ats_unregister_host_buffer": (i32, [vp, vp]),
        "ats_debug_decode_buffer": (i32, [vp, P(ats_layer_desc), u32, u32, P(vp), P(u64)]),
        "ats_debug_prefill_buffer": (i32, [vp, P(ats_layer_desc), u32, u32, P(vp), P(u64)]),
        "ats_host_solve_placement": (i32, [vp, vp, vp, vp, u32, C.c_int64, vp, P(C.c_int64)]),
        "ats_host_repack_q4": (i32, [vp, vp, vp, u32, u32]),
        "ats_host_unpack_q4": (i32, [vp, vp, vp, u32, u32]),
        "ats_host_group_pairs": (i32, [vp, u32, u32, vp, vp, vp, vp]),
        "ats_profile_tensor": (i32, [vp, i32, vp, vp, u32, u32, P(C.c_double), P(C.c_double)]),
        "ats_set_tensor_value": (i32, [vp, i32, C.c_int64, C.c_int64]),
        "ats_host_dynamic_transfer": (i32, [vp, vp, vp, vp, vp, u32, vp, vp, P(C.c_double)]),
        "ats_host_transfer_latency": (i32, [vp, vp, vp, vp, vp, vp, vp, u32, P(C.c_double)]),
        "ats_host_deviation": (C.c_double, [vp, vp, u32]),
        "ats_host_reschedule": (i32, [vp, u32, vp, vp, C.c_double, C.c_double, C.c_double, P(C.c_double), vp, vp, P(C.c_int32)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()
for _name in EXPORTS:
    globals()[_name] = getattr(lib, _name)


class AtsError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"ats error {code}: {msg}")
        self.code = code


def _ptr(t):
    """Device/host address of a torch tensor, numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def layer_desc(*, hidden, ffn, attn_norm=-1, wq=-1, wk=-1, wv=-1, wo=-1, ffn_norm=-1, w_gate=-1, w_up=-1, w_down=-1,
               router=-1, n_q_heads=0, n_kv_heads=0, head_dim=0, n_experts=0, top_k=0, kv_capacity=0, rms_eps=1e-5,
               rope_theta=10000.0, flags=0) -> ats_layer_desc:
    return ats_layer_desc(attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down, router, hidden, n_q_heads, n_kv_heads,
                          head_dim, ffn, n_experts, top_k, kv_capacity, rms_eps, rope_theta, flags)


class Context:
    """Owns an arena, two streams and an ats_ctx.  Methods raise AtsError on a negative status."""

    def __init__(self, arena_bytes, workspace_bytes=0, ring_slots=0, slot_bytes=0, chunk_bytes=0, device=0, flags=0,
                 compute_stream=None):
        import torch
        self.torch = torch
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.arena = torch.empty(int(arena_bytes), dtype=torch.uint8, device=self.device)
        self.compute = compute_stream if compute_stream is not None else torch.cuda.Stream(device=self.device)
        self.transfer = torch.cuda.Stream(device=self.device)
        self.cfg = ats_config(self.arena.data_ptr(), int(arena_bytes), self.compute.cuda_stream, self.transfer.cuda_stream,
                              int(ring_slots), int(slot_bytes), int(chunk_bytes), int(workspace_bytes), int(device), int(flags))
        h = C.c_void_p()
        st = lib.ats_init(C.byref(self.cfg), C.byref(h))
        if st != ATS_OK:
            raise AtsError(st, "ats_init failed")
        self.h = h

    # ---- plumbing
    def check(self, st):
        if st != ATS_OK:
            raise AtsError(st, lib.ats_last_error(self.h).decode())
        return st

    def last_error(self):
        return lib.ats_last_error(self.h).decode()

    def close(self):
        if getattr(self, "h", None):
            lib.ats_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- registry / placement
    def register_q4(self, packed: np.ndarray, scales: np.ndarray, layer=0, role=0, value=-1, switch_cost=0) -> int:
        """A 4-bit block tensor: fp16 scales select the integer-code format, uint8 scale bytes the microscaling format."""
        if np.asarray(scales).dtype == np.uint8:
            return self.register_mxfp4(packed, scales, layer, role, value, switch_cost)
        packed = np.ascontiguousarray(packed, dtype=np.uint8)
        scales = np.ascontiguousarray(scales, dtype=np.float16)
        E = packed.shape[0] if packed.ndim == 3 else 1
        n_out, k_in = packed.shape[-2], packed.shape[-1] * 2
        d = ats_tensor_desc(ATS_FMT_Q4B32, E, n_out, k_in, layer, role, value, switch_cost)
        out = C.c_int32(-1)
        self.check(lib.ats_register_tensor(self.h, C.byref(d), packed.ctypes.data, scales.ctypes.data, C.byref(out)))
        return out.value

    def register_mxfp4(self, packed: np.ndarray, scale_bytes: np.ndarray, layer=0, role=0, value=-1, switch_cost=0) -> int:
        """Microscaling 4-bit floats [E][n_out][k_in/2] with one biased-exponent byte per block of 32."""
        packed = np.ascontiguousarray(packed, dtype=np.uint8)
        scale_bytes = np.ascontiguousarray(scale_bytes, dtype=np.uint8)
        E = packed.shape[0] if packed.ndim == 3 else 1
        n_out, k_in = packed.shape[-2], packed.shape[-1] * 2
        d = ats_tensor_desc(ATS_FMT_MXFP4, E, n_out, k_in, layer, role, value, switch_cost)
        out = C.c_int32(-1)
        self.check(lib.ats_register_tensor(self.h, C.byref(d), packed.ctypes.data, scale_bytes.ctypes.data, C.byref(out)))
        return out.value

    def register_w16(self, w: np.ndarray, layer=0, role=0, value=-1, switch_cost=0) -> int:
        """An unquantized fp16 weight matrix [n_out][k_in] (placed and streamed like a quantized tensor)."""
        w = np.ascontiguousarray(w, dtype=np.float16)
        n_out, k_in = w.shape
        d = ats_tensor_desc(ATS_FMT_W16, 1, n_out, k_in, layer, role, value, switch_cost)
        out = C.c_int32(-1)
        self.check(lib.ats_register_tensor(self.h, C.byref(d), w.ctypes.data, None, C.byref(out)))
        return out.value

    def profile_tensor(self, tid, x, y, M, iters=20):
        """Measured operator time of a dense weight tensor, resident and host-placed: (t_resident_us, t_host_us)."""
        a, b = C.c_double(), C.c_double()
        self.check(lib.ats_profile_tensor(self.h, tid, _ptr(x), _ptr(y), M, iters, C.byref(a), C.byref(b)))
        return a.value, b.value

    def set_tensor_value(self, tid, value, switch_cost=0):
        self.check(lib.ats_set_tensor_value(self.h, tid, int(value), int(switch_cost)))

    def register_f16(self, data: np.ndarray, layer=0, role=0) -> int:
        data = np.ascontiguousarray(data, dtype=np.float16)
        k_in, n_out = (1, data.shape[0]) if data.ndim == 1 else data.shape
        d = ats_tensor_desc(ATS_FMT_F16, 1, n_out, k_in, layer, role, -1, 0)
        out = C.c_int32(-1)
        self.check(lib.ats_register_tensor(self.h, C.byref(d), data.ctypes.data, None, C.byref(out)))
        return out.value

    def slice_bytes(self, tid) -> int:
        v = C.c_uint64()
        self.check(lib.ats_tensor_slice_bytes(self.h, tid, C.byref(v)))
        return v.value

    def set_placement(self, entries):
        """entries: iterable of (id, expert or -1, ATS_HOST/ATS_GPU)."""
        entries = list(entries)
        ids = np.array([e[0] for e in entries], dtype=np.int32)
        ex = np.array([e[1] for e in entries], dtype=np.int32)
        wh = np.array([e[2] for e in entries], dtype=np.uint8)
        return self.check(lib.ats_set_placement(self.h, ids.ctypes.data, ex.ctypes.data, wh.ctypes.data, len(entries)))

    def plan_placement(self, budget_bytes, n_q4, granule_bytes=0) -> np.ndarray:
        out = np.zeros(n_q4, dtype=np.uint8)
        self.check(lib.ats_plan_placement(self.h, int(budget_bytes), int(granule_bytes), out.ctypes.data, n_q4))
        return out

    def get_placement(self, tid, expert=0) -> int:
        v = C.c_uint8()
        self.check(lib.ats_get_placement(self.h, tid, expert, C.byref(v)))
        return v.value

    # ---- operators (device tensors in, device tensors out; all asynchronous)
    def linear(self, tid, x, y, M):
        return self.check(lib.ats_linear(self.h, tid, _ptr(x), _ptr(y), M))

    def linear_static_scratch(self, tid, x, y, M):
        """ats_linear with the split-K scratch in the library's fixed device array (allocates nothing)."""
        return self.check(lib.ats_linear_static_scratch(self.h, tid, _ptr(x), _ptr(y), M))

    def route_topk(self, router_id, h, M, k, ids, gates):
        return self.check(lib.ats_route_topk(self.h, router_id, _ptr(h), M, k, _ptr(ids), _ptr(gates)))

    def moe_linear(self, tid, x, ids, y, M, k, x_per_slot=0):
        return self.check(lib.ats_moe_linear(self.h, tid, _ptr(x), _ptr(ids), _ptr(y), M, k, x_per_slot))

    def layer_decode(self, desc, x_in, x_out, k_cache, v_cache, pos, M=1):
        return self.check(lib.ats_layer_decode(self.h, C.byref(desc), _ptr(x_in), _ptr(x_out), _ptr(k_cache), _ptr(v_cache), pos, M))

    def layer_decode_host(self, desc, x_in_host, x_out_host, k_cache, v_cache, pos, M=1):
        return self.check(lib.ats_layer_decode_host(self.h, C.byref(desc), _ptr(x_in_host), _ptr(x_out_host), _ptr(k_cache),
                                                    _ptr(v_cache), pos, M))

    def register_host_buffer(self, t):
        """Registers a pinned host tensor (torch) for host-driven calls; keep it alive until unregister_host_buffer/close."""
        return self.check(lib.ats_register_host_buffer(self.h, _ptr(t), int(t.numel() * t.element_size())))

    def unregister_host_buffer(self, t):
        return self.check(lib.ats_unregister_host_buffer(self.h, _ptr(t)))

    def embed(self, tid, token_ids, out, M):
        """Rows token_ids[m] (device int32) of a Q4B32 table as fp16 rows of `out` (device)."""
        return self.check(lib.ats_embed(self.h, tid, _ptr(token_ids), M, _ptr(out)))

    def lm_head(self, norm_id, head_id, eps, x, logits, M=1, scratch=None):
        """logits = W_head * RMSNorm(x); `scratch` (device fp16 [M][hidden]) is needed unless the one-launch form applies."""
        return self.check(lib.ats_lm_head(self.h, norm_id, head_id, eps, _ptr(x), _ptr(logits), M, _ptr(scratch)))

    def layer_prefill(self, desc, x_in, x_out, k_cache, v_cache, pos0, T):
        return self.check(lib.ats_layer_prefill(self.h, C.byref(desc), _ptr(x_in), _ptr(x_out), _ptr(k_cache), _ptr(v_cache), pos0, T))

    def dequantize(self, tid, expert, out, out_fmt):
        return self.check(lib.ats_dequantize(self.h, tid, expert, _ptr(out), out_fmt))

    def numerics(self, mode):
        m, w = C.c_uint32(), C.c_uint32()
        self.check(lib.ats_get_numerics(self.h, mode, C.byref(m), C.byref(w)))
        return frozenset(n for i, n in enumerate(EDGES) if m.value >> i & 1), w.value

    def stats(self) -> ats_stats:
        s = ats_stats()
        self.check(lib.ats_get_stats(self.h, C.byref(s)))
        return s

    def set_flags(self, flags):
        return self.check(lib.ats_set_flags(self.h, flags))

    def reset_stats(self):
        return self.check(lib.ats_reset_stats(self.h))

    def sync(self, timeout_ms=0):
        return self.check(lib.ats_sync(self.h, timeout_ms))

    def debug_gemv_wait(self, limit_cycles, withhold_tile=-1):
        return self.check(lib.ats_debug_gemv_wait(self.h, int(limit_cycles), int(withhold_tile)))

    def debug_skip_stages(self, mask):
        return self.check(lib.ats_debug_skip_stages(self.h, int(mask)))

    def debug_decode_buffer(self, desc, M, which, dtype):
        """Copy of an intermediate of the last ats_layer_decode call (see ats_debug_decode_buffer) as a numpy array."""
        ptr, nb = C.c_void_p(), C.c_uint64()
        self.check(lib.ats_debug_decode_buffer(self.h, C.byref(desc), M, which, C.byref(ptr), C.byref(nb)))
        off = ptr.value - self.arena.data_ptr()
        raw = self.arena[off:off + nb.value].cpu().numpy()
        return raw.view(dtype)

    def debug_prefill_buffer(self, desc, T, which):
        """fp16 copy of an intermediate of the last ats_layer_prefill call (see ats_debug_prefill_buffer)."""
        ptr, nb = C.c_void_p(), C.c_uint64()
        self.check(lib.ats_debug_prefill_buffer(self.h, C.byref(desc), T, which, C.byref(ptr), C.byref(nb)))
        off = ptr.value - self.arena.data_ptr()
        return self.arena[off:off + nb.value].cpu().numpy().view(np.float16).reshape(T, -1)

    def measure_h2d(self, nbytes, reps=10) -> float:
        v = C.c_double()
        self.check(lib.ats_measure_h2d(self.h, int(nbytes), reps, C.byref(v)))
        return v.value


def _measure_hbm_read(self, nbytes, reps=5) -> float:
    v = C.c_double()
    self.check(lib.ats_measure_hbm_read(self.h, int(nbytes), reps, C.byref(v)))
    return v.value


Context.measure_hbm_read = _measure_hbm_read


def workspace_bytes(desc: ats_layer_desc, max_tokens: int) -> int:
    return int(lib.ats_workspace_bytes(C.byref(desc), max_tokens))


def host_group_pairs(ids, E):
    """Stable sort of (token, slot) pairs by expert (host only).  Returns (order, pos, off, max_rows)."""
    ids = np.ascontiguousarray(ids, dtype=np.int32).reshape(-1)
    P = ids.size
    order, pos, off = np.zeros(P, np.int32), np.zeros(P, np.int32), np.zeros(E + 1, np.int32)
    mx = C.c_int32()
    st = lib.ats_host_group_pairs(ids.ctypes.data, P, E, order.ctypes.data, pos.ctypes.data, off.ctypes.data, C.byref(mx))
    if st != ATS_OK:
        raise AtsError(st, "ats_host_group_pairs")
    return order, pos, off, mx.value


ATS_ROUND_START, ATS_NO_TRANSFER = -1, -2


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def host_dynamic_transfer(b, t_gpu, t_host, c, w):
    """Algorithm 2 on plain arrays (host only).  Returns (latency, rb uint8 array, start int32 array)."""
    b = np.ascontiguousarray(b, dtype=np.uint8)
    tg, th, cc, ww = _f64(t_gpu), _f64(t_host), _f64(c), _f64(w)
    n = b.size
    rb, start, lat = np.zeros(n, np.uint8), np.zeros(n, np.int32), C.c_double()
    st = lib.ats_host_dynamic_transfer(b.ctypes.data, tg.ctypes.data, th.ctypes.data, cc.ctypes.data, ww.ctypes.data, n,
                                       rb.ctypes.data, start.ctypes.data, C.byref(lat))
    if st != ATS_OK:
        raise AtsError(st, "ats_host_dynamic_transfer")
    return lat.value, rb, start


def host_transfer_latency(rb, start, b, t_gpu, t_host, c, w):
    """The round latency T of Section 4.4.1 for a given plan (host only)."""
    rb, b = np.ascontiguousarray(rb, dtype=np.uint8), np.ascontiguousarray(b, dtype=np.uint8)
    start = np.ascontiguousarray(start, dtype=np.int32)
    tg, th, cc, ww = _f64(t_gpu), _f64(t_host), _f64(c), _f64(w)
    lat = C.c_double()
    st = lib.ats_host_transfer_latency(rb.ctypes.data, start.ctypes.data, b.ctypes.data, tg.ctypes.data, th.ctypes.data,
                                       cc.ctypes.data, ww.ctypes.data, b.size, C.byref(lat))
    if st != ATS_OK:
        raise AtsError(st, "ats_host_transfer_latency")
    return lat.value


def host_deviation(m_prev, m_cur):
    a, b = _f64(m_prev).reshape(-1), _f64(m_cur).reshape(-1)
    return float(lib.ats_host_deviation(a.ctypes.data, b.ctypes.data, a.size))


def host_reschedule(b, m_ref, m_cur, eps, tau, t_now, t_last, rb, start=None):
    """Algorithm 3 (host only).  m_ref (float64 [4n], updated in place), rb (uint8 [n]) and start (int32 [n], optional) are
    the caller's state arrays.  Returns (t_last, replanned)."""
    b = np.ascontiguousarray(b, dtype=np.uint8)
    assert m_ref.dtype == np.float64 and m_ref.flags.c_contiguous and rb.dtype == np.uint8
    cur = _f64(m_cur).reshape(-1)
    tl, did = C.c_double(t_last), C.c_int32()
    st = lib.ats_host_reschedule(b.ctypes.data, b.size, m_ref.ctypes.data, cur.ctypes.data, eps, tau, t_now, C.byref(tl),
                                 rb.ctypes.data, None if start is None else start.ctypes.data, C.byref(did))
    if st != ATS_OK:
        raise AtsError(st, "ats_host_reschedule")
    return tl.value, bool(did.value)


def host_solve_placement(s, r, c, M, is_expert=None):
    """Algorithm 1 on plain arrays (host only).  Returns (b uint8 array, objective)."""
    s = np.ascontiguousarray(s, dtype=np.int64)
    r = np.ascontiguousarray(r, dtype=np.int64)
    c = np.ascontiguousarray(c, dtype=np.int64)
    e = None if is_expert is None else np.ascontiguousarray(is_expert, dtype=np.uint8)
    b = np.zeros(len(s), dtype=np.uint8)
    obj = C.c_int64()
    st = lib.ats_host_solve_placement(s.ctypes.data, r.ctypes.data, c.ctypes.data, None if e is None else e.ctypes.data,
                                      len(s), int(M), b.ctypes.data, C.byref(obj))
    if st != ATS_OK:
        raise AtsError(st, "ats_host_solve_placement")
    return b, obj.value
