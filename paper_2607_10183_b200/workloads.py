"""Seeded synthetic inputs for the block-quantized per-tensor forward path.

This module only *draws inputs*: it holds none of the method's arithmetic (no
dequantization, no matmul, no routing, no placement).  Both the CPU oracle's
tests and the CUDA path's tests/benchmarks take their inputs from here, so the
two sides see byte-identical tensors without sharing any computation.

The tensors stand in for the dense and MoE checkpoints the paper evaluates
(Section 5.1: INT4 weights, batch 1, prompts of 512..4096 tokens): the real
weights are not available, so shapes and value distributions follow the
workload configurations instead:

* 4-bit codes uniform in [-8, 7], stored in the interchange format of the C
  ABI: row-major ``[N][K/2]`` bytes, byte ``j`` of a row holds code ``2j`` in
  its low nibble and code ``2j+1`` in its high nibble, both as two's-complement
  nibbles.  Drawing the *bytes* uniformly in [0, 255] gives exactly that
  distribution for every code, and is far cheaper than drawing codes one by one.
* one fp16 scale per block of 32 consecutive k of a row, ``|N(0, 0.02)|``.
* the microscaling 4-bit format (MXFP4, Section 5.1): element bytes uniform in [0, 255] (every 4-bit float encoding
  equally likely), one shared-exponent byte per block of 32 uniform in [119, 123] (block scales 2^-8 .. 2^-4, which
  gives weights of standard deviation about 0.1 like the other formats).
* unquantized fp16 weight matrices (the FP16 model of Section 5.1) ``N(0, 0.09)`` rounded to fp16: the
  standard deviation a dequantized weight of the recipe above has.
* activations and KV-cache entries ``N(0, 1)`` rounded to fp16.
* router weights ``N(0, 0.02)`` rounded to fp16.
* RMSNorm gains zero-mean normal, rounded to fp16: std 0.25 in the dense layers, std 1 in the MoE
  block.  Zero-mean gains keep a deep stack of such synthetic layers inside the fp16 range (all-ones
  gains overflow in the second layer).  The dense std of 0.25 keeps attention logits at an LLM-like
  magnitude (std about 2): with unit-variance gains the new token's self-score has std about 36, the
  softmax degenerates to a near-argmax, and a one-ulp difference in the fp16 rounding of a cached key
  moves the layer output by 1e-3, which no fp32 implementation can avoid and no tolerance can absorb.

Every stream is ``numpy.random.default_rng([0, config, layer, role, part, step])``
so "all values come from seed 0" and any tensor can be regenerated alone.
"""
from __future__ import annotations

import dataclasses
import numpy as np

# roles (the tag that selects a random stream)
ROLE_Q, ROLE_K, ROLE_V, ROLE_O, ROLE_GATE, ROLE_UP, ROLE_DOWN = 0, 1, 2, 3, 4, 5, 6
ROLE_ROUTER, ROLE_ATTN_NORM, ROLE_FFN_NORM, ROLE_X, ROLE_KCACHE, ROLE_VCACHE = 7, 8, 9, 10, 11, 12
PART_CODES, PART_SCALES, PART_W16, PART_MXSCALE = 0, 1, 2, 3

BLOCK = 32  # weights per quantization block


def stream(config: int, layer: int, role: int, part: int = 0, step: int = 0) -> np.random.Generator:
    """The random stream of one tensor part (seed 0 plus a tag)."""
    return np.random.default_rng([0, int(config), int(layer), int(role), int(part), int(step)])


def q4_packed(config: int, layer: int, role: int, n_out: int, k_in: int, n_experts: int = 1):
    """A block-quantized weight in the interchange format.

    Returns ``(packed, scales)``: ``packed`` uint8 ``[E][N][K/2]`` (``[N][K/2]``
    when ``n_experts == 1``), ``scales`` float16 ``[E][N][K/32]``.
    """
    assert k_in % BLOCK == 0
    shape_c = (n_out, k_in // 2) if n_experts == 1 else (n_experts, n_out, k_in // 2)
    shape_s = (n_out, k_in // BLOCK) if n_experts == 1 else (n_experts, n_out, k_in // BLOCK)
    packed = stream(config, layer, role, PART_CODES).integers(0, 256, size=shape_c, dtype=np.uint8)
    scales = np.abs(stream(config, layer, role, PART_SCALES).normal(0.0, 0.02, size=shape_s)).astype(np.float16)
    return packed, scales


def codes_to_packed(codes: np.ndarray) -> np.ndarray:
    """Lay signed codes in [-8, 7] (int8 ``[..., K]``) out as interchange bytes ``[..., K/2]``.

    Pure byte layout (the ABI's input format); used by tests that want to choose
    the codes themselves.
    """
    c = np.asarray(codes)
    assert c.shape[-1] % 2 == 0 and c.min() >= -8 and c.max() <= 7
    u = (c.astype(np.int16) & 0xF).astype(np.uint8)
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def mxfp4_packed(config: int, layer: int, role: int, n_out: int, k_in: int, n_experts: int = 1):
    """A weight in the microscaling 4-bit format: ``(packed, scale_bytes)`` with ``packed`` uint8 ``[E][N][K/2]``
    (two elements per byte, even k in the low nibble) and ``scale_bytes`` uint8 ``[E][N][K/32]`` (biased exponents)."""
    assert k_in % BLOCK == 0
    shape_c = (n_out, k_in // 2) if n_experts == 1 else (n_experts, n_out, k_in // 2)
    shape_s = (n_out, k_in // BLOCK) if n_experts == 1 else (n_experts, n_out, k_in // BLOCK)
    packed = stream(config, layer, role, PART_CODES).integers(0, 256, size=shape_c, dtype=np.uint8)
    scale_bytes = stream(config, layer, role, PART_MXSCALE).integers(119, 124, size=shape_s, dtype=np.uint8)
    return packed, scale_bytes


def activations(config: int, layer: int, shape, step: int = 0, role: int = ROLE_X) -> np.ndarray:
    """fp16 activations ~N(0,1)."""
    return stream(config, layer, role, 0, step).normal(0.0, 1.0, size=shape).astype(np.float16)


DENSE_GAIN_STD = 0.25
MOE_GAIN_STD = 1.0


def norm_gain(config: int, layer: int, role: int, hidden: int, std: float = DENSE_GAIN_STD) -> np.ndarray:
    return stream(config, layer, role, 0).normal(0.0, std, size=(hidden,)).astype(np.float16)


def router_weight(config: int, layer: int, hidden: int, n_experts: int) -> np.ndarray:
    """fp16 router weight ``[hidden][n_experts]`` ~N(0, 0.02)."""
    return stream(config, layer, ROLE_ROUTER, 0).normal(0.0, 0.02, size=(hidden, n_experts)).astype(np.float16)


def kv_cache(config: int, layer: int, n_kv_heads: int, capacity: int, head_dim: int, filled: int):
    """fp16 K and V caches ``[n_kv][capacity][head_dim]``; the first ``filled`` positions ~N(0,1), rest zero."""
    k = np.zeros((n_kv_heads, capacity, head_dim), dtype=np.float16)
    v = np.zeros((n_kv_heads, capacity, head_dim), dtype=np.float16)
    if filled:
        k[:, :filled] = stream(config, layer, ROLE_KCACHE, 0).normal(0.0, 1.0, size=(n_kv_heads, filled, head_dim)).astype(np.float16)
        v[:, :filled] = stream(config, layer, ROLE_VCACHE, 0).normal(0.0, 1.0, size=(n_kv_heads, filled, head_dim)).astype(np.float16)
    return k, v


@dataclasses.dataclass(frozen=True)
class DenseShape:
    hidden: int = 4096
    n_q_heads: int = 32
    n_kv_heads: int = 8
    head_dim: int = 128
    ffn: int = 14336
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    def tensor_shapes(self):
        """(role, n_out, k_in) of the seven projections in execution order."""
        qd, kvd = self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim
        return [(ROLE_Q, qd, self.hidden), (ROLE_K, kvd, self.hidden), (ROLE_V, kvd, self.hidden),
                (ROLE_O, self.hidden, qd), (ROLE_GATE, self.ffn, self.hidden), (ROLE_UP, self.ffn, self.hidden),
                (ROLE_DOWN, self.hidden, self.ffn)]


@dataclasses.dataclass(frozen=True)
class MoEShape:
    hidden: int = 2048
    n_experts: int = 128
    ffn: int = 768
    top_k: int = 8
    rms_eps: float = 1e-5


# small shapes with the same structure, for tests the oracle finishes in seconds
DENSE_SMALL = DenseShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=448)
DENSE_FULL = DenseShape()
MOE_SMALL = MoEShape(hidden=128, n_experts=16, ffn=96, top_k=4)
MOE_FULL = MoEShape()


def dense_layer(config: int, layer: int, shape: DenseShape = DENSE_FULL, gain_std: float = DENSE_GAIN_STD) -> dict:
    """All tensors of one dense decoder layer: ``{role: (packed, scales)}`` plus the two norm gains ~N(0, gain_std)."""
    out = {"shape": shape}
    for role, n_out, k_in in shape.tensor_shapes():
        out[role] = q4_packed(config, layer, role, n_out, k_in)
    out[ROLE_ATTN_NORM] = norm_gain(config, layer, ROLE_ATTN_NORM, shape.hidden, gain_std)
    out[ROLE_FFN_NORM] = norm_gain(config, layer, ROLE_FFN_NORM, shape.hidden, gain_std)
    return out


def w16_matrix(config: int, layer: int, role: int, n_out: int, k_in: int) -> np.ndarray:
    """An unquantized fp16 weight matrix ``[N][K]``."""
    return stream(config, layer, role, PART_W16).normal(0.0, 0.09, size=(n_out, k_in)).astype(np.float16)


def dense_layer_w16(config: int, layer: int, shape: DenseShape = DENSE_FULL) -> dict:
    """A dense decoder layer whose seven matrices are unquantized fp16: ``{role: (w16,)}`` plus the norm gains."""
    out = {"shape": shape}
    for role, n_out, k_in in shape.tensor_shapes():
        out[role] = (w16_matrix(config, layer, role, n_out, k_in),)
    out[ROLE_ATTN_NORM] = norm_gain(config, layer, ROLE_ATTN_NORM, shape.hidden)
    out[ROLE_FFN_NORM] = norm_gain(config, layer, ROLE_FFN_NORM, shape.hidden)
    return out


def dense_layer_mxfp4(config: int, layer: int, shape: DenseShape = DENSE_FULL) -> dict:
    """A dense decoder layer whose seven matrices are in the microscaling 4-bit format: ``{role: (packed, scale_bytes)}``."""
    out = {"shape": shape}
    for role, n_out, k_in in shape.tensor_shapes():
        out[role] = mxfp4_packed(config, layer, role, n_out, k_in)
    out[ROLE_ATTN_NORM] = norm_gain(config, layer, ROLE_ATTN_NORM, shape.hidden)
    out[ROLE_FFN_NORM] = norm_gain(config, layer, ROLE_FFN_NORM, shape.hidden)
    return out


def moe_block(config: int, layer: int, shape: MoEShape = MOE_FULL) -> dict:
    """All tensors of one MoE FFN block: stacked expert gate/up/down, router, norm gain."""
    out = {"shape": shape}
    out[ROLE_GATE] = q4_packed(config, layer, ROLE_GATE, shape.ffn, shape.hidden, shape.n_experts)
    out[ROLE_UP] = q4_packed(config, layer, ROLE_UP, shape.ffn, shape.hidden, shape.n_experts)
    out[ROLE_DOWN] = q4_packed(config, layer, ROLE_DOWN, shape.hidden, shape.ffn, shape.n_experts)
    out[ROLE_ROUTER] = router_weight(config, layer, shape.hidden, shape.n_experts)
    out[ROLE_FFN_NORM] = norm_gain(config, layer, ROLE_FFN_NORM, shape.hidden, MOE_GAIN_STD)
    return out


def moe_block_mxfp4(config: int, layer: int, shape: MoEShape = MOE_FULL) -> dict:
    """An MoE FFN block whose stacked expert tensors are in the microscaling 4-bit format (router and gain as before)."""
    out = moe_block(config, layer, shape)
    out[ROLE_GATE] = mxfp4_packed(config, layer, ROLE_GATE, shape.ffn, shape.hidden, shape.n_experts)
    out[ROLE_UP] = mxfp4_packed(config, layer, ROLE_UP, shape.ffn, shape.hidden, shape.n_experts)
    out[ROLE_DOWN] = mxfp4_packed(config, layer, ROLE_DOWN, shape.hidden, shape.ffn, shape.n_experts)
    return out


def q4_bytes(n_out: int, k_in: int) -> int:
    """Bytes of one block-quantized matrix: 4-bit codes plus one fp16 scale per 32 weights."""
    return n_out * k_in // 2 + n_out * (k_in // BLOCK) * 2
