"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle's callers.

This module holds none of the method's arithmetic: it only draws numbers.  Every
tensor is a pure function of (seed, tensor_id, element index) through a counter-based
generator (splitmix64 -> Box-Muller), so any slice of any tensor can be regenerated
anywhere without state.  Values are drawn in fp64, scaled, and rounded ONCE to the
storage type (fp32, or bf16 with round-to-nearest-even); the rounded buffer is what
both the CPU oracle and the GPU path consume.

bf16 tensors are carried in numpy as uint16 bit patterns.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """One splitmix64 output step on an array of uint64 counters (wraps mod 2^64)."""
    with np.errstate(over="ignore"):
        z = x + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def uniform_bits(seed: int, tensor_id: int, n: int, lane: int = 0) -> np.ndarray:
    """n 64-bit words; word e depends only on (seed, tensor_id, e, lane)."""
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([np.uint64(seed) ^ (np.uint64(tensor_id) << np.uint64(32))], dtype=np.uint64))
        key = _splitmix64(key + np.uint64(lane))
        ctr = np.arange(n, dtype=np.uint64) * np.uint64(2) + key
        return _splitmix64(ctr)


def normal_f64(seed: int, tensor_id: int, shape, std: float = 1.0, mean: float = 0.0) -> np.ndarray:
    """N(mean, std^2) samples in fp64 (Box-Muller on two counter-based uniforms per element)."""
    n = int(np.prod(shape)) if len(shape) else 1
    a = uniform_bits(seed, tensor_id, n, 0)
    b = uniform_bits(seed, tensor_id, n, 1)
    # 53-bit uniforms; u1 in (0,1], u2 in [0,1)
    u1 = ((a >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
    u2 = (b >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (z * std + mean).reshape(shape)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern (uint16), round to nearest even.  No NaN inputs expected."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rnd = ((bits >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    with np.errstate(over="ignore"):
        return ((bits + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> exact fp64 value."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 via fp32 (the double rounding is harmless for test data)."""
    return f32_to_bf16_bits(np.asarray(x, dtype=np.float64).astype(np.float32))


def normal(seed: int, tensor_id: int, shape, std: float = 1.0, mean: float = 0.0, dtype: str = "f32") -> np.ndarray:
    """Storage-typed tensor: float32 array for "f32", uint16 bf16 bit patterns for "bf16"."""
    z = normal_f64(seed, tensor_id, shape, std, mean)
    if dtype == "f32":
        return z.astype(np.float32)
    if dtype == "bf16":
        return f64_to_bf16_bits(z).reshape(shape)
    raise ValueError(f"unknown dtype {dtype!r}")


def to_f64(a: np.ndarray) -> np.ndarray:
    """Exact fp64 value of a storage-typed tensor (uint16 is read as bf16 bits)."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f64(a).reshape(a.shape)
    return a.astype(np.float64)


# ----------------------------------------------------------------------------------------
# Workload recipes.  Shapes are those of Swin / LLM / diffusion-style transformer blocks;
# values are random and stand in for trained weights and real activations.
# ----------------------------------------------------------------------------------------

SEED_BASE = 0x5EED0000


def swin_inputs(config_id: int, B: int, H: int, W: int, C: int, heads: int, window: int,
                mlp_ratio: int, dtype: str, perturbed_affine: bool = True, zero_bias: bool = False,
                weight_set: int = 0) -> dict:
    """Tensors of one Swin block.  Linear weights are [out, in] (reduction dim contiguous).

    perturbed_affine: LayerNorm gamma = 1 + 0.02 N(0,1), beta = 0.02 N(0,1) (else 1 / 0).
    zero_bias:        linear biases exactly 0 (else 0.02 N(0,1)).
    weight_set:       selects an independent set of weights (for a block pair).
    """
    seed = SEED_BASE + config_id
    t = 100 * weight_set
    nb = (2 * window - 1) ** 2
    hid = C * mlp_ratio

    def affine(idx, n, one):
        if perturbed_affine:
            return normal(seed, idx, (n,), 0.02, 1.0 if one else 0.0, dtype)
        v = np.full((n,), 1.0 if one else 0.0)
        return v.astype(np.float32) if dtype == "f32" else f64_to_bf16_bits(v)

    def bias(idx, n):
        if zero_bias:
            v = np.zeros((n,))
            return v.astype(np.float32) if dtype == "f32" else f64_to_bf16_bits(v)
        return normal(seed, idx, (n,), 0.02, 0.0, dtype)

    d = {
        "x": normal(seed, 0, (B, H, W, C), 1.0, 0.0, dtype),
        "ln1_g": affine(t + 1, C, True), "ln1_b": affine(t + 2, C, False),
        "w_qkv": normal(seed, t + 3, (3 * C, C), 0.02, 0.0, dtype), "b_qkv": bias(t + 4, 3 * C),
        "rel_bias_table": normal(seed, t + 5, (nb, heads), 0.02, 0.0, dtype),
        "w_proj": normal(seed, t + 6, (C, C), 0.02, 0.0, dtype), "b_proj": bias(t + 7, C),
    }
    if mlp_ratio > 0:
        d.update({
            "ln2_g": affine(t + 8, C, True), "ln2_b": affine(t + 9, C, False),
            "w_fc1": normal(seed, t + 10, (hid, C), 0.02, 0.0, dtype), "b_fc1": bias(t + 11, hid),
            "w_fc2": normal(seed, t + 12, (C, hid), 0.02, 0.0, dtype), "b_fc2": bias(t + 13, C),
        })
    return d


def attn_layer_inputs(config_id: int, S: int, hidden: int, dtype: str = "bf16", B: int = 1) -> dict:
    """Tensors of one decoder attention layer (RMSNorm gain, fused QKV weight, output weight)."""
    seed = SEED_BASE + config_id
    return {
        "x": normal(seed, 0, (B, S, hidden), 1.0, 0.0, dtype),
        "rms_g": normal(seed, 1, (hidden,), 0.02, 1.0, dtype),
        "w_qkv": normal(seed, 2, (3 * hidden, hidden), 0.02, 0.0, dtype),
        "w_o": normal(seed, 3, (hidden, hidden), 0.02, 0.0, dtype),
    }


def decode_inputs(config_id: int, B: int, pos: int, hidden: int, heads: int, dtype: str = "bf16") -> dict:
    """Tensors of one decode step of the decoder attention layer: the layer's weights, one new token per
    sequence and a key/value cache of `pos` positions, logical shape [B, pos, heads, head_dim] (unit-variance
    values, like the keys and values a prefill of unit-variance activations leaves)."""
    seed = SEED_BASE + config_id
    d = attn_layer_inputs(config_id, 1, hidden, dtype, B)
    d["x"] = d["x"].reshape(B, hidden)
    d["k_cache"] = normal(seed, 4, (B, pos, heads, hidden // heads), 1.0, 0.0, dtype)
    d["v_cache"] = normal(seed, 5, (B, pos, heads, hidden // heads), 1.0, 0.0, dtype)
    return d


def chain_inputs(config_id: int, which: str, dtype: str = "bf16", small: bool = False) -> dict:
    """Inputs of the pure layout chains.

    "2a": two [B,S,H*D] activations (each goes reshape -> transpose(0,2,1,3) -> [B,H,S,D]).
    "2b": one NCHW activation and a [N,K] weight.
    """
    seed = SEED_BASE + config_id
    if which == "2a":
        B, S, H, D = (2, 96, 4, 64) if small else (8, 1024, 16, 64)
        return {"xq": normal(seed, 0, (B, S, H * D), 1.0, 0.0, dtype),
                "xk": normal(seed, 1, (B, S, H * D), 1.0, 0.0, dtype), "dims": (B, S, H, D)}
    if which == "2b":
        B, C, Hh, Ww, N = (2, 64, 8, 32, 128) if small else (8, 256, 64, 64, 256)
        return {"x": normal(seed, 2, (B, C, Hh, Ww), 1.0, 0.0, dtype),
                "w": normal(seed, 3, (N, C), 0.02, 0.0, dtype), "dims": (B, C, Hh, Ww, N)}
    raise ValueError(which)
