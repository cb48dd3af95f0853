"""CPU oracle of the target decoder-only LM forward (the verifier of Section 5.1).

TEST INFRASTRUCTURE ONLY: the product path never imports this package.  It shares
no code with the CUDA implementation.

The paper names the model families (Llama-3, Qwen2.5 style SLMs) but not the
architecture, which therefore follows the benchmark shapes: pre-norm decoder with
  x <- x + W_o Attn(RoPE(W_qkv RMSNorm(x)))
  x <- x + W_down (SiLU(W_gate h) * (W_up h)),  h = RMSNorm(x)
  logits = W_lm RMSNorm(x)
RMSNorm(x) = x / sqrt(mean(x^2) + eps) * g; causal softmax attention with scale
1/sqrt(head_dim); grouped-query attention, query head h reads KV head h // (n_q / n_kv);
RoPE in the rotate-half pairing (element i with i + head_dim/2), angle pos * base^(-2i/head_dim)
evaluated in float64 and rounded to the working type.

Arithmetic is plain numpy in ``dtype`` (float32 by default, float64 for the
pins); matrix products are numpy matmul calls, nothing is blocked or fused.
One sequence at a time; a batch is a loop.

Storage precision.  The paper fixes none; the benchmark's "decoder in bf16" configurations fix the
storage type of the model's state: weight matrices AND the KV cache hold bf16 values (the shapes'
``dtype`` field says so: storage type of weights and KV).  The oracle therefore receives weights that are
already rounded to bf16 and, for a bf16 shape, rounds K (after RoPE) and V to bf16, round-to-nearest-even,
at the moment they are written to the cache; everything is computed in ``dtype`` from those stored values.
(With a float32 cache the logits of the 28-layer shape at a 1,024-token context move by up to 3e-2, more
than the whole tolerance of the comparison -- the cache format is part of what is computed, not noise.)
``kv_storage=None`` keeps the cache in ``dtype`` (float32 shapes, and the float64 pins).
"""
from __future__ import annotations

import numpy as np


def to_bf16_storage(x):
    """The value a bf16 memory cell holds after x is written to it: the nearest number with an 8-bit significand
    (7 stored bits), ties to the even significand.  Computed on the float32 bit pattern: add 0x7FFF plus the lowest
    kept bit, then clear the 16 dropped bits."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lowest_kept = (bits >> np.uint32(16)) & np.uint32(1)
    return ((bits + np.uint32(0x7FFF) + lowest_kept) & np.uint32(0xFFFF0000)).view(np.float32)


class KVCache:
    """Per-layer K and V of one sequence: arrays [n_kv_heads, capacity, head_dim], ``length`` valid.
    ``storage`` = "bf16": values are rounded to bf16 when they are written (see the module header)."""

    def __init__(self, shape, capacity: int, dtype=np.float32, storage=None):
        self.k = [np.zeros((shape.n_kv_heads, capacity, shape.head_dim), dtype) for _ in range(shape.n_layers)]
        self.v = [np.zeros((shape.n_kv_heads, capacity, shape.head_dim), dtype) for _ in range(shape.n_layers)]
        self.length = 0
        self.storage = storage

    def stored(self, x):
        return to_bf16_storage(x).astype(x.dtype) if self.storage == "bf16" else x

    def truncate(self, length: int):
        """Roll back: positions >= length are dead and will be overwritten."""
        self.length = length


def rms_norm(x, g, eps):
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + x.dtype.type(eps)) * g


def rope_tables(positions, head_dim: int, base: float, dtype):
    half = head_dim // 2
    inv = np.float64(base) ** (-2.0 * np.arange(half, dtype=np.float64) / head_dim)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(dtype), np.sin(ang).astype(dtype)


def apply_rope(x, cos, sin):
    """x [rows, heads, head_dim]; cos, sin [rows, head_dim/2]."""
    half = x.shape[-1] // 2
    a, b = x[..., :half], x[..., half:]
    c, s = cos[:, None, :], sin[:, None, :]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x):
    return x / (1 + np.exp(-x))


class OracleModel:
    def __init__(self, shape, weights: dict, dtype=np.float32, kv_storage="shape"):
        self.s = shape
        self.dtype = dtype
        # "shape": the cache stores what the shape's dtype says (bf16 shapes: bf16 cells); None: cells of ``dtype``
        self.kv_storage = (("bf16" if shape.dtype == "bf16" else None) if kv_storage == "shape" else kv_storage)
        cast = lambda a: np.asarray(a, dtype=dtype)
        self.embed = cast(weights["embed"])
        self.lm_head = self.embed if weights["lm_head"] is weights["embed"] else cast(weights["lm_head"])
        self.final_norm = cast(weights["final_norm"])
        self.layers = [{k: cast(v) for k, v in lw.items()} for lw in weights["layers"]]

    def new_cache(self, capacity: int) -> KVCache:
        return KVCache(self.s, capacity, self.dtype, self.kv_storage)

    def hidden(self, tokens, cache: KVCache):
        """Final-norm hidden states [R, d] of R new tokens at positions cache.length..+R-1;
        appends their K and V to the cache."""
        s = self.s
        tokens = np.asarray(tokens, dtype=np.int64)
        R = tokens.size
        p0 = cache.length
        cos, sin = rope_tables(np.arange(p0, p0 + R), s.head_dim, s.rope_base, self.dtype)
        g = s.n_q_heads // s.n_kv_heads
        scale = self.dtype(1.0 / np.sqrt(s.head_dim))
        x = self.embed[tokens]
        for l, w in enumerate(self.layers):
            h = rms_norm(x, w["attn_norm"], s.rms_eps)
            qkv = h @ w["wqkv"].T
            q = qkv[:, :s.q_dim].reshape(R, s.n_q_heads, s.head_dim)
            k = qkv[:, s.q_dim:s.q_dim + s.kv_dim].reshape(R, s.n_kv_heads, s.head_dim)
            v = qkv[:, s.q_dim + s.kv_dim:].reshape(R, s.n_kv_heads, s.head_dim)
            q = apply_rope(q, cos, sin)
            k = apply_rope(k, cos, sin)
            cache.k[l][:, p0:p0 + R] = cache.stored(k.transpose(1, 0, 2))
            cache.v[l][:, p0:p0 + R] = cache.stored(v.transpose(1, 0, 2))
            attn = np.zeros((R, s.n_q_heads, s.head_dim), self.dtype)
            for hq in range(s.n_q_heads):
                K = cache.k[l][hq // g, :p0 + R]
                V = cache.v[l][hq // g, :p0 + R]
                sc = (q[:, hq] @ K.T) * scale                                  # [R, p0 + R]
                visible = np.arange(p0 + R)[None, :] <= (p0 + np.arange(R))[:, None]
                sc = np.where(visible, sc, -np.inf)
                sc = np.exp(sc - sc.max(axis=-1, keepdims=True))
                attn[:, hq] = (sc / sc.sum(axis=-1, keepdims=True)) @ V
            x = x + attn.reshape(R, s.q_dim) @ w["wo"].T
            h = rms_norm(x, w["mlp_norm"], s.rms_eps)
            gu = h @ w["w_gate_up"].T
            x = x + (silu(gu[:, :s.d_ff]) * gu[:, s.d_ff:]) @ w["w_down"].T
        cache.length = p0 + R
        return rms_norm(x, self.final_norm, s.rms_eps)

    def forward(self, tokens, cache: KVCache):
        """Logits [R, V] of R new tokens; appends their K and V to the cache."""
        return self.hidden(tokens, cache) @ self.lm_head.T

    def prefill(self, tokens, cache: KVCache, chunk: int = 256):
        """Run tokens through the model for their K and V only (no logits)."""
        tokens = np.asarray(tokens)
        for c0 in range(0, tokens.size, chunk):
            self.hidden(tokens[c0:c0 + chunk], cache)


def argmax_and_gap(logits):
    """Per row: (argmax with the smallest id on ties, top-1 minus top-2 logit)."""
    idx = np.argmax(logits, axis=-1)
    if logits.shape[-1] < 2:
        return idx, np.full(idx.shape, np.inf)
    top2 = np.partition(logits, -2, axis=-1)[..., -2:]
    return idx, (top2[..., 1] - top2[..., 0]).astype(np.float64)


def linear(x, w):
    """y = x W^T for row-major W [out_features, in_features] (the projection every layer uses)."""
    return x @ w.T
