"""Seeded random-init weights of a decoder shape, N(0, init_std^2), as float32 arrays.

For "bf16" shapes every value is rounded to the nearest-even bf16 and widened
back to float32, so both the CPU oracle and the device path consume exactly the
same numbers.  Data generation and format conversion only.

Layout (row-major, [out_features, in_features]):
  embed    [V, d]            lm_head = embed when tied
  per layer l:
    attn_norm [d]   wqkv [(n_q + 2 n_kv) * hd, d]  (q heads, then k heads, then v heads)
    wo        [d, n_q * hd]
    mlp_norm  [d]   w_gate_up [2 * d_ff, d]        (gate rows, then up rows)
    w_down    [d, d_ff]
  final_norm [d]
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np

from . import rng
from .configs import ModelShape

_CHUNK = 1 << 22


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> float32 holding the round-to-nearest-even bf16 value."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 (already bf16-representable) -> uint16 bit pattern."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _tensor(seed: int, tid: int, shape, std: float, bf16: bool) -> np.ndarray:
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)

    def fill(c0):
        c = min(_CHUNK, n - c0)
        v = rng.normal(seed, 1000 + tid, c0, c, std)
        out[c0:c0 + c] = round_to_bf16(v) if bf16 else v

    starts = range(0, n, _CHUNK)
    if n > _CHUNK:
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, starts))
    else:
        for c0 in starts:
            fill(c0)
    return out.reshape(shape)


def make_weights(m: ModelShape, seed: int = 0, *, gain_jitter: float = 0.0) -> dict:
    """All tensors of the decoder.  ``gain_jitter`` > 0 draws norm gains 1 + N(0, jitter^2)
    instead of exactly 1 (used by tests so that a misplaced gain is visible)."""
    bf = m.dtype == "bf16"
    d = m.d_model

    def gain(tid):
        g = np.ones(d, dtype=np.float32)
        if gain_jitter > 0:
            g = g + rng.normal(seed, 1000 + tid, 0, d, gain_jitter)
            g = round_to_bf16(g) if bf else g.astype(np.float32)
        return g

    w = {"embed": _tensor(seed, 1, (m.vocab, d), m.init_std, bf), "final_norm": gain(2), "layers": []}
    w["lm_head"] = w["embed"] if m.tied else _tensor(seed, 3, (m.vocab, d), m.init_std, bf)
    for l in range(m.n_layers):
        t = 16 * (l + 1)
        w["layers"].append({
            "attn_norm": gain(t + 0),
            "wqkv": _tensor(seed, t + 1, (m.qkv_rows, d), m.init_std, bf),
            "wo": _tensor(seed, t + 2, (d, m.q_dim), m.init_std, bf),
            "mlp_norm": gain(t + 3),
            "w_gate_up": _tensor(seed, t + 4, (2 * m.d_ff, d), m.init_std, bf),
            "w_down": _tensor(seed, t + 5, (d, m.d_ff), m.init_std, bf),
        })
    return w
