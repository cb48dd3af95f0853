"""Pins of the forward oracle: closed forms, invariants, and the same decoder assembled from
torch's CPU float64 library routines (linear, rms_norm, scaled_dot_product_attention, silu,
complex-number rotary embedding) as a second opinion."""
import copy

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle.model import OracleModel, apply_rope, argmax_and_gap, rms_norm, rope_tables
from workload import weights as W
from workload.configs import ModelShape

SHAPE = ModelShape(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ff=96, vocab=50,
                   dtype="f32", init_std=0.3)


def make(shape=SHAPE, dtype=np.float64, jitter=0.2, untie=True):
    w = W.make_weights(shape, seed=3, gain_jitter=jitter)
    if untie:
        w["lm_head"] = W.make_weights(ModelShape(0, shape.d_model, 1, 1, 2, 2, shape.vocab, "f32", init_std=0.3),
                                      seed=9)["embed"]
    return OracleModel(shape, w, dtype), w


def torch_forward(shape, w, tokens):
    """Full-sequence causal forward in float64 from torch library routines."""
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    s = shape
    x = t(w["embed"])[torch.tensor(tokens)]
    R = len(tokens)
    half = s.head_dim // 2
    inv = 1.0 / (s.rope_base ** (torch.arange(0, half, dtype=torch.float64) * 2 / s.head_dim))
    rot = torch.polar(torch.ones(R, half, dtype=torch.float64), torch.arange(R, dtype=torch.float64)[:, None] * inv)

    def rope(u):  # u [R, H, hd]: pair element i with i + half, rotate as a complex number
        z = torch.complex(u[..., :half], u[..., half:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for lw in w["layers"]:
        h = F.rms_norm(x, (s.d_model,), t(lw["attn_norm"]), s.rms_eps)
        qkv = F.linear(h, t(lw["wqkv"]))
        q, k, v = qkv.split([s.q_dim, s.kv_dim, s.kv_dim], dim=-1)
        q = rope(q.view(R, s.n_q_heads, s.head_dim)).transpose(0, 1)
        k = rope(k.view(R, s.n_kv_heads, s.head_dim)).transpose(0, 1)
        v = v.view(R, s.n_kv_heads, s.head_dim).transpose(0, 1)
        o = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True, enable_gqa=True)[0]
        x = x + F.linear(o.transpose(0, 1).reshape(R, s.q_dim), t(lw["wo"]))
        h = F.rms_norm(x, (s.d_model,), t(lw["mlp_norm"]), s.rms_eps)
        g, u = F.linear(h, t(lw["w_gate_up"])).split([s.d_ff, s.d_ff], dim=-1)
        x = x + F.linear(F.silu(g) * u, t(lw["w_down"]))
    return F.linear(F.rms_norm(x, (s.d_model,), t(w["final_norm"]), s.rms_eps), t(w["lm_head"])).numpy()


def test_matches_torch_float64_library_decoder():
    m, w = make()
    tokens = np.random.default_rng(0).integers(0, SHAPE.vocab, 23).tolist()
    got = m.forward(tokens, m.new_cache(32))
    want = torch_forward(SHAPE, w, tokens)
    assert np.abs(got - want).max() < 1e-10
    assert np.abs(want).max() > 0.5   # the comparison is not vacuous


def test_float32_oracle_close_to_float64():
    m64, w = make()
    m32 = OracleModel(SHAPE, w, np.float32)
    tokens = np.random.default_rng(1).integers(0, SHAPE.vocab, 17).tolist()
    a = m64.forward(tokens, m64.new_cache(32))
    b = m32.forward(tokens, m32.new_cache(32))
    assert b.dtype == np.float32
    assert np.abs(a - b).max() < 1e-4


def test_incremental_with_cache_equals_full_and_chunked():
    m, _ = make()
    tokens = np.random.default_rng(2).integers(0, SHAPE.vocab, 19).tolist()
    full = m.forward(tokens, m.new_cache(32))
    c = m.new_cache(32)
    inc = np.concatenate([m.forward([t], c) for t in tokens])
    assert np.abs(full - inc).max() < 1e-11
    c = m.new_cache(32)
    chunked = np.concatenate([m.forward(tokens[:7], c), m.forward(tokens[7:12], c), m.forward(tokens[12:], c)])
    assert np.abs(full - chunked).max() < 1e-11


def test_rollback_then_recompute():
    m, _ = make()
    tokens = np.random.default_rng(3).integers(0, SHAPE.vocab, 12).tolist()
    c = m.new_cache(32)
    m.forward(tokens[:8], c)
    m.forward([1, 2, 3, 4], c)            # speculative rows that get rejected
    c.truncate(8)
    again = m.forward(tokens[8:], c)
    ref = m.forward(tokens, m.new_cache(32))[8:]
    assert np.abs(again - ref).max() < 1e-11


def test_causality_bitwise():
    m, _ = make(dtype=np.float32)
    r = np.random.default_rng(4)
    a = r.integers(0, SHAPE.vocab, 16).tolist()
    b = a[:9] + r.integers(0, SHAPE.vocab, 7).tolist()
    la = m.forward(a, m.new_cache(16))
    lb = m.forward(b, m.new_cache(16))
    assert np.array_equal(la[:9], lb[:9]) and not np.array_equal(la[9:], lb[9:])


def test_zero_blocks_reduce_to_norm_times_lm_head():
    m, w = make()
    for lw in m.layers:
        lw["wo"] = np.zeros_like(lw["wo"])
        lw["w_down"] = np.zeros_like(lw["w_down"])
    tokens = [3, 8, 8, 1]
    e = np.asarray(w["embed"], np.float64)[tokens]
    want = (e / np.sqrt((e * e).mean(-1, keepdims=True) + SHAPE.rms_eps) * w["final_norm"]) @ np.asarray(w["lm_head"], np.float64).T
    assert np.abs(m.forward(tokens, m.new_cache(8)) - want).max() < 1e-12


def test_rope_properties():
    hd = 16
    r = np.random.default_rng(5)
    q, k = r.standard_normal((1, 1, hd)), r.standard_normal((1, 1, hd))
    c0, s0 = rope_tables([0], hd, 10000.0, np.float64)
    assert np.array_equal(apply_rope(q, c0, s0), q)                       # position 0 is the identity
    def at(x, p):
        c, s = rope_tables([p], hd, 10000.0, np.float64)
        return apply_rope(x, c, s)
    assert abs(np.linalg.norm(at(q, 37)) - np.linalg.norm(q)) < 1e-12     # a rotation
    d1 = float((at(q, 11) * at(k, 4)).sum())
    d2 = float((at(q, 107) * at(k, 100)).sum())
    assert abs(d1 - d2) < 1e-12                                           # depends on the offset only
    # first pair rotates by exactly `pos` radians (frequency base^0 = 1); last pair by pos * base^(-(hd-2)/hd)
    x = np.zeros((1, 1, hd)); x[0, 0, 0] = 1.0
    y = at(x, 2)
    assert abs(y[0, 0, 0] - np.cos(2.0)) < 1e-15 and abs(y[0, 0, hd // 2] - np.sin(2.0)) < 1e-15
    x = np.zeros((1, 1, hd)); x[0, 0, hd // 2 - 1] = 1.0
    y = at(x, 3)
    ang = 3.0 * 10000.0 ** (-(hd - 2) / hd)
    assert abs(y[0, 0, hd // 2 - 1] - np.cos(ang)) < 1e-15 and abs(y[0, 0, hd - 1] - np.sin(ang)) < 1e-15


def attention_probe(q_zero: bool):
    """One layer whose residual output exposes the attention result: W_o = identity, MLP off."""
    shape = ModelShape(1, 32, 2, 1, 16, 8, 20, "f32", init_std=0.5)
    w = W.make_weights(shape, seed=11)
    lw = w["layers"][0]
    lw["wo"] = np.eye(32, dtype=np.float32)
    lw["w_down"] = np.zeros_like(lw["w_down"])
    if q_zero:
        lw["wqkv"][:shape.q_dim] = 0
    return shape, w


def test_zero_queries_average_the_values_causally():
    shape, w = attention_probe(q_zero=True)
    m = OracleModel(shape, w, np.float64)
    tokens = [1, 5, 9, 5, 2]
    e = np.asarray(w["embed"], np.float64)[tokens]
    h = rms_norm(e, np.ones(32), shape.rms_eps)
    v = h @ np.asarray(w["layers"][0]["wqkv"], np.float64)[shape.q_dim + shape.kv_dim:].T      # [R, 16], one KV head
    x_after = e + np.concatenate([np.cumsum(v, 0) / np.arange(1, 6)[:, None]] * 2, axis=1)      # both q heads read KV head 0
    want = rms_norm(x_after, np.ones(32), shape.rms_eps) @ np.asarray(w["embed"], np.float64).T
    assert np.abs(m.forward(tokens, m.new_cache(8)) - want).max() < 1e-12


def test_single_token_attention_returns_its_value():
    shape, w = attention_probe(q_zero=False)
    m = OracleModel(shape, w, np.float64)
    e = np.asarray(w["embed"], np.float64)[[7]]
    h = rms_norm(e, np.ones(32), shape.rms_eps)
    v = h @ np.asarray(w["layers"][0]["wqkv"], np.float64)[shape.q_dim + shape.kv_dim:].T
    want = rms_norm(e + np.concatenate([v, v], axis=1), np.ones(32), shape.rms_eps) @ np.asarray(w["embed"], np.float64).T
    assert np.abs(m.forward([7], m.new_cache(2)) - want).max() < 1e-12


def test_gqa_head_mapping_against_expanded_mha():
    """A GQA model equals the MHA model whose K/V projections repeat each KV head n_q/n_kv times."""
    m, w = make()
    s = SHAPE
    g = s.n_q_heads // s.n_kv_heads
    w2 = copy.deepcopy(w)
    for lw in w2["layers"]:
        q = lw["wqkv"][:s.q_dim]
        k = lw["wqkv"][s.q_dim:s.q_dim + s.kv_dim].reshape(s.n_kv_heads, s.head_dim, -1)
        v = lw["wqkv"][s.q_dim + s.kv_dim:].reshape(s.n_kv_heads, s.head_dim, -1)
        lw["wqkv"] = np.concatenate([q, np.repeat(k, g, 0).reshape(s.q_dim, -1), np.repeat(v, g, 0).reshape(s.q_dim, -1)])
    mha = OracleModel(ModelShape(s.n_layers, s.d_model, s.n_q_heads, s.n_q_heads, s.head_dim, s.d_ff, s.vocab, "f32"),
                      w2, np.float64)
    tokens = [4, 9, 1, 1, 30, 2]
    assert np.abs(m.forward(tokens, m.new_cache(8)) - mha.forward(tokens, mha.new_cache(8))).max() < 1e-11


def test_argmax_smallest_id_on_ties_and_gap():
    l = np.array([[0.0, 2.0, 2.0, 1.0], [5.0, 1.0, 4.5, 0.0]])
    idx, gap = argmax_and_gap(l)
    assert idx.tolist() == [1, 0] and gap.tolist() == [0.0, 0.5]


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -3.14159, 1e-30], dtype=np.float32)
    want = torch.tensor(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(W.round_to_bf16(x), want)
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    assert np.array_equal(W.round_to_bf16(r), torch.tensor(r).to(torch.bfloat16).to(torch.float32).numpy())
    assert np.array_equal(W.bf16_bits(W.round_to_bf16(r)).view(np.int16),
                          torch.tensor(r).to(torch.bfloat16).view(torch.int16).numpy())


def test_bf16_cache_cells_round_to_nearest_even():
    """The oracle's own model of a bf16 memory cell against the published format: hand-picked ties and halves,
    a library conversion (torch) on random values, and idempotence."""
    from oracle.model import to_bf16_storage
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1); 1 + 3 * 2^-8 is a tie -> even (1 + 2^-6)
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -2.5, 0.0],
                 dtype=np.float32)
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -2.5, 0.0], dtype=np.float32)
    assert np.array_equal(to_bf16_storage(x), want)
    r = (np.random.default_rng(1).standard_normal(20000) * np.float32(37.0)).astype(np.float32)
    got = to_bf16_storage(r)
    assert np.array_equal(got, torch.tensor(r).to(torch.bfloat16).to(torch.float32).numpy())
    assert np.array_equal(to_bf16_storage(got), got)
    assert np.all(np.abs(got - r) <= np.abs(r) * 2.0 ** -8)            # half a unit in the last of 8 significand bits


def test_bf16_shapes_store_their_cache_in_bf16_and_float32_shapes_do_not():
    from dataclasses import replace
    from oracle.model import to_bf16_storage
    shape16 = replace(SHAPE, dtype="bf16")
    w = W.make_weights(shape16, seed=3, gain_jitter=0.2)
    toks = [3, 14, 15, 9, 2, 6]
    m16 = OracleModel(shape16, w, np.float32)
    c16 = m16.new_cache(8)
    m16.forward(toks, c16)
    for l in range(shape16.n_layers):                                   # every cell holds a bf16 value
        assert np.array_equal(to_bf16_storage(c16.k[l]), c16.k[l]) and np.array_equal(to_bf16_storage(c16.v[l]), c16.v[l])
    # what is stored is the rounding of what the float32-cache model computes for the first layer ...
    m32 = OracleModel(shape16, w, np.float32, kv_storage=None)
    c32 = m32.new_cache(8)
    m32.forward(toks, c32)
    assert np.array_equal(c16.k[0], to_bf16_storage(c32.k[0])) and np.array_equal(c16.v[0], to_bf16_storage(c32.v[0]))
    assert not np.array_equal(c32.k[0], c16.k[0])
    # ... incremental decoding reads the same stored cells as the one-pass forward: identical logits up to the
    # float32 order of operations, and a rolled-back cache recomputes the same cells
    c_inc = m16.new_cache(8)
    inc = np.concatenate([m16.forward([t], c_inc) for t in toks])
    c_one = m16.new_cache(8)
    one = m16.forward(toks, c_one)
    assert np.abs(inc - one).max() < 1e-5
    assert all(np.array_equal(c_inc.k[l][:, :6], c_one.k[l][:, :6]) for l in range(shape16.n_layers))
    # a float32 shape keeps float32 cells
    c = OracleModel(SHAPE, w, np.float32).new_cache(8)
    assert c.storage is None
