"""Pins of the model-derived bigram drafter (the comparison drafter of Section 6.2)."""
import numpy as np

from oracle import drafter as D
from oracle import ngrammys as NG
from oracle.model import OracleModel
from workload import weights as W
from workload.configs import ModelShape

SHAPE = ModelShape(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ff=48, vocab=40, dtype="f32")


def test_table_is_the_argmax_of_a_single_token_forward():
    om = OracleModel(SHAPE, W.make_weights(SHAPE, 3, gain_jitter=0.2), np.float64)
    table, gap = NG.bigram_table(om)
    assert table.shape == (SHAPE.vocab,) and (gap >= 0).all()
    # the same through one long "batch" of unrelated sequences is not allowed to matter: every row is its own sequence
    for t in (0, 7, 39):
        logits = om.forward([t], om.new_cache(4))
        assert table[t] == int(np.argmax(logits[0]))
    # a single token attends to itself only: the table does not change when the same token is fed at position 0 of a
    # longer sequence (causality)
    for t in (3, 11):
        logits = om.forward([t, 5, 9], om.new_cache(4))
        assert table[t] == int(np.argmax(logits[0]))


def test_closed_form_with_zeroed_blocks():
    """With the attention and MLP blocks zeroed the logits of token t are RMSNorm(E[t]) . E[x]: for unit gains the table
    is the nearest embedding by inner product, computed here directly."""
    w = W.make_weights(SHAPE, 5)
    for lw in w["layers"]:
        lw["wo"] = np.zeros_like(lw["wo"])
        lw["w_down"] = np.zeros_like(lw["w_down"])
    om = OracleModel(SHAPE, w, np.float64)
    E = np.asarray(w["embed"], np.float64)
    want = np.argmax(E @ E.T, axis=1)               # the positive RMS factor of row t does not move its argmax
    table, _ = NG.bigram_table(om)
    assert np.array_equal(table, want)


def test_drafting_from_the_table():
    table = np.array([1, 2, 3, 4, 0, 5])
    ng = NG.as_ngram_model(table)
    assert ng.canonical() == [(1, (t,), int(x), 1) for t, x in enumerate(table)]
    # weight 1: the chain t -> table[t] -> table[table[t]] ...
    assert D.draft(ng, [5, 0], 4, 1, 1) == [1, 2, 3, 4]
    # the point mass wins from lambda = 1/2 on, whatever the context says
    ctx = [0, 3, 9, 0, 3, 9, 0]                     # the context drafter predicts 3 after 0, the bigram 1
    assert D.draft(ng, ctx, 1, 3, 4) == [1]
    assert D.draft(ng, ctx, 1, 1, 2) == [1]          # tie 1/2 : 1/2 -> smallest id
    # small weight: the context drafter where it has a match, the bigram elsewhere
    assert D.draft(ng, ctx, 3, 1, 256) == [3, 9, 0]
    assert D.draft(ng, [7, 7, 2], 2, 1, 256) == [3, 4]     # no earlier occurrence of 2: the bigram
    # weight 0: context only; without a match the last resort (token 0)
    assert D.draft(ng, [7, 7, 2], 1, 0, 1) == [0]
