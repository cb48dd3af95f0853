"""Pins of the corpus-statistics oracle: closed forms, hand-worked corpora, a library routine as a second
opinion, brute force, and properties that a dropped term, a wrong base or a crossed document boundary breaks."""
import math

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import corpus_stats as S


def test_hand_worked_corpus():
    # documents [1 2 1 2 3] and [1 2]: pairs (1,2) x3, (2,1) x1, (2,3) x1 -> p = 3/5, 1/5, 1/5
    tokens = np.array([1, 2, 1, 2, 3, 1, 2])
    offsets = np.array([0, 5, 7])
    bg = S.bigram_counts(tokens, offsets)
    assert dict(bg) == {(1, 2): 3, (2, 1): 1, (2, 3): 1}
    h = -(0.6 * math.log2(0.6) + 2 * 0.2 * math.log2(0.2))
    assert abs(h - 1.3709505944546687) < 1e-15
    r = S.corpus_stats(tokens, offsets, vocab=8)
    assert r["n_tokens"] == 7 and r["n_bigrams"] == 5 and r["n_unique_bigrams"] == 3 and r["n_unique_tokens"] == 3
    assert abs(r["bigram_entropy_bits"] - h) < 1e-12
    assert r["bigrams_for_cdf"] == 2                      # 3/5 < 0.8 <= 4/5
    # tokens: 1 x3, 2 x3, 3 x1
    ht = -(2 * (3 / 7) * math.log2(3 / 7) + (1 / 7) * math.log2(1 / 7))
    assert abs(r["token_entropy_bits"] - ht) < 1e-12
    assert abs(r["token_entropy_normalised"] - ht / 3.0) < 1e-12          # log2 8 = 3
    assert abs(r["token_renyi2_bits"] + math.log2((9 + 9 + 1) / 49)) < 1e-12
    assert abs(r["typical_set_size"] - 2 ** h) < 1e-12


def test_pairs_do_not_cross_document_boundaries():
    tokens = np.array([4, 5, 6])
    assert sum(S.bigram_counts(tokens, np.array([0, 1, 2, 3])).values()) == 0
    assert dict(S.bigram_counts(tokens, np.array([0, 2, 3]))) == {(4, 5): 1}
    assert dict(S.bigram_counts(tokens, np.array([0, 0, 3, 3]))) == {(4, 5): 1, (5, 6): 1}
    r = S.corpus_stats(np.zeros(0, np.int64), np.array([0]), vocab=16)
    assert r["n_bigrams"] == 0 and r["bigram_entropy_bits"] == 0.0 and r["bigrams_for_cdf"] == 0


@pytest.mark.parametrize("n", [1, 2, 5, 64, 1000])
def test_uniform_distribution_closed_forms(n):
    counts = [7] * n
    assert abs(S.shannon_entropy_bits(counts) - math.log2(n)) < 1e-10
    assert abs(S.renyi_entropy_bits(counts, 2.0) - math.log2(n)) < 1e-10     # every Renyi order equals log n
    assert abs(S.renyi_entropy_bits(counts, 0.5) - math.log2(n)) < 1e-10
    assert S.n_for_cdf(counts, 4, 5) == math.ceil(0.8 * n - 1e-12)           # typical set = the whole support
    assert S.n_for_cdf(counts, 1, 1) == n


def test_two_point_distribution():
    counts = [1, 3]                                                          # p = 1/4, 3/4
    assert abs(S.shannon_entropy_bits(counts) - 0.8112781244591328) < 1e-15  # the binary entropy of 1/4
    assert abs(S.renyi_entropy_bits(counts, 2.0) + math.log2(10 / 16)) < 1e-15
    assert S.n_for_cdf(counts, 3, 4) == 1 and S.n_for_cdf(counts, 4, 5) == 2
    assert S.shannon_entropy_bits([5]) == 0.0 and S.n_for_cdf([5]) == 1       # a single bigram: no uncertainty


@settings(max_examples=200, deadline=None)
@given(st.lists(st.integers(1, 10_000), min_size=1, max_size=200))
def test_against_scipy_and_orderings(counts):
    from scipy.stats import entropy
    h = S.shannon_entropy_bits(counts)
    assert abs(h - entropy(np.array(counts, float), base=2)) < 1e-9
    h2 = S.renyi_entropy_bits(counts, 2.0)
    hmin = -math.log2(max(counts) / sum(counts))
    assert hmin - 1e-9 <= h2 <= h + 1e-9 <= math.log2(len(counts)) + 2e-9      # H_inf <= H_2 <= H_1 <= H_0
    assert abs(S.renyi_entropy_bits(counts, 1.0 + 1e-7) - h) < 1e-4            # alpha -> 1 is Shannon's entropy
    # brute force for the coverage count: try every m
    srt = sorted(counts, reverse=True)
    want = next(m for m in range(1, len(srt) + 1) if sum(srt[:m]) * 5 >= 4 * sum(srt))
    assert S.n_for_cdf(counts, 4, 5) == want
    assert S.n_for_cdf(list(reversed(counts)), 4, 5) == want                    # order of the input does not matter


def test_synthetic_task_corpus_is_more_concentrated_than_uniform_text():
    """The property Section 3 builds on: a phrase-structured output corpus has a far smaller typical set than
    free text over the same vocabulary."""
    from workload import configs, corpus
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=400)
    task = S.corpus_stats(tokens, offsets, cfg.model.vocab)
    r = np.random.default_rng(0)
    free = S.corpus_stats(r.integers(0, cfg.model.vocab, tokens.size), offsets, cfg.model.vocab)
    assert task["bigram_entropy_bits"] < free["bigram_entropy_bits"] - 1.0
    assert task["bigrams_for_cdf"] < free["bigrams_for_cdf"]
    assert task["n_bigrams"] == free["n_bigrams"] == int(np.maximum(np.diff(offsets) - 1, 0).sum())
