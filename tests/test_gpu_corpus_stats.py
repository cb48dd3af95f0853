"""Corpus statistics on the device against the oracle: every integer bit-exact, entropies to 1e-9 relative
(both sides evaluate the same sums of c log2 c in float64; only the order of the additions and the library's
log2 differ)."""
import numpy as np
import pytest
import torch

from oracle import corpus_stats as S
from tests.gpu_harness import need_gpu
from workload import configs, corpus

INT_FIELDS = ("n_tokens", "n_bigrams", "n_unique_tokens", "n_unique_bigrams", "bigrams_for_cdf")
REAL_FIELDS = ("bigram_entropy_bits", "typical_set_size", "token_entropy_bits", "token_entropy_normalised", "token_renyi2_bits")


def both(tokens, offsets, vocab, cdf=(4, 5)):
    b = need_gpu()
    got = b.tasc_corpus_stats(torch.from_numpy(np.asarray(tokens, np.int32)).cuda(),
                              torch.from_numpy(np.asarray(offsets, np.int64)).cuda(), vocab, cdf[0], cdf[1])
    want = S.corpus_stats(tokens, offsets, vocab, cdf)
    for f in INT_FIELDS:
        assert got[f] == want[f], (f, got[f], want[f])
    for f in REAL_FIELDS:
        rel = 1e-7 if f == "typical_set_size" else 1e-9          # 2^H multiplies the entropy's absolute error by H ln 2
        assert abs(got[f] - want[f]) <= rel * max(1.0, abs(want[f])), (f, got[f], want[f])
    return got


@pytest.mark.gpu
def test_hand_worked_and_degenerate_corpora():
    both(np.array([1, 2, 1, 2, 3, 1, 2]), np.array([0, 5, 7]), 8)
    both(np.zeros(0, np.int64), np.array([0]), 16)                          # no documents
    both(np.array([4, 5, 6]), np.array([0, 1, 2, 3]), 16)                   # documents of one token: no bigram
    both(np.array([7, 7, 7, 7, 7, 7]), np.array([0, 6]), 16)                # a single bigram: entropy 0
    r = both(np.arange(64), np.array([0, 64]), 64, cdf=(1, 1))              # uniform tokens: normalised entropy 1
    assert abs(r["token_entropy_normalised"] - 1.0) < 1e-12 and r["bigrams_for_cdf"] == 63


@pytest.mark.gpu
@pytest.mark.parametrize("which,n_docs,cdf", [(0, None, (4, 5)), (0, 300, (1, 2)), (1, 20000, (4, 5)), (4, 20000, (9, 10))])
def test_benchmark_corpora(which, n_docs, cdf):
    cfg = configs.get(which)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=n_docs)
    r = both(tokens, offsets, cfg.model.vocab, cdf)
    assert r["bigrams_for_cdf"] < r["n_unique_bigrams"]


@pytest.mark.gpu
def test_counts_beyond_the_direct_bins_and_repeatability():
    """One bigram occurring 1.5 M times (count values from 2^20 on are listed, not binned) among ordinary ones; and the
    same call twice gives bit-identical results although the hash table's slot placement depends on thread timing."""
    b = need_gpu()
    r = np.random.default_rng(8)
    heavy = np.full(1_500_001, 3, np.int64)
    tail = r.integers(0, 1000, 200_000)
    tokens = np.concatenate([heavy, tail])
    offsets = np.array([0, heavy.size, tokens.size])
    first = both(tokens, offsets, 1000)
    t, o = torch.from_numpy(tokens.astype(np.int32)).cuda(), torch.from_numpy(offsets).cuda()
    assert b.tasc_corpus_stats(t, o, 1000) == b.tasc_corpus_stats(t, o, 1000) == first
    assert first["bigrams_for_cdf"] == 1


@pytest.mark.gpu
def test_rejects_bad_arguments():
    b = need_gpu()
    t = torch.tensor([1, 2, 99], dtype=torch.int32).cuda()
    o = torch.tensor([0, 3], dtype=torch.int64).cuda()
    with pytest.raises(b.TascError) as e:
        b.tasc_corpus_stats(t, o, 50)                                        # token id outside the vocabulary
    assert e.value.code == b.EINVAL
    with pytest.raises(b.TascError):
        b.tasc_corpus_stats(t, o, 100, 6, 5)                                 # coverage above 1
