"""CPU oracle of the task-corpus statistics of the paper (Section 3, Eq. 1-2 and Table 1; the normalised
token entropy of Section 4.1 / Appendix "Uniform Information Density"; the order-2 Renyi entropy of Section 6.1 /
Appendix "Predicting Model Speedup").

TEST INFRASTRUCTURE ONLY: the product path never imports this package.  It shares no code with the
CUDA implementation.  Every function is the definition written out over plain dictionaries / numpy.

What the paper fixes and how the open points are read:

* Bigram distribution of the task's output corpus C_task: the empirical distribution of adjacent token
  pairs.  (The paper's table uses word bigrams "for simplicity"; here the unit is the token id, as
  everywhere on this path.)  A pair never spans two documents.
* Table 1 reports the Shannon entropy of that distribution and "the number of unique bigrams that cover
  80 % of the empirical distribution": read as the smallest m such that the m most frequent bigrams
  together hold at least 80 % of the bigram occurrences.
* Entropies are reported in bits: Table 1's values (an entropy of 14.5 next to 33.5 K bigrams for 80 %
  of the mass) only make sense in base 2.  Eq. 2's typical-set size exp(H) is then 2^H.
* Normalised token entropy = H(token distribution of the corpus) / log |V| (any base), |V| the
  vocabulary size.
* Renyi entropy of order alpha != 1 of the token distribution: H_alpha = log(sum_x p(x)^alpha) / (1 - alpha);
  the paper uses alpha = 2.
"""
from __future__ import annotations

import math
from collections import Counter

import numpy as np


def bigram_counts(tokens, offsets) -> Counter:
    """Counter {(a, b): occurrences} of adjacent pairs inside one document."""
    tokens = np.asarray(tokens)
    c = Counter()
    for d in range(len(offsets) - 1):
        doc = tokens[offsets[d]:offsets[d + 1]].tolist()
        for i in range(len(doc) - 1):
            c[(doc[i], doc[i + 1])] += 1
    return c


def token_counts(tokens) -> Counter:
    return Counter(np.asarray(tokens).tolist())


def shannon_entropy_bits(counts) -> float:
    """H = - sum p log2 p of the empirical distribution given by the (positive) counts; 0 for no data."""
    vals = [c for c in counts if c > 0]
    n = sum(vals)
    if n == 0:
        return 0.0
    return -math.fsum((c / n) * math.log2(c / n) for c in vals)


def renyi_entropy_bits(counts, alpha: float = 2.0) -> float:
    """H_alpha = log2(sum p^alpha) / (1 - alpha), alpha != 1; 0 for no data."""
    assert alpha != 1.0
    vals = [c for c in counts if c > 0]
    n = sum(vals)
    if n == 0:
        return 0.0
    return math.log2(math.fsum((c / n) ** alpha for c in vals)) / (1.0 - alpha)


def n_for_cdf(counts, num: int = 4, den: int = 5) -> int:
    """Smallest m such that the m largest counts sum to at least num/den of the total (0 for no data)."""
    vals = sorted((c for c in counts if c > 0), reverse=True)
    total = sum(vals)
    if total == 0:
        return 0
    run = 0
    for m, c in enumerate(vals, 1):
        run += c
        if run * den >= num * total:      # integers: no rounding decides the answer
            return m
    return len(vals)


def corpus_stats(tokens, offsets, vocab: int, cdf=(4, 5)) -> dict:
    """All statistics of one corpus (integers exact, entropies float64)."""
    bg = bigram_counts(tokens, offsets)
    tk = token_counts(tokens)
    h_bigram = shannon_entropy_bits(bg.values())
    h_token = shannon_entropy_bits(tk.values())
    return {
        "n_tokens": int(np.asarray(tokens).size),
        "n_bigrams": int(sum(bg.values())),
        "n_unique_tokens": len(tk),
        "n_unique_bigrams": len(bg),
        "bigrams_for_cdf": n_for_cdf(bg.values(), *cdf),
        "bigram_entropy_bits": h_bigram,
        "typical_set_size": 2.0 ** h_bigram,
        "token_entropy_bits": h_token,
        "token_entropy_normalised": h_token / math.log2(vocab) if vocab > 1 else 0.0,
        "token_renyi2_bits": renyi_entropy_bits(tk.values(), 2.0),
    }
