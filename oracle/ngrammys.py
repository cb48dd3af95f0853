"""CPU oracle of the comparison drafter of Section 6.2 (the "N-Grammys" bigram): a bigram model obtained from the
target model itself by taking, for every token of the vocabulary, the most probable next token under the model's
conditional distribution; and its mixing with the context n-gram drafter p_prompt.

TEST INFRASTRUCTURE ONLY: the product path never imports this package.  It shares no code with the CUDA path.

Readings (the paper describes the baseline in one sentence):
* "the conditional distribution for each element of the vocabulary": the model is run on the single token t as its
  whole context (position 0, empty cache); table[t] = argmax of those logits, smallest id on ties.
* The bigram is a point mass on table[t].  "Mixed" with the context drafter it enters the mixture of Section 5.2 in the
  place of p_corp:  p = lambda * [x = table[t]] + (1 - lambda) * p_prompt(x | c), with the same abstention rule (a
  component without a match, or with zero weight, takes no part).  For lambda >= 1/2 the point mass always wins, so the
  mixed baseline is meaningful for small lambda: the context drafter where it has a match, the bigram elsewhere.
  [parity unpinned by the paper: it gives neither the mixing rule nor its weight for this baseline.]
"""
from __future__ import annotations

import numpy as np

from .drafter import CorpusNgrams
from .model import OracleModel, argmax_and_gap


def bigram_table(model: OracleModel, tokens=None):
    """(table, gap): table[t] = argmax_x p_model(x | t) for every token t (or the given ones), and the top-2 logit gap
    of each row.  One forward pass per token, each on an empty cache."""
    V = model.s.vocab
    tokens = range(V) if tokens is None else tokens
    table, gaps = [], []
    for t in tokens:
        logits = model.forward([int(t)], model.new_cache(1))
        y, gap = argmax_and_gap(logits)
        table.append(int(y[0]))
        gaps.append(float(gap[0]))
    return np.array(table, dtype=np.int64), np.array(gaps)


def as_ngram_model(table) -> CorpusNgrams:
    """The bigram as an order-1 model with one successor of count 1 per context, so that oracle.drafter.draft mixes it
    with the context drafter exactly as it mixes p_corp.  The last-resort token (used only when the bigram has weight
    zero and the context drafter has no match) is token 0."""
    return CorpusNgrams(1, 1, {1: {(t,): {int(x): 1} for t, x in enumerate(np.asarray(table).tolist())}}, 0)
