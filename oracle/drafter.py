"""CPU oracle of the n-gram drafter (TASC-draft, Section 5.2 of the paper).

TEST INFRASTRUCTURE ONLY: the product path never imports this package.  It shares
no code with the CUDA implementation.

What the paper fixes (Section 5.2) and how each ambiguity is read:

* The drafter is a family of n-gram models M_n, n <= n_max, built from the
  n-gram frequencies of the task's output corpus C_task.  Here n is the CONTEXT
  length: M_n maps a context of n tokens to the counts of the tokens that follow
  it.  n-grams never cross a document boundary and no padding symbols exist.
* Pruning: every (context, next) element whose count is below p_min is removed
  (absolute count threshold, every order).
* p_corp(.|c): query M_n in descending n with the last n tokens of c; the first
  order whose context still has a surviving element gives the distribution
  count(x) / T, T = sum of the surviving counts of that context.  If no order
  matches, the paper falls back to the most frequent token of the corpus.
* p_prompt is "obtained similarly, but based on the available context": the same
  construction over the sequence's own committed tokens (prompt + generated so
  far), without pruning, with its own back-off.  Tokens drafted but not yet
  verified extend the query suffix only, never the statistics.
* p_mixed(x|c) = lambda p_corp(x|c) + (1 - lambda) p_prompt(x|c)   (Section 5.2, display equation).
  The draft token is argmax_x p_mixed, smallest token id on ties, evaluated
  exactly in integers: with lambda = a/b,
      p_mixed(x) * b * T_corp * T_prompt = a * c_corp(x) * T_prompt + (b - a) * c_prompt(x) * T_corp.
* A component takes part iff its mixture weight is non-zero and it has a match at
  some order; otherwise it abstains and the other component is used alone.  The
  corpus-wide most frequent token is the draft only if both abstain.  With
  lambda = 1 this is exactly the paper's p_corp rule (first match, else the most
  frequent token); with lambda = 0 it is the pure context drafter.
  [parity unpinned by the paper: it prints no worked example of the mixture.]
"""
from __future__ import annotations

from collections import defaultdict

import numpy as np

MAX_ORDER = 5


class CorpusNgrams:
    """Pruned models M_1..M_n_max plus the fallback token.

    ``models[n]`` maps a context tuple of n token ids to a dict {next: count}.
    """

    def __init__(self, n_max: int, p_min: int, models, fallback: int):
        self.n_max, self.p_min, self.models, self.fallback = n_max, p_min, models, fallback

    def canonical(self):
        """Entries sorted by (n, context, next): list of (n, ctx tuple, next, count)."""
        out = []
        for n in range(1, self.n_max + 1):
            for ctx in sorted(self.models[n]):
                for x in sorted(self.models[n][ctx]):
                    out.append((n, ctx, x, self.models[n][ctx][x]))
        return out

    def canonical_array(self) -> np.ndarray:
        """int64[E, MAX_ORDER + 3] rows (n, ctx padded with -1, next, count) in canonical order."""
        ent = self.canonical()
        a = np.full((len(ent), MAX_ORDER + 3), -1, dtype=np.int64)
        for i, (n, ctx, x, c) in enumerate(ent):
            a[i, 0] = n
            a[i, 1:1 + n] = ctx
            a[i, MAX_ORDER + 1] = x
            a[i, MAX_ORDER + 2] = c
        return a


def most_frequent_token(tokens: np.ndarray, vocab: int) -> int:
    """Most frequent token of the corpus, smallest id on ties; 0 for an empty corpus."""
    if tokens.size == 0:
        return 0
    return int(np.argmax(np.bincount(tokens, minlength=vocab)))  # argmax returns the first maximum


def build_corpus_ngrams(tokens, offsets, n_max: int, p_min: int, vocab: int) -> CorpusNgrams:
    """Count, then prune: the definition written out with dictionaries (slow)."""
    tokens = np.asarray(tokens)
    models = {n: defaultdict(lambda: defaultdict(int)) for n in range(1, n_max + 1)}
    for d in range(len(offsets) - 1):
        doc = tokens[offsets[d]:offsets[d + 1]].tolist()
        for n in range(1, n_max + 1):
            for i in range(0, len(doc) - n):
                models[n][tuple(doc[i:i + n])][doc[i + n]] += 1
    pruned = {}
    for n in range(1, n_max + 1):
        pruned[n] = {}
        for ctx, succ in models[n].items():
            kept = {x: c for x, c in succ.items() if c >= p_min}
            if kept:
                pruned[n][ctx] = kept
    return CorpusNgrams(n_max, p_min, pruned, most_frequent_token(tokens, vocab))


def build_corpus_ngrams_sorted(tokens, offsets, n_max: int, p_min: int, vocab: int) -> CorpusNgrams:
    """Same tables for large corpora: per order, sort all (context, next) windows and count
    equal runs (the sort is a library primitive).  Pinned to ``build_corpus_ngrams`` by tests."""
    tokens = np.asarray(tokens, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    T = tokens.size
    doc_of = np.repeat(np.arange(offsets.size - 1), np.diff(offsets))
    doc_end = offsets[1:][doc_of] if T else np.zeros(0, np.int64)
    pos = np.arange(T, dtype=np.int64)
    models = {}
    for n in range(1, n_max + 1):
        start = pos[pos + n < doc_end]                    # window start: successor inside the same doc
        cols = [tokens[start + j] for j in range(n + 1)]  # ctx_0..ctx_{n-1}, next
        order = np.lexsort(cols[::-1])
        cols = [c[order] for c in cols]
        if start.size == 0:
            models[n] = {}
            continue
        new = np.zeros(start.size, dtype=bool)
        new[0] = True
        for c in cols:
            new[1:] |= c[1:] != c[:-1]
        first = np.flatnonzero(new)
        counts = np.diff(np.append(first, start.size))
        keep = counts >= p_min
        first, counts = first[keep], counts[keep]
        rows = np.stack([c[first] for c in cols], axis=1)
        m = {}
        for r, cnt in zip(rows.tolist(), counts.tolist()):
            m.setdefault(tuple(r[:n]), {})[r[n]] = cnt
        models[n] = m
    return CorpusNgrams(n_max, p_min, models, most_frequent_token(tokens, vocab))


def p_corp(ng: CorpusNgrams, query):
    """Back-off query: (n, {next: count}, total) at the longest matching order, or None."""
    for n in range(min(ng.n_max, len(query)), 0, -1):
        succ = ng.models[n].get(tuple(query[len(query) - n:]))
        if succ:
            return n, succ, sum(succ.values())
    return None


def p_prompt(committed, query, n_max: int):
    """Context n-gram model of the committed tokens, queried with the last tokens of ``query``.

    An occurrence of the n-token context at position i counts iff its successor
    committed[i + n] exists.  Returns (n, {next: count}, total) or None.
    """
    committed = list(committed)
    L = len(committed)
    for n in range(min(n_max, len(query)), 0, -1):
        suf = list(query[len(query) - n:])
        succ = defaultdict(int)
        for i in range(0, L - n):
            if committed[i:i + n] == suf:
                succ[committed[i + n]] += 1
        if succ:
            return n, dict(succ), sum(succ.values())
    return None


def mix_argmax(corp, prompt, lam_num: int, lam_den: int, fallback: int) -> int:
    """argmax_x [lambda p_corp(x) + (1 - lambda) p_prompt(x)], exact, smallest id on ties."""
    if lam_num == 0:
        corp = None          # weight lambda = 0: the corpus component takes no part
    if lam_num == lam_den:
        prompt = None        # weight 1 - lambda = 0: the context component takes no part
    if corp is None and prompt is None:
        return fallback
    if corp is None:
        _, cp, _ = prompt
        return min(cp, key=lambda x: (-cp[x], x))
    if prompt is None:
        _, cc, _ = corp
        return min(cc, key=lambda x: (-cc[x], x))
    _, cc, t_corp = corp
    _, cp, t_prompt = prompt
    best, best_score = None, -1
    for x in sorted(set(cc) | set(cp)):
        score = lam_num * cc.get(x, 0) * t_prompt + (lam_den - lam_num) * cp.get(x, 0) * t_corp
        if score > best_score:
            best, best_score = x, score
    return best


def draft(ng: CorpusNgrams, committed, k: int, lam_num: int = 3, lam_den: int = 4):
    """k draft tokens for one sequence; each draft is appended to the query suffix only."""
    query = list(committed)
    out = []
    for _ in range(k):
        x = mix_argmax(p_corp(ng, query), p_prompt(committed, query, ng.n_max), lam_num, lam_den, ng.fallback)
        out.append(int(x))
        query.append(int(x))
    return out
