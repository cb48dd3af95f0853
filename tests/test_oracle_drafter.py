"""Pins of the drafter oracle: brute-force recounts, conservation laws, hand-worked mixture
cases in exact fractions, and special cases the paper's text fixes (Section 5.2)."""
import os
from fractions import Fraction

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import drafter as D
from workload import configs, corpus

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def brute_force_entries(tokens, offsets, n_max, p_min):
    """Recount with nothing but loops and a linear-search list: [(n, ctx, next, count)] sorted."""
    found = []  # [n, ctx list, next, count]
    for d in range(len(offsets) - 1):
        doc = [int(t) for t in tokens[offsets[d]:offsets[d + 1]]]
        for n in range(1, n_max + 1):
            i = 0
            while i + n < len(doc):
                ctx, nxt = doc[i:i + n], doc[i + n]
                for e in found:
                    if e[0] == n and e[1] == ctx and e[2] == nxt:
                        e[3] += 1
                        break
                else:
                    found.append([n, ctx, nxt, 1])
                i += 1
    return sorted((n, tuple(c), x, cnt) for n, c, x, cnt in found if cnt >= p_min)


def tiny_corpus(seed, n_docs=12, vocab=6, lo=0, hi=14):
    r = np.random.default_rng(seed)
    lens = r.integers(lo, hi + 1, n_docs)
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    return r.integers(0, vocab, offsets[-1]).astype(np.int32), offsets


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("p_min", [1, 2, 3])
def test_tables_equal_brute_force(seed, p_min):
    tokens, offsets = tiny_corpus(seed)
    want = brute_force_entries(tokens, offsets, 3, p_min)
    assert D.build_corpus_ngrams(tokens, offsets, 3, p_min, 6).canonical() == want
    assert D.build_corpus_ngrams_sorted(tokens, offsets, 3, p_min, 6).canonical() == want


def test_sorted_builder_equals_dict_builder_on_config0():
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=300)
    a = D.build_corpus_ngrams(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    b = D.build_corpus_ngrams_sorted(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    assert a.canonical() == b.canonical() and a.fallback == b.fallback
    assert len(a.canonical()) > 100


def test_conservation_and_no_pruning_at_pmin_1():
    tokens, offsets = tiny_corpus(7, n_docs=40, vocab=5, hi=20)
    ng = D.build_corpus_ngrams(tokens, offsets, 4, 1, 5)
    lens = np.diff(offsets)
    for n in range(1, 5):
        total = sum(c for ctx in ng.models[n].values() for c in ctx.values())
        assert total == int(np.maximum(0, lens - n).sum())
    # pruning only removes: the p_min = 3 table is the subset with count >= 3
    ng3 = D.build_corpus_ngrams(tokens, offsets, 4, 3, 5)
    assert ng3.canonical() == [e for e in ng.canonical() if e[3] >= 3]


def test_no_ngram_crosses_a_document_boundary():
    tokens = np.array([1, 2, 3, 4], dtype=np.int32)
    one = D.build_corpus_ngrams(tokens, np.array([0, 4]), 2, 1, 8).canonical()
    two = D.build_corpus_ngrams(tokens, np.array([0, 2, 4]), 2, 1, 8).canonical()
    assert (1, (2,), 3, 1) in one and (2, (1, 2), 3, 1) in one
    assert two == [(1, (1,), 2, 1), (1, (3,), 4, 1)]


def test_fallback_is_most_frequent_token_smallest_on_ties():
    tokens = np.array([4, 2, 4, 2, 7], dtype=np.int32)
    assert D.build_corpus_ngrams(tokens, np.array([0, 5]), 1, 1, 8).fallback == 2
    assert D.most_frequent_token(np.zeros(0, np.int32), 8) == 0


def test_repeated_document_is_reproduced():
    doc = [5, 9, 2, 7, 7, 3, 1, 8, 4, 6, 0, 11]
    reps = 6
    tokens = np.array(doc * reps, dtype=np.int32)
    offsets = np.arange(reps + 1) * len(doc)
    ng = D.build_corpus_ngrams(tokens, offsets, 3, 5, 16)
    # order-3 contexts are unique inside the document, so corpus drafting alone continues it
    assert D.draft(ng, doc[:4], 6, 1, 1) == doc[4:10]
    # the context drafter alone copies from the sequence's own history
    hist = doc + doc[:5]
    assert D.draft(D.CorpusNgrams(3, 5, {1: {}, 2: {}, 3: {}}, 0), hist, 5, 0, 1) == doc[5:10]


def _parse_succ(s):
    s = s.strip()
    if s == "-":
        return None
    d = {int(a): int(b) for a, b in (kv.split(":") for kv in s.split(","))}
    return (1, d, sum(d.values()))


def golden_mixture_cases():
    for line in open(os.path.join(GOLDEN, "mixture_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lam, cc, cp, fb, want = line.split("|")
        num, den = map(int, lam.split())
        yield num, den, _parse_succ(cc), _parse_succ(cp), int(fb), int(want)


def test_hand_worked_mixture_cases():
    cases = list(golden_mixture_cases())
    assert len(cases) >= 12
    for num, den, cc, cp, fb, want in cases:
        assert D.mix_argmax(cc, cp, num, den, fb) == want, (num, den, cc, cp)


def rational_mixture_argmax(cc, cp, lam: Fraction, fallback):
    """The display equation of Section 5.2 in exact rationals."""
    use_c = cc is not None and lam != 0
    use_p = cp is not None and lam != 1
    if not use_c and not use_p:
        return fallback
    w_c, w_p = (lam, 1 - lam) if (use_c and use_p) else ((1, 0) if use_c else (0, 1))
    p = {}
    if use_c:
        for x, c in cc[1].items():
            p[x] = p.get(x, 0) + w_c * Fraction(c, cc[2])
    if use_p:
        for x, c in cp[1].items():
            p[x] = p.get(x, 0) + w_p * Fraction(c, cp[2])
    best = max(p.values())
    return min(x for x in p if p[x] == best)


succ_strategy = st.one_of(
    st.none(),
    st.dictionaries(st.integers(0, 9), st.integers(1, 40), min_size=1, max_size=6).map(
        lambda d: (1, d, sum(d.values()))))


@settings(max_examples=400, deadline=None)
@given(succ_strategy, succ_strategy, st.integers(0, 8), st.integers(0, 9))
def test_integer_mixture_equals_rational_mixture(cc, cp, num, fb):
    assert D.mix_argmax(cc, cp, num, 8, fb) == rational_mixture_argmax(cc, cp, Fraction(num, 8), fb)


def test_lambda_one_is_the_papers_p_corp_rule():
    """First match in descending order, else the most frequent token."""
    tokens, offsets = tiny_corpus(3, n_docs=30, vocab=5, hi=16)
    ng = D.build_corpus_ngrams(tokens, offsets, 3, 2, 5)
    r = np.random.default_rng(0)
    for _ in range(200):
        q = r.integers(0, 6, r.integers(1, 6)).tolist()   # token 5 never occurs: forces back-off / fallback
        want = None
        for n in (3, 2, 1):
            if n <= len(q) and tuple(q[-n:]) in ng.models[n]:
                succ = ng.models[n][tuple(q[-n:])]
                want = min(succ, key=lambda x: (-succ[x], x))
                break
        if want is None:
            want = ng.fallback
        assert D.draft(ng, q, 1, 1, 1) == [want]


def prompt_counts_by_scan(committed, query, n_max):
    """Independent formulation: match lengths measured backwards from every successor position."""
    L = len(committed)
    best_n, hits = 0, []
    for p in range(1, L):
        m = 0
        while m < n_max and m < p and m < len(query) and committed[p - 1 - m] == query[len(query) - 1 - m]:
            m += 1
        if m > best_n:
            best_n, hits = m, [p]
        elif m == best_n and m > 0:
            hits.append(p)
    if best_n == 0:
        return None
    d = {}
    for p in hits:
        d[committed[p]] = d.get(committed[p], 0) + 1
    return best_n, d, len(hits)


@settings(max_examples=300, deadline=None)
@given(st.lists(st.integers(0, 3), min_size=1, max_size=30), st.lists(st.integers(0, 3), max_size=4),
       st.integers(1, 4))
def test_p_prompt_equals_backward_scan(committed, drafts, n_max):
    query = committed + drafts
    assert D.p_prompt(committed, query, n_max) == prompt_counts_by_scan(committed, query, n_max)


def test_in_flight_drafts_extend_the_query_only():
    committed = [1, 2, 3, 1, 2]
    # suffix (1, 2) occurred once before, followed by 3; its own last occurrence has no successor yet
    assert D.p_prompt(committed, committed, 2) == (2, {3: 1}, 1)
    # after drafting 3 the query suffix is (2, 3), seen at positions 1..2, followed by 1
    assert D.p_prompt(committed, committed + [3], 2) == (2, {1: 1}, 1)
    # a draft that never occurred in the committed tokens contributes no statistics
    assert D.p_prompt(committed, committed + [9], 2) is None


def test_draft_returns_k_tokens_in_vocab():
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=400)
    ng = D.build_corpus_ngrams_sorted(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    prompts = corpus.make_prompts(cfg, 3)
    for b in range(3):
        d = D.draft(ng, prompts[b].tolist(), cfg.k)
        assert len(d) == cfg.k and all(0 <= t < cfg.model.vocab for t in d)


def test_canonical_array_layout():
    ng = D.CorpusNgrams(2, 1, {1: {(3,): {4: 2}}, 2: {(1, 2): {0: 5, 7: 1}}}, 0)
    a = ng.canonical_array()
    assert a.tolist() == [[1, 3, -1, -1, -1, -1, 4, 2], [2, 1, 2, -1, -1, -1, 0, 5], [2, 1, 2, -1, -1, -1, 7, 1]]
