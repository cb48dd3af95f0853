"""CPU oracle of the tokenizer-enrichment method (TASC-tok): Algorithm 1 and the merge reward of Section 4.1, the
mean-of-constituents initialisation of the new embedding / LM-head rows (Section 4.2), and the encoding of text with
the enriched vocabulary (Appendix "Byte-Pair Encoding": the added tokens are queried before the base tokenizer).

TEST INFRASTRUCTURE ONLY: the product path never imports this package.  It shares no code with the CUDA path.

The steps follow Algorithm 1 in its order and notation: starting from V_0 = the base vocabulary, every iteration
collects the token n-grams (2 <= n <= n_max) of the task corpus as it is tokenised with the current vocabulary V_i,
scores each with f_merge(t^n) = freq(t^n) * (n - 1), takes the argmax t*, adds it to the vocabulary as one new token
and goes on, until the budget of M tokens is reached.

Readings where the paper is silent or needs token strings that synthetic ids do not have:
* freq(t^n) counts every window of the corpus (overlapping occurrences included); windows never span two documents.
* Prefix Collision Score: needs the tokens' strings; with bare ids it cannot be evaluated, so every candidate passes
  (threshold alpha = infinity).  `usedNgrams` then never excludes anything: a merged n-gram no longer occurs.
* "collectNgrams(V_i, ...)": BPE-inspired, so adding t* re-tokenises the corpus: its occurrences are replaced by the
  new token, left to right, non-overlapping, inside each document; later iterations see the new token as a symbol
  (n-grams of merged tokens can be merged again).
* argmax ties: the longer n-gram, then the one whose first occurrence comes first (document order, then position).
* The loop also ends when no n-gram is left (every document shorter than two tokens).
* New rows (Section 4.2): e_new = (1/n) sum_j e_{t_j} over the n constituents as they were at merge time (a constituent
  may itself be an added token, whose row is then the one computed for it), summed left to right in float32 and
  divided by n; rounded to bf16 (nearest even) for a bf16 model.  The same for the LM head.
* Encoding new text: the added tokens are matched first and greedily -- at every position the added token with the
  longest expansion (into base tokens) that matches the upcoming base tokens and ends inside the document replaces
  them; where none matches the base token stays.
"""
from __future__ import annotations

import numpy as np


def _split_docs(tokens, offsets):
    tokens = np.asarray(tokens)
    return [tokens[offsets[d]:offsets[d + 1]].tolist() for d in range(len(offsets) - 1)]


def collect_ngrams(docs, n_max: int):
    """({n-gram: freq}, {n-gram: (document, position) of its first occurrence}) over the current tokenisation."""
    freq, first = {}, {}
    for d, doc in enumerate(docs):
        for i in range(len(doc)):
            for n in range(2, n_max + 1):
                if i + n > len(doc):
                    break
                g = tuple(doc[i:i + n])
                freq[g] = freq.get(g, 0) + 1
                if g not in first:
                    first[g] = (d, i)
    return freq, first


def merge_reward(freq: int, n: int) -> int:
    """f_merge(t^n) = freq(t^n) * (n - 1): tokens saved if every counted occurrence became one token."""
    return freq * (n - 1)


def replace_ngram(doc, g, new_id: int):
    """Left to right, non-overlapping."""
    out, i, n = [], 0, len(g)
    g = list(g)
    while i < len(doc):
        if doc[i:i + n] == g:
            out.append(new_id)
            i += n
        else:
            out.append(doc[i])
            i += 1
    return out


def enrich(tokens, offsets, base_vocab: int, budget: int, n_max: int):
    """Algorithm 1.  Returns (merges, docs): merges[i] = the constituents (ids of the vocabulary at that time) of
    added token base_vocab + i; docs = the corpus tokenised with the enriched vocabulary."""
    docs = _split_docs(tokens, offsets)
    merges = []
    while len(merges) < budget:
        freq, first = collect_ngrams(docs, n_max)
        if not freq:
            break
        best = max(freq, key=lambda g: (merge_reward(freq[g], len(g)), len(g), (-first[g][0], -first[g][1])))
        new_id = base_vocab + len(merges)
        merges.append(best)
        docs = [replace_ngram(doc, best, new_id) for doc in docs]
    return merges, docs


def expansion(merges, base_vocab: int, token: int):
    """Base-token sequence an id stands for."""
    if token < base_vocab:
        return [token]
    out = []
    for c in merges[token - base_vocab]:
        out.extend(expansion(merges, base_vocab, c))
    return out


def new_rows(matrix, merges, base_vocab: int, bf16: bool):
    """Rows of the added tokens for an embedding or LM-head matrix [base_vocab, d] (float32 values)."""
    rows = [np.asarray(r, dtype=np.float32) for r in matrix]
    out = []
    for g in merges:
        acc = np.zeros(rows[0].shape, dtype=np.float32)
        for c in g:
            acc = (acc + rows[c]).astype(np.float32)
        r = (acc / np.float32(len(g))).astype(np.float32)
        if bf16:
            bits = r.view(np.uint32)
            r = ((bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)).view(np.float32)
        rows.append(r)
        out.append(r)
    return np.stack(out) if out else np.zeros((0, np.asarray(matrix).shape[1]), np.float32)


def encode(doc, merges, base_vocab: int):
    """Greedy longest match of the added tokens' expansions, added tokens before base tokens."""
    table = {}
    for i in range(len(merges)):
        e = tuple(expansion(merges, base_vocab, base_vocab + i))
        table.setdefault(e, base_vocab + i)            # two added tokens with one expansion: the earlier one
    lens = sorted({len(e) for e in table}, reverse=True)
    doc = list(doc)
    out, i = [], 0
    while i < len(doc):
        for L in lens:
            t = table.get(tuple(doc[i:i + L])) if i + L <= len(doc) else None
            if t is not None:
                out.append(t)
                i += L
                break
        else:
            out.append(doc[i])
            i += 1
    return out
