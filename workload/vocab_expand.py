"""Vocabulary expansion for the tokenizer-augmentation variant (configuration 3): input preparation only.

The paper's TASC-tok (Section 4) adds frequent task n-grams to the vocabulary as single tokens, scored by the
merge reward f_merge(t^n) = freq(t^n) * (n - 1) (Section 4.1), initialises every new embedding and LM-head row
as the mean of its constituents' rows (Section 4.2) and encodes text by greedy longest match with the added
tokens taking precedence (Appendix B).  The decoding hot path only needs the RESULT of that procedure as
input data: a larger embedding / LM-head matrix and a corpus written in the larger vocabulary.  This module
produces that input with a one-pass selection (all n-grams of the base-token corpus ranked by the merge
reward; no prefix-collision test, which needs token strings that synthetic ids do not have; no fine-tuning).
Nothing here is used by the drafter, the decoder or their oracle.
"""
from __future__ import annotations

import numpy as np

from .weights import round_to_bf16


def select_merges(tokens: np.ndarray, offsets: np.ndarray, n_merged: int, *, n_max: int = 4, vocab: int):
    """The n_merged n-grams (2 <= n <= n_max, within a document) with the largest freq * (n - 1);
    ties go to the longer, then the lexicographically smaller n-gram.  Returns a list of tuples; merge i
    becomes token id vocab + i."""
    tokens = np.asarray(tokens, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    doc_of = np.repeat(np.arange(offsets.size - 1), np.diff(offsets))
    doc_end = offsets[1:][doc_of] if tokens.size else np.zeros(0, np.int64)
    pos = np.arange(tokens.size, dtype=np.int64)
    cand = []
    for n in range(2, n_max + 1):
        start = pos[pos + n <= doc_end]
        if start.size == 0:
            continue
        cols = [tokens[start + j] for j in range(n)]
        order = np.lexsort(cols[::-1])                       # sort the windows, then count equal runs
        cols = [c[order] for c in cols]
        new = np.zeros(start.size, dtype=bool)
        new[0] = True
        for c in cols:
            new[1:] |= c[1:] != c[:-1]
        first = np.flatnonzero(new)
        cnt = np.diff(np.append(first, start.size))
        keep = np.argsort(-(cnt * (n - 1)), kind="stable")[:n_merged]
        rows = np.stack([c[first[keep]] for c in cols], axis=1)
        for g, c in zip(rows.tolist(), cnt[keep].tolist()):
            cand.append((-(c * (n - 1)), -n, tuple(g)))
    cand.sort()
    return [g for _, _, g in cand[:n_merged]]


def expand_weights(weights: dict, merges, *, bf16: bool = True) -> dict:
    """Appends one embedding (and LM-head) row per merge: the float32 mean of the constituents' rows,
    rounded to bf16 for bf16 models.  Layer weights are shared with the input dict."""
    def grow(mat):
        idx = np.zeros((len(merges), max(len(g) for g in merges)), dtype=np.int64)
        w = np.zeros(idx.shape, dtype=np.float32)
        for i, g in enumerate(merges):
            idx[i, :len(g)] = g
            w[i, :len(g)] = 1.0 / len(g)
        new = np.einsum("ij,ijd->id", w, mat[idx].astype(np.float32)).astype(np.float32)
        return np.concatenate([mat, round_to_bf16(new) if bf16 else new], axis=0)
    out = dict(weights)
    out["embed"] = grow(weights["embed"])
    out["lm_head"] = out["embed"] if weights["lm_head"] is weights["embed"] else grow(weights["lm_head"])
    return out


def retokenize(tokens: np.ndarray, offsets: np.ndarray, merges, *, vocab: int):
    """Greedy longest match, added tokens first: at every position the longest merge that starts there (and
    ends inside the document) replaces its constituents.  Returns (tokens, offsets) in the larger vocabulary."""
    table = {g: vocab + i for i, g in enumerate(merges)}
    lens = sorted({len(g) for g in merges}, reverse=True)
    tokens = np.asarray(tokens)
    out, offs = [], [0]
    for d in range(len(offsets) - 1):
        doc = tokens[offsets[d]:offsets[d + 1]].tolist()
        i, n = 0, len(doc)
        while i < n:
            for L in lens:
                if i + L <= n:
                    t = table.get(tuple(doc[i:i + L]))
                    if t is not None:
                        out.append(t)
                        i += L
                        break
            else:
                out.append(doc[i])
                i += 1
        offs.append(len(out))
    return np.asarray(out, dtype=np.int32), np.asarray(offs, dtype=np.int64)


def expand_back(tokens, merges, *, vocab: int) -> list:
    """Inverse of retokenize for one token sequence (merged ids -> their constituents)."""
    out = []
    for t in np.asarray(tokens).tolist():
        out.extend(merges[t - vocab] if t >= vocab else (t,))
    return out
