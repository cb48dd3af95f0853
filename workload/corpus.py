"""Synthetic task corpus, prompts and held-out continuations.

Stands in for the paper's task datasets (low-variability outputs): an output
document is a concatenation of phrases drawn by Zipf rank from a fixed phrase
pool, with uniform random tokens inserted between tokens at a fixed rate.
Data generation only; no drafter or model arithmetic lives here.
"""
from __future__ import annotations

import numpy as np

from . import rng
from .configs import CorpusRecipe, RunConfig

# stream ids of the counter-based generator
_S_PLEN, _S_PTOK = 1, 2
_S_DLEN, _S_PHRASE, _S_INS, _S_RTOK = 3, 4, 5, 6
_S_PR_KIND, _S_PR_PICK, _S_PR_LEN, _S_PR_TOK = 7, 8, 9, 10
_S_CT_KIND, _S_CT_PICK, _S_CT_INS, _S_CT_TOK = 11, 12, 13, 14


class PhrasePool:
    """``pool_size`` phrases of phrase_lo..phrase_hi uniform random token ids."""

    def __init__(self, recipe: CorpusRecipe, vocab: int, seed: int):
        n = recipe.pool_size
        self.lens = rng.randint(seed, _S_PLEN, np.arange(n), recipe.phrase_lo, recipe.phrase_hi + 1)
        self.offs = np.zeros(n + 1, dtype=np.int64)
        np.cumsum(self.lens, out=self.offs[1:])
        self.tokens = rng.randint(seed, _S_PTOK, np.arange(self.offs[-1]), 0, vocab).astype(np.int32)
        # Zipf(s) over ranks 1..n: P(rank r) proportional to r^-s
        w = np.arange(1, n + 1, dtype=np.float64) ** (-recipe.zipf_s)
        self.cdf = np.cumsum(w / w.sum())
        self.cdf[-1] = 1.0

    def phrase(self, i: int) -> np.ndarray:
        return self.tokens[self.offs[i]:self.offs[i + 1]]

    def zipf_rank(self, u: np.ndarray) -> np.ndarray:
        return np.minimum(np.searchsorted(self.cdf, u, side="right"), self.lens.size - 1)


def _gen_docs(pool: PhrasePool, recipe: CorpusRecipe, vocab: int, seed: int, d0: int, d1: int):
    """Documents d0..d1-1 as (tokens, lengths)."""
    D = d1 - d0
    docs = np.arange(d0, d1, dtype=np.int64)
    lens = rng.randint(seed, _S_DLEN, docs, recipe.len_lo, recipe.len_hi + 1)
    hi = recipe.len_hi
    max_ph = -(-hi // recipe.phrase_lo)
    # per output position: inserted random token or next phrase-stream token
    pos = docs[:, None] * hi + np.arange(hi, dtype=np.int64)[None, :]
    ins = rng.uniform(seed, _S_INS, pos) < recipe.insert_rate
    rtok = rng.randint(seed, _S_RTOK, pos, 0, vocab).astype(np.int32)
    valid = np.arange(hi)[None, :] < lens[:, None]
    # phrase stream of each document
    pidx = docs[:, None] * max_ph + np.arange(max_ph, dtype=np.int64)[None, :]
    ranks = pool.zipf_rank(rng.uniform(seed, _S_PHRASE, pidx))            # [D, max_ph]
    pl = pool.lens[ranks]
    flat_rank = ranks.ravel()
    flat_len = pl.ravel()
    starts = np.zeros(flat_len.size + 1, dtype=np.int64)
    np.cumsum(flat_len, out=starts[1:])
    rep_phrase = np.repeat(np.arange(flat_len.size, dtype=np.int64), flat_len)
    within = np.arange(starts[-1], dtype=np.int64) - starts[rep_phrase]
    stream = pool.tokens[pool.offs[flat_rank[rep_phrase]] + within]        # all documents' streams
    doc_stream_start = starts[np.arange(D, dtype=np.int64) * max_ph]
    # stream index consumed at output position j = number of non-inserted positions before j
    non_ins_before = np.cumsum(~ins, axis=1) - (~ins)
    src = doc_stream_start[:, None] + non_ins_before
    out = np.where(ins, rtok, stream[np.minimum(src, stream.size - 1)])
    return out[valid].astype(np.int32), lens


def make_corpus(cfg: RunConfig, *, n_docs: int | None = None, chunk: int = 20000):
    """(tokens int32[T], offsets int64[D+1]) for the configuration's task corpus."""
    recipe = cfg.corpus
    D = recipe.n_docs if n_docs is None else n_docs
    pool = PhrasePool(recipe, base_vocab(cfg), cfg.seed_pool)
    toks, lens = [], []
    for d0 in range(0, D, chunk):
        t, l = _gen_docs(pool, recipe, base_vocab(cfg), cfg.seed_corpus, d0, min(D, d0 + chunk))
        toks.append(t)
        lens.append(l)
    tokens = np.concatenate(toks) if toks else np.zeros(0, np.int32)
    offsets = np.zeros(D + 1, dtype=np.int64)
    if lens:
        np.cumsum(np.concatenate(lens), out=offsets[1:])
    return tokens, offsets


def base_vocab(cfg: RunConfig) -> int:
    """Vocabulary the corpus generator draws from (merged tokens are added on top of it)."""
    return cfg.model.vocab


def make_prompts(cfg: RunConfig, batch: int, *, prompt_len: int | None = None) -> np.ndarray:
    """int32[batch, prompt_len]: about half uniform random tokens, half pool phrases drawn uniformly."""
    P = cfg.prompt_len if prompt_len is None else prompt_len
    V = base_vocab(cfg)
    pool = PhrasePool(cfg.corpus, V, cfg.seed_pool)
    out = np.zeros((batch, P), dtype=np.int32)
    for b in range(batch):
        n, seg = 0, 0
        while n < P:
            c = b * 4 * P + seg
            if rng.uniform(cfg.seed_prompts, _S_PR_KIND, [c])[0] < 0.5:
                piece = pool.phrase(int(rng.randint(cfg.seed_prompts, _S_PR_PICK, [c], 0, pool.lens.size)[0]))
            else:
                r = int(rng.randint(cfg.seed_prompts, _S_PR_LEN, [c], cfg.corpus.phrase_lo, cfg.corpus.phrase_hi + 1)[0])
                piece = rng.randint(cfg.seed_prompts, _S_PR_TOK, np.arange(c * 8, c * 8 + r), 0, V).astype(np.int32)
            m = min(piece.size, P - n)
            out[b, n:n + m] = piece[:m]
            n += m
            seg += 1
    return out


def make_continuations(cfg: RunConfig, prompts: np.ndarray, length: int, *, reuse_prob: float = 0.3) -> np.ndarray:
    """int32[batch, length] held-out continuations for the teacher-forced mode.

    Built like a corpus document (Zipf phrases + random insertions), except that
    with probability ``reuse_prob`` a phrase is an 3..8-token span copied from the
    sequence's own prompt, so a context-based drafter has something to find.
    """
    V = base_vocab(cfg)
    rc = cfg.corpus
    pool = PhrasePool(rc, V, cfg.seed_pool)
    B, P = prompts.shape
    out = np.zeros((B, length), dtype=np.int32)
    for b in range(B):
        n, seg = 0, 0
        while n < length:
            c = b * 4 * length + seg
            u = rng.uniform(cfg.seed_cont, _S_CT_KIND, [c])[0]
            if u < reuse_prob and P > rc.phrase_hi:
                L = int(rng.randint(cfg.seed_cont, _S_PR_LEN, [c], rc.phrase_lo, rc.phrase_hi + 1)[0])
                s = int(rng.randint(cfg.seed_cont, _S_CT_PICK, [c], 0, P - L + 1)[0])
                piece = prompts[b, s:s + L]
            else:
                r = int(pool.zipf_rank(rng.uniform(cfg.seed_cont, _S_CT_PICK, [c]))[0])
                piece = pool.phrase(r)
            for t in piece:
                if n >= length:
                    break
                cc = b * 16 * length + 2 * n
                if rng.uniform(cfg.seed_cont, _S_CT_INS, [cc])[0] < rc.insert_rate:
                    out[b, n] = int(rng.randint(cfg.seed_cont, _S_CT_TOK, [cc], 0, V)[0])
                    n += 1
                    if n >= length:
                        break
                out[b, n] = t
                n += 1
            seg += 1
    return out
