"""CPU oracle of greedy decoding and of draft-then-verify speculative decoding
(Section 5.1 of the paper: draft gamma tokens, verify them with one forward pass
of the target, keep an accepted prefix; here gamma is called k and verification is
greedy, i.e. beam size 1 as in the paper's experiments).

TEST INFRASTRUCTURE ONLY: the product path never imports this package.

One speculative step for a sequence with committed tokens c_0..c_{L-1} whose KV
cache holds positions 0..L-2:
  inputs  [c_{L-1}, d_1, ..., d_k] at positions L-1 .. L-1+k
  y_i   = argmax of the logits of row i (smallest id on ties), i = 0..k
  a     = largest j with d_1..d_j == y_0..y_{j-1}            (0 <= a <= k)
  commit  d_1..d_a and y_a  ->  L grows by a+1 (between 1 and k+1 tokens)
  KV positions beyond the new L-2 are dead (rolled back).
With forced targets (teacher-forced mode) y is replaced by the given tokens in the
accept rule and in what is committed; the forward still runs.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import drafter as D
from .model import OracleModel, argmax_and_gap


@dataclass
class StepTrace:
    ctx_len: int                 # committed length L before the step
    last_token: int
    drafts: list
    y: list                      # model argmax of rows 0..k
    gap: list                    # top-1 minus top-2 logit of rows 0..k
    targets: list                # y, or the forced targets
    n_accepted: int
    next_token: int
    logits: np.ndarray | None = None


@dataclass
class GenResult:
    tokens: list                 # generated tokens (max_new of them)
    steps: list = field(default_factory=list)
    n_forward: int = 0


def accept(drafts, targets):
    """(a, next): longest prefix of drafts equal to the targets, and the token committed after it."""
    a = 0
    while a < len(drafts) and drafts[a] == targets[a]:
        a += 1
    return a, int(targets[a])


def greedy_plain(model: OracleModel, prompt, max_new: int, capacity: int | None = None) -> GenResult:
    """One token per forward pass."""
    prompt = list(map(int, prompt))
    cache = model.new_cache(capacity or len(prompt) + max_new + 1)
    model.prefill(prompt[:-1], cache)
    last = prompt[-1]
    out = GenResult([])
    for _ in range(max_new):
        logits = model.forward([last], cache)
        y, _ = argmax_and_gap(logits)
        last = int(y[0])
        out.tokens.append(last)
        out.n_forward += 1
    return out


def verify_step(model: OracleModel, cache, last_token: int, drafts, forced_targets=None, keep_logits=False):
    """One verify forward + accept + KV rollback.  Returns a StepTrace (ctx_len filled by caller)."""
    L1 = cache.length                                  # = L - 1
    logits = model.forward([last_token] + list(drafts), cache)
    y, gap = argmax_and_gap(logits)
    targets = list(map(int, y)) if forced_targets is None else list(map(int, forced_targets))
    a, nxt = accept(list(drafts), targets)
    cache.truncate(L1 + a + 1)
    return StepTrace(L1 + 1, int(last_token), list(map(int, drafts)), list(map(int, y)), list(map(float, gap)),
                     targets, a, nxt, logits if keep_logits else None)


def forced_targets_for_accept_len(drafts, a: int, vocab: int):
    """Targets under which exactly ``a`` drafts are accepted: rows < a repeat the drafts,
    row a (and later rows) is the draft id plus one modulo the vocabulary; row k, which has no
    draft to compare with, is the last draft plus one."""
    k = len(drafts)
    t = []
    for i in range(k + 1):
        if i < a:
            t.append(int(drafts[i]))
        else:
            t.append(int((drafts[min(i, k - 1)] + 1) % vocab))
    return t


def greedy_speculative(model: OracleModel, ngrams: D.CorpusNgrams, prompt, max_new: int, k: int,
                       lam_num: int = 3, lam_den: int = 4, *, draft_fn=None, continuation=None,
                       forced_accept: int | None = None, keep_logits: bool = False,
                       capacity: int | None = None) -> GenResult:
    """Speculative greedy decoding of one sequence.

    ``draft_fn(committed, k)`` overrides the n-gram drafter (tests use arbitrary drafts).
    ``continuation`` (teacher-forced): targets of a step are continuation[g : g+k+1], g = tokens generated so far.
    ``forced_accept`` (teacher-forced): every step accepts exactly that many drafts.
    """
    committed = list(map(int, prompt))
    P = len(committed)
    cache = model.new_cache(capacity or P + max_new + k + 1)
    model.prefill(committed[:-1], cache)
    out = GenResult([])
    while len(committed) - P < max_new:
        drafts = draft_fn(committed, k) if draft_fn else D.draft(ngrams, committed, k, lam_num, lam_den)
        forced = None
        g = len(committed) - P
        if continuation is not None:
            forced = [int(t) for t in continuation[g:g + k + 1]]
        elif forced_accept is not None:
            forced = forced_targets_for_accept_len(drafts, forced_accept, model.s.vocab)
        st = verify_step(model, cache, committed[-1], drafts, forced, keep_logits)
        committed.extend(st.drafts[:st.n_accepted])
        committed.append(st.next_token)
        out.steps.append(st)
        out.n_forward += 1
    out.tokens = committed[P:P + max_new]
    return out
