"""Shared helpers of the GPU parity tests: build the device model from the seeded weights, run the
oracle, and drive the library step by step in lock-step with the oracle's committed state."""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from oracle import decode as G
from oracle import drafter as D
from oracle.model import OracleModel
from workload import corpus, weights as W


def need_gpu():
    import pytest
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2602_24174_b200 import binding  # noqa: F401  (raises if the library is missing)
    return binding


@dataclass
class Setup:
    cfg: object
    shape: object
    host_w: dict
    oracle: OracleModel
    ngrams: D.CorpusNgrams
    corpus_tokens: np.ndarray
    corpus_offsets: np.ndarray
    model: object = None
    drafter: object = None


def make_setup(cfg, *, n_docs=None, gain_jitter=0.0, build_drafter=True, oracle_ngrams=True, host_w=None,
               corpus_tokens=None) -> Setup:
    """``host_w`` / ``corpus_tokens`` = (tokens, offsets) replace the configuration's generated weights / corpus
    (cfg.model must then describe the given weights)."""
    b = need_gpu()
    shape = cfg.model
    if host_w is None:
        host_w = W.make_weights(shape, cfg.seed_weights, gain_jitter=gain_jitter)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=n_docs) if corpus_tokens is None else corpus_tokens
    ng = D.build_corpus_ngrams_sorted(tokens, offsets, cfg.n_max, cfg.p_min, shape.vocab) if oracle_ngrams else None
    s = Setup(cfg, shape, host_w, OracleModel(shape, host_w, np.float32), ng, tokens, offsets)
    dev_w = b.weights_to_device(host_w, shape.dtype)
    s.model = b.Model(shape, dev_w, max_positions=cfg.prompt_len + cfg.max_new + 2 * b.MAX_ROWS, page_size=cfg.page_size)
    if build_drafter:
        s.drafter = b.tasc_drafter_build(torch.from_numpy(tokens).cuda(), torch.from_numpy(offsets).cuda(), cfg.n_max,
                                         cfg.p_min, shape.vocab)
    return s


@dataclass
class LockstepReport:
    steps: int = 0
    rows: int = 0
    near_tie_mismatches: int = 0          # rows where GPU argmax != oracle argmax and the oracle top-2 gap < gap_tol
    hard_mismatches: list = field(default_factory=list)
    max_logit_err: float = 0.0
    draft_mismatches: int = 0
    accept_mismatches: int = 0


def lockstep(s: Setup, prompts: np.ndarray, max_new: int, k: int, *, logit_atol: float, logit_rtol: float, gap_tol: float,
             check_logits: bool = True, lam=(3, 4), oracle_kwargs=None, forced_mode=None) -> LockstepReport:
    """Run the oracle's speculative decoding per sequence, then replay every step on the GPU from the
    oracle's committed state and compare drafts (bit-exact), logits, argmax rows, accepted length and next token."""
    b = need_gpu()
    B, P = prompts.shape
    traces = []
    for i in range(B):
        kw = dict(oracle_kwargs[i]) if oracle_kwargs else {}
        traces.append(G.greedy_speculative(s.oracle, s.ngrams, prompts[i], max_new, k, lam[0], lam[1],
                                           keep_logits=check_logits, **kw))
    n_steps = min(len(t.steps) for t in traces)
    stride = P + max_new + 2 * k + 2
    tokens = torch.zeros((B, stride), dtype=torch.int32, device="cuda")
    tokens[:, :P] = torch.from_numpy(prompts).cuda()
    length = torch.full((B,), P, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(B, stride + b.MAX_ROWS)
    ws = s.model.new_workspace(B, k)
    seqs = b.make_seqs(tokens, length)
    b.tasc_prefill(s.model, kv, seqs, B, P, ws)
    rep = LockstepReport()
    committed = [list(map(int, prompts[i])) for i in range(B)]
    for step in range(n_steps):
        sts = [traces[i].steps[step] for i in range(B)]
        for i in range(B):
            assert len(committed[i]) == sts[i].ctx_len
        host_tok = np.zeros((B, stride), dtype=np.int32)
        for i in range(B):
            host_tok[i, :len(committed[i])] = committed[i]
        tokens.copy_(torch.from_numpy(host_tok))
        length.copy_(torch.tensor([len(c) for c in committed], dtype=torch.int32))
        drafts = b.tasc_draft(s.drafter, tokens, length, k, lam[0], lam[1])
        want_drafts = np.array([st.drafts for st in sts], dtype=np.int32)
        got_drafts = drafts.cpu().numpy()
        if not np.array_equal(got_drafts, want_drafts):
            rep.draft_mismatches += 1
            drafts = torch.from_numpy(want_drafts).cuda()
        forced = None
        if forced_mode is not None:
            forced = torch.tensor([st.targets for st in sts], dtype=torch.int32, device="cuda")
        n_acc, nxt, tgt, logits = b.tasc_verify_step(s.model, kv, seqs, drafts, ws, forced_targets=forced,
                                                     want_targets=True, want_logits=check_logits)
        b.tasc_poll_status(ws)
        tgt = tgt.cpu().numpy()
        n_acc = n_acc.cpu().numpy()
        nxt = nxt.cpu().numpy()
        if check_logits:
            lg = logits.cpu().numpy()
        for i in range(B):
            st = sts[i]
            row_ok = True
            for r in range(k + 1):
                rep.rows += 1
                if int(tgt[i, r]) != st.y[r]:
                    if st.gap[r] < gap_tol:
                        rep.near_tie_mismatches += 1
                    else:
                        rep.hard_mismatches.append((step, i, r, int(tgt[i, r]), st.y[r], st.gap[r]))
                    row_ok = False
            if check_logits:
                ref = st.logits
                err = np.abs(lg[i] - ref)
                rep.max_logit_err = max(rep.max_logit_err, float(err.max()))
                bad = err > logit_atol + logit_rtol * np.abs(ref)
                if bad.any():
                    rep.hard_mismatches.append(("logits", step, i, float(err.max())))
            if row_ok or forced_mode is not None:
                if int(n_acc[i]) != st.n_accepted or int(nxt[i]) != st.next_token:
                    rep.accept_mismatches += 1
            committed[i] = committed[i] + st.drafts[:st.n_accepted] + [st.next_token]
        rep.steps += 1
    return rep
