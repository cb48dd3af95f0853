"""Shared helpers of the GPU parity tests: build the device model from the seeded weights, run the
oracle, and drive the library step by step in lock-step with the oracle's committed state."""
from __future__ import annotations

import json
import os
from dataclasses import asdict, dataclass, field

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


CANARY = 0x5A


class Guarded:
    """A device buffer with a band of canary bytes before and after it: the library is handed the inside; check()
    fails if a kernel wrote outside what it was given (the substitute for a memory checker on these machines)."""
    BAND = 4096

    def __init__(self, shape, dtype, align=256):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % align
        self.raw = torch.full((self.BAND + n + pad + self.BAND,), CANARY, dtype=torch.uint8, device="cuda")
        assert self.raw.data_ptr() % align == 0
        self.n = n
        self.inner = self.raw[self.BAND:self.BAND + n].view(dtype).view(*shape)

    def check(self, what):
        before, after = self.raw[:self.BAND], self.raw[self.BAND + self.n:]
        assert bool((before == CANARY).all()) and bool((after == CANARY).all()), f"write outside {what}"


@dataclass
class LockstepReport:
    steps: int = 0
    rows: int = 0
    near_tie_mismatches: int = 0          # rows where GPU argmax != oracle argmax and the oracle top-2 gap < gap_tol
    hard_mismatches: list = field(default_factory=list)
    max_logit_err: float = 0.0
    max_err_over_or_bound: float = 0.0    # largest err / max(atol, rtol |ref|): below 1 the tighter "either bound" reading holds too
    draft_mismatches: int = 0
    accept_mismatches: int = 0


REPORT_PATH = os.environ.get("TASC_PARITY_REPORT",
                             os.path.join(os.path.dirname(os.path.abspath(__file__)), "_out", "parity_counts.jsonl"))


def record_parity(name: str, rep: LockstepReport, **extra):
    """Appends the counts of one lock-step comparison (rows compared, near-tie mismatches, largest logit
    error) as a JSON line to REPORT_PATH, so that a run leaves them behind as an artefact."""
    try:
        os.makedirs(os.path.dirname(REPORT_PATH), exist_ok=True)
        d = asdict(rep)
        d["hard_mismatches"] = len(rep.hard_mismatches)
        with open(REPORT_PATH, "a") as f:
            f.write(json.dumps({"test": name, **d, **extra}) + "\n")
    except OSError:
        pass


def lockstep(s: Setup, prompts: np.ndarray, max_new: int, k: int, *, logit_atol: float, logit_rtol: float, gap_tol: float,
             check_logits: bool = True, lam=(3, 4), oracle_kwargs=None, forced_mode=None, oracle_rows=None) -> LockstepReport:
    """Run the oracle's speculative decoding per sequence, then replay every step on the GPU from the
    oracle's committed state and compare drafts (bit-exact), logits, argmax rows, accepted length and next token.

    ``oracle_rows``: the sequences of the batch the oracle runs and the comparison covers (all by default); the
    other sequences of the batch decode on from whatever the device committed for them."""
    b = need_gpu()
    B, P = prompts.shape
    checked = list(range(B)) if oracle_rows is None else list(oracle_rows)
    traces = {}
    for i in checked:
        kw = dict(oracle_kwargs[i]) if oracle_kwargs else {}
        traces[i] = G.greedy_speculative(s.oracle, s.ngrams, prompts[i], max_new, k, lam[0], lam[1],
                                         keep_logits=check_logits, **kw)
    n_steps = min(len(traces[i].steps) for i in checked)
    stride = P + max(max_new, n_steps * (k + 1)) + 2 * k + 2
    tokens = torch.zeros((B, stride), dtype=torch.int32, device="cuda")
    tokens[:, :P] = torch.from_numpy(prompts).cuda()
    length = torch.full((B,), P, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(B, stride + b.MAX_ROWS)
    # workspace and every output of the step sit between canary bands, checked after every call
    g_ws = Guarded((s.model.workspace_bytes(B, k),), torch.uint8)
    g_ws.inner.zero_()
    ws = g_ws.inner
    g_acc, g_nxt = Guarded((B,), torch.int32), Guarded((B,), torch.int32)
    g_tgt = Guarded((B, k + 1), torch.int32)
    g_lg = Guarded((B, k + 1, s.shape.vocab), torch.float32) if check_logits else None
    guards = [(g_ws, "the workspace"), (g_acc, "n_accepted"), (g_nxt, "next_token"), (g_tgt, "target_tokens")]
    if g_lg is not None:
        guards.append((g_lg, "logits"))
    seqs = b.make_seqs(tokens, length)
    b.tasc_prefill(s.model, kv, seqs, B, P, ws)
    g_ws.check("the workspace (prefill)")
    rep = LockstepReport()
    committed = {i: list(map(int, prompts[i])) for i in checked}
    sel = torch.tensor(checked, dtype=torch.long, device="cuda")
    for step in range(n_steps):
        sts = {i: traces[i].steps[step] for i in checked}
        for i in checked:
            assert len(committed[i]) == sts[i].ctx_len
        host_tok = np.zeros((len(checked), stride), dtype=np.int32)
        for j, i in enumerate(checked):
            host_tok[j, :len(committed[i])] = committed[i]
        tokens[sel] = torch.from_numpy(host_tok).cuda()
        length[sel] = torch.tensor([len(committed[i]) for i in checked], dtype=torch.int32, device="cuda")
        drafts = b.tasc_draft(s.drafter, tokens, length, k, lam[0], lam[1])
        want_drafts = np.array([sts[i].drafts for i in checked], dtype=np.int32)
        got_drafts = drafts[sel].cpu().numpy()
        if not np.array_equal(got_drafts, want_drafts):
            rep.draft_mismatches += 1
            drafts[sel] = torch.from_numpy(want_drafts).cuda()
        forced = None
        if forced_mode is not None:
            assert len(checked) == B
            forced = torch.tensor([sts[i].targets for i in checked], dtype=torch.int32, device="cuda")
        n_acc, nxt, tgt, logits = b.tasc_verify_step(s.model, kv, seqs, drafts, ws, forced_targets=forced,
                                                     out=(g_acc.inner, g_nxt.inner, g_tgt.inner, g_lg.inner if g_lg else None))
        b.tasc_poll_status(ws)
        for g, what in guards:
            g.check(what)
        tgt = tgt.cpu().numpy()
        n_acc = n_acc.cpu().numpy()
        nxt = nxt.cpu().numpy()
        if check_logits:
            lg = logits[sel].cpu().numpy()
        for j, i in enumerate(checked):
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
                err = np.abs(lg[j] - ref)
                rep.max_logit_err = max(rep.max_logit_err, float(err.max()))
                rep.max_err_over_or_bound = max(rep.max_err_over_or_bound,
                                                float((err / np.maximum(logit_atol, logit_rtol * np.abs(ref))).max()))
                bad = err > np.maximum(logit_atol, logit_rtol * np.abs(ref))      # within the absolute OR the relative bound
                if bad.any():
                    rep.hard_mismatches.append(("logits", step, i, float(err.max())))
            if row_ok or forced_mode is not None:
                if int(n_acc[i]) != st.n_accepted or int(nxt[i]) != st.next_token:
                    rep.accept_mismatches += 1
            committed[i] = committed[i] + st.drafts[:st.n_accepted] + [st.next_token]
        rep.steps += 1
    return rep
