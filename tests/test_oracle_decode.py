"""Pins of the decoding oracle: speculative greedy decoding must reproduce plain greedy decoding
token for token whatever the drafts are (Section 5.1: verification keeps only what the target
itself would have produced), commits between 1 and k+1 tokens per step, and the teacher-forced
modes accept exactly what they are told to."""
import numpy as np
import pytest

from oracle import decode as G
from oracle import drafter as D
from oracle.model import OracleModel
from workload import configs, corpus, weights as W
from workload.configs import ModelShape

SHAPE = ModelShape(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ff=96, vocab=40,
                   dtype="f32", init_std=0.3)


@pytest.fixture(scope="module")
def model():
    return OracleModel(SHAPE, W.make_weights(SHAPE, seed=5, gain_jitter=0.1), np.float64)


PROMPT = [3, 17, 4, 4, 29, 8, 1, 17, 4]


def test_accept_rule():
    assert G.accept([5, 6, 7], [5, 6, 7, 9]) == (3, 9)
    assert G.accept([5, 6, 7], [5, 8, 7, 9]) == (1, 8)
    assert G.accept([5, 6, 7], [1, 6, 7, 9]) == (0, 1)
    assert G.accept([], [4]) == (0, 4)


@pytest.mark.parametrize("k", [1, 3, 6])
def test_speculative_equals_plain_for_random_drafts(model, k):
    plain = G.greedy_plain(model, PROMPT, 30)
    r = np.random.default_rng(k)
    spec = G.greedy_speculative(model, None, PROMPT, 30, k,
                                draft_fn=lambda c, kk: r.integers(0, SHAPE.vocab, kk).tolist())
    assert spec.tokens == plain.tokens
    assert all(0 <= s.n_accepted <= k for s in spec.steps)


def test_all_wrong_drafts_commit_one_token_per_step(model):
    plain = G.greedy_plain(model, PROMPT, 12)
    # a draft that is never the model's next token: the true token plus one
    def wrong(c, k):
        g = len(c) - len(PROMPT)
        return [(plain.tokens[min(g + i, 11)] + 1) % SHAPE.vocab for i in range(k)]
    spec = G.greedy_speculative(model, None, PROMPT, 12, 4, draft_fn=wrong)
    assert spec.tokens == plain.tokens
    assert [s.n_accepted for s in spec.steps] == [0] * 12 and spec.n_forward == 12


def test_perfect_drafts_commit_k_plus_one_per_step(model):
    k = 4
    plain = G.greedy_plain(model, PROMPT, 40)
    def perfect(c, kk):
        g = len(c) - len(PROMPT)
        return plain.tokens[g:g + kk]
    spec = G.greedy_speculative(model, None, PROMPT, 30, k, draft_fn=perfect)
    assert spec.tokens == plain.tokens[:30]
    assert all(s.n_accepted == k for s in spec.steps) and spec.n_forward == 6


def test_ngram_drafter_on_config0_equals_plain_float32_with_gap_report():
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=500)
    ng = D.build_corpus_ngrams_sorted(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    m = OracleModel(cfg.model, W.make_weights(cfg.model, cfg.seed_weights), np.float32)
    prompt = corpus.make_prompts(cfg, 1)[0]
    plain = G.greedy_plain(m, prompt, 24)
    spec = G.greedy_speculative(m, ng, prompt, 24, cfg.k)
    # float32 rows of a multi-row forward may round differently from single-row forwards, so a
    # mismatch is only legitimate at a near-tie of the top two logits
    for i, (a, b) in enumerate(zip(spec.tokens, plain.tokens)):
        if a != b:
            gaps = [g for s in spec.steps for g in s.gap]
            assert min(gaps) < 1e-5, f"token {i} differs without a near-tie"
            break
    assert all(1 <= s.n_accepted + 1 <= cfg.k + 1 for s in spec.steps)


def test_forced_accept_length(model):
    for a in range(0, 4):
        spec = G.greedy_speculative(model, None, PROMPT, 13, 3, forced_accept=a,
                                    draft_fn=lambda c, k: [(c[-1] + 1 + i) % SHAPE.vocab for i in range(k)])
        assert all(s.n_accepted == a for s in spec.steps)
        assert spec.n_forward == -(-13 // (a + 1))


def test_forced_targets_builder():
    assert G.forced_targets_for_accept_len([5, 6, 7], 0, 10) == [6, 7, 8, 8]
    assert G.forced_targets_for_accept_len([5, 6, 7], 2, 10) == [5, 6, 8, 8]
    assert G.forced_targets_for_accept_len([5, 6, 9], 3, 10) == [5, 6, 9, 0]
    for a in range(4):
        assert G.accept([5, 6, 7], G.forced_targets_for_accept_len([5, 6, 7], a, 10))[0] == a


def test_teacher_forced_continuation_commits_the_continuation(model):
    cont = np.random.default_rng(0).integers(0, SHAPE.vocab, 40)
    # drafts that agree with the continuation for two tokens, then deviate
    def d(c, k):
        g = len(c) - len(PROMPT)
        return [int(cont[g]), int(cont[g + 1]), int((cont[g + 2] + 1) % SHAPE.vocab)]
    spec = G.greedy_speculative(model, None, PROMPT, 18, 3, continuation=cont, draft_fn=d)
    assert spec.tokens == cont[:18].tolist()
    assert all(s.n_accepted == 2 for s in spec.steps)


def test_kv_length_after_each_step(model):
    k = 3
    cache_lens = []
    r = np.random.default_rng(1)
    committed = list(PROMPT)
    cache = model.new_cache(64)
    model.prefill(committed[:-1], cache)
    for _ in range(6):
        drafts = r.integers(0, SHAPE.vocab, k).tolist()
        st = G.verify_step(model, cache, committed[-1], drafts)
        committed += st.drafts[:st.n_accepted] + [st.next_token]
        assert st.ctx_len + st.n_accepted + 1 == len(committed)
        assert cache.length == len(committed) - 1
