"""On-device drafter against the oracle: exported tables and fallback token bit-exact, drafts bit-exact."""
import numpy as np
import pytest
import torch

from oracle import drafter as D
from tests.gpu_harness import need_gpu
from workload import configs, corpus


def build_both(tokens, offsets, n_max, p_min, vocab):
    b = need_gpu()
    dr = b.tasc_drafter_build(torch.from_numpy(np.asarray(tokens, np.int32)).cuda(),
                              torch.from_numpy(np.asarray(offsets, np.int64)).cuda(), n_max, p_min, vocab)
    ng = D.build_corpus_ngrams_sorted(tokens, offsets, n_max, p_min, vocab)
    return b, dr, ng


def assert_tables_equal(dr, ng):
    got, fb = dr.export()
    want = ng.canonical_array()
    assert fb == ng.fallback
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.array_equal(got, want)


def draft_contexts(cfg, tokens, offsets, n_ctx, max_len, seed):
    """Contexts that exercise every branch: corpus document prefixes, prompts, and prompts followed by document pieces."""
    r = np.random.default_rng(seed)
    prompts = corpus.make_prompts(cfg, max(2, n_ctx // 3), prompt_len=min(cfg.prompt_len, max_len - 8))
    out = []
    for i in range(n_ctx):
        d = int(r.integers(0, len(offsets) - 1))
        doc = tokens[offsets[d]:offsets[d + 1]]
        cut = int(r.integers(1, len(doc) + 1))
        kind = i % 3
        if kind == 0:
            c = doc[:cut]
        elif kind == 1:
            c = prompts[i % len(prompts)]
        else:
            c = np.concatenate([prompts[i % len(prompts)][:int(r.integers(1, prompts.shape[1]))], doc[:cut]])
        out.append(np.asarray(c[-max_len:], dtype=np.int32))
    return out


def assert_drafts_equal(b, dr, ng, contexts, k, lams, stride):
    B = len(contexts)
    tok = np.zeros((B, stride), dtype=np.int32)
    ln = np.zeros(B, dtype=np.int32)
    for i, c in enumerate(contexts):
        tok[i, :len(c)] = c
        ln[i] = len(c)
    t_dev, l_dev = torch.from_numpy(tok).cuda(), torch.from_numpy(ln).cuda()
    for num, den in lams:
        got = b.tasc_draft(dr, t_dev, l_dev, k, num, den).cpu().numpy()
        want = np.array([D.draft(ng, c.tolist(), k, num, den) for c in contexts], dtype=np.int32)
        assert np.array_equal(got, want), (num, den, np.argwhere(got != want)[:5])


@pytest.mark.gpu
def test_config0_tables_and_drafts():
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg)
    b, dr, ng = build_both(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    assert_tables_equal(dr, ng)
    ctxs = draft_contexts(cfg, tokens, offsets, 96, 100, seed=1)
    assert_drafts_equal(b, dr, ng, ctxs, cfg.k, [(3, 4), (1, 2), (1, 1), (0, 1), (255, 256)], stride=128)


@pytest.mark.gpu
@pytest.mark.parametrize("p_min", [1, 5])
def test_config1_tables_and_drafts(p_min):
    cfg = configs.get(1)
    tokens, offsets = corpus.make_corpus(cfg)
    b, dr, ng = build_both(tokens, offsets, cfg.n_max, p_min, cfg.model.vocab)
    assert_tables_equal(dr, ng)
    if p_min == 5:
        ctxs = draft_contexts(cfg, tokens, offsets, 48, 400, seed=2)
        assert_drafts_equal(b, dr, ng, ctxs, cfg.k, [(3, 4), (1, 1), (0, 1)], stride=416)


@pytest.mark.gpu
def test_max_order_and_wide_ids():
    """n_max = 5 with token ids that need all 20 bits, documents shorter than the order, empty documents."""
    r = np.random.default_rng(5)
    vocab = 1 << 20
    base = r.integers(vocab - 50, vocab, 40)
    docs = [base[r.integers(0, 40, r.integers(0, 30))] for _ in range(300)]
    docs += [np.zeros(0, np.int64), base[:1], base[:3]]
    tokens = np.concatenate(docs).astype(np.int32)
    offsets = np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int64)
    b, dr, ng = build_both(tokens, offsets, 5, 2, vocab)
    assert_tables_equal(dr, ng)
    assert len(ng.canonical()) > 50
    ctxs = [base[r.integers(0, 40, n)].astype(np.int32) for n in (1, 2, 3, 4, 5, 6, 9, 40)]
    assert_drafts_equal(b, dr, ng, ctxs, 6, [(3, 4), (1, 1)], stride=64)


@pytest.mark.gpu
def test_empty_and_degenerate_corpora():
    b, dr, ng = build_both(np.zeros(0, np.int32), np.array([0], np.int64), 3, 1, 16)
    assert_tables_equal(dr, ng)                                     # no documents: no entries, fallback 0
    ctxs = [np.array([3, 3, 3, 3], np.int32), np.array([1], np.int32)]
    assert_drafts_equal(b, dr, ng, ctxs, 3, [(3, 4)], stride=8)     # context drafter alone, then fallback
    b, dr, ng = build_both(np.array([7], np.int32), np.array([0, 0, 1, 1], np.int64), 3, 1, 16)
    assert_tables_equal(dr, ng)                                     # one single-token document: fallback 7, no n-grams
    doc = np.array([5, 9, 2, 7, 7, 3, 1, 8, 4, 6, 0, 11] * 6, np.int32)
    b, dr, ng = build_both(doc, np.arange(7, dtype=np.int64) * 12, 3, 5, 16)
    assert_tables_equal(dr, ng)
    got = b.tasc_draft(dr, torch.tensor([[5, 9, 2, 7] + [0] * 12], dtype=torch.int32).cuda(),
                       torch.tensor([4], dtype=torch.int32).cuda(), 6, 1, 1).cpu().numpy()
    assert got.tolist() == [[7, 3, 1, 8, 4, 6]]                     # a repeated document is continued verbatim


@pytest.mark.gpu
def test_build_rejects_bad_input():
    b = need_gpu()
    toks = torch.tensor([1, 2, 99], dtype=torch.int32).cuda()
    offs = torch.tensor([0, 3], dtype=torch.int64).cuda()
    with pytest.raises(b.TascError) as e:
        b.tasc_drafter_build(toks, offs, 3, 1, 50)                  # token id outside the vocabulary
    assert e.value.code == b.EINVAL
    with pytest.raises(b.TascError):
        b.tasc_drafter_build(toks, offs, 6, 1, 100)                 # n_max above TASC_MAX_ORDER
    with pytest.raises(b.TascError):
        b.tasc_drafter_build(toks, torch.tensor([1, 3], dtype=torch.int64).cuda(), 3, 1, 100)   # offsets[0] != 0


@pytest.mark.gpu
def test_drafts_do_not_depend_on_table_layout():
    """Slot placement depends on thread timing; two builds must still answer identically."""
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=800)
    b, dr1, ng = build_both(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    _, dr2, _ = build_both(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    ctxs = draft_contexts(cfg, tokens, offsets, 32, 60, seed=3)
    tok = np.zeros((32, 64), dtype=np.int32); ln = np.zeros(32, np.int32)
    for i, c in enumerate(ctxs):
        tok[i, :len(c)] = c; ln[i] = len(c)
    t, l = torch.from_numpy(tok).cuda(), torch.from_numpy(ln).cuda()
    assert torch.equal(b.tasc_draft(dr1, t, l, 4), b.tasc_draft(dr2, t, l, 4))


@pytest.mark.gpu
def test_config2_full_corpus_tables():
    """All 200,000 documents (14 M tokens) of configuration 2's corpus, n_max 4, p_min 5: export bit-exact."""
    cfg = configs.get(2)
    tokens, offsets = corpus.make_corpus(cfg)
    assert len(offsets) - 1 == 200000
    b, dr, ng = build_both(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    assert_tables_equal(dr, ng)


@pytest.mark.gpu
def test_config4_corpus_slice_tables_at_order_5():
    """The first 200,000 of configuration 4's 1,000,000 documents (22 M tokens, 110 M count updates at n_max 5,
    the 20,000-phrase pool): the largest slice the sort-based oracle builder handles in about two minutes."""
    cfg = configs.get(4)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=200000)
    b, dr, ng = build_both(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    assert_tables_equal(dr, ng)
    ctxs = draft_contexts(cfg, tokens, offsets, 24, 600, seed=4)
    assert_drafts_equal(b, dr, ng, ctxs, cfg.k, [(3, 4), (1, 1)], stride=640)


@pytest.mark.gpu
def test_export_then_import_gives_the_same_drafter():
    """A drafter rebuilt from its own canonical export (without the corpus) exports the same entries and drafts the same."""
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=1200)
    b, dr, ng = build_both(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    ent, fb = dr.export()
    r = np.random.default_rng(0)
    dr2 = b.tasc_drafter_import(ent[r.permutation(len(ent))], fb, cfg.n_max, cfg.model.vocab)      # any order of the entries
    ent2, fb2 = dr2.export()
    assert fb2 == fb and np.array_equal(ent2, ent)
    assert_tables_equal(dr2, ng)
    ctxs = draft_contexts(cfg, tokens, offsets, 48, 100, seed=7)
    assert_drafts_equal(b, dr2, ng, ctxs, cfg.k, [(3, 4), (1, 1), (0, 1)], stride=128)
    empty = b.tasc_drafter_import(np.zeros((0, D.MAX_ORDER + 3), np.int64), 5, 3, 16)
    ent3, fb3 = empty.export()
    assert fb3 == 5 and len(ent3) == 0
    bad = ent.copy()
    bad[0, D.MAX_ORDER + 1] = cfg.model.vocab                                                      # next token outside the vocabulary
    with pytest.raises(b.TascError):
        b.tasc_drafter_import(bad, fb, cfg.n_max, cfg.model.vocab)
