"""Tokenizer enrichment (Section 4) on the device against the oracle: the merge list of Algorithm 1 and the re-tokenised
corpus bit-exact, the added tokens' rows bit-exact (same float32 operations in the same order), and the longest-match
encoding bit-exact."""
import numpy as np
import pytest
import torch

from oracle import tasc_tok as T
from tests.gpu_harness import need_gpu
from workload import configs, corpus
from workload.weights import round_to_bf16


def to_dev(tokens, offsets):
    return (torch.from_numpy(np.asarray(tokens, np.int32)).cuda(), torch.from_numpy(np.asarray(offsets, np.int64)).cuda())


def merges_as_tuples(m):
    return [tuple(int(t) for t in row if t >= 0) for row in m.cpu().numpy()]


def flat(docs):
    toks = np.array([t for d in docs for t in d], dtype=np.int32)
    offs = np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int64)
    return toks, offs


def check_enrich(b, tokens, offsets, base_vocab, budget, n_max):
    want_merges, want_docs = T.enrich(tokens, offsets, base_vocab, budget, n_max)
    merges, toks, offs = b.tasc_tok_enrich(*to_dev(tokens, offsets), base_vocab, budget, n_max)
    assert merges_as_tuples(merges) == want_merges
    wt, wo = flat(want_docs)
    assert np.array_equal(offs.cpu().numpy(), wo) and np.array_equal(toks.cpu().numpy(), wt)
    return merges, want_merges


@pytest.mark.gpu
def test_textbook_and_degenerate_corpora():
    b = need_gpu()
    # the classic byte-pair example with n_max = 2 (a=0 b=1 c=2 d=3)
    check_enrich(b, *flat([[0, 0, 0, 1, 3, 0, 0, 0, 1, 0, 2]]), 4, 3, 2)
    # ties between the longer and the more frequent n-gram, a singleton 4-gram beating a frequent pair
    check_enrich(b, *flat([[1, 2, 3, 4, 9], [1, 2, 3, 4], [7, 1, 2, 3], [1, 2, 5]]), 16, 4, 4)
    # self-overlapping n-grams, documents of one token, empty documents, a budget larger than what can be merged
    check_enrich(b, *flat([[8, 8, 8, 8, 8], [1], [], [8, 8], [1, 2, 1, 2, 1]]), 16, 12, 3)
    check_enrich(b, *flat([[1], [2], [1], [2]]), 4, 5, 3)
    check_enrich(b, np.zeros(0, np.int32), np.array([0], np.int64), 4, 3, 2)
    check_enrich(b, *flat([[5, 6, 7, 5, 6, 7, 5, 6]]), 8, 0, 4)                 # budget 0: the corpus comes back unchanged


@pytest.mark.gpu
@pytest.mark.parametrize("n_max,budget", [(2, 40), (4, 48), (6, 24)])
def test_synthetic_task_corpus(n_max, budget):
    b = need_gpu()
    cfg = configs.get(0)
    tokens, offsets = corpus.make_corpus(cfg, n_docs=250)
    merges, want = check_enrich(b, tokens, offsets, cfg.model.vocab, budget, n_max)
    assert len(want) == budget and max(len(g) for g in want) <= n_max
    assert any(t >= cfg.model.vocab for g in want for t in g)                      # merges of merges do occur

    # rows of the added tokens: float32 and bf16 matrices
    r = np.random.default_rng(3)
    E = r.standard_normal((cfg.model.vocab, 96)).astype(np.float32)
    rows = b.tasc_tok_init_rows(torch.from_numpy(E).cuda(), merges).cpu().numpy()
    assert np.array_equal(rows, T.new_rows(E, want, cfg.model.vocab, bf16=False))
    E16 = round_to_bf16(E)
    rows16 = b.tasc_tok_init_rows(torch.from_numpy(E16).cuda().bfloat16(), merges).float().cpu().numpy()
    assert np.array_equal(rows16, T.new_rows(E16, want, cfg.model.vocab, bf16=True))

    # encoding fresh text (prompts and other documents of the same generator) with the enriched vocabulary
    other, ooffs = corpus.make_corpus(cfg, n_docs=320)
    other, ooffs = other[ooffs[250]:], ooffs[250:] - ooffs[250]
    prompts = corpus.make_prompts(cfg, 6)
    docs = [other[ooffs[i]:ooffs[i + 1]].tolist() for i in range(len(ooffs) - 1)] + [p.tolist() for p in prompts] + [[], [3]]
    toks, offs = b.tasc_tok_encode(*to_dev(*flat(docs)), cfg.model.vocab, merges)
    want_docs = [T.encode(d, want, cfg.model.vocab) for d in docs]
    wt, wo = flat(want_docs)
    assert np.array_equal(offs.cpu().numpy(), wo) and np.array_equal(toks.cpu().numpy(), wt)
    assert len(wt) < sum(map(len, docs))                                           # the text did get shorter


@pytest.mark.gpu
def test_rejects_bad_arguments():
    b = need_gpu()
    t, o = to_dev([1, 2, 3], [0, 3])
    with pytest.raises(b.TascError):
        b.tasc_tok_enrich(t, o, 8, 2, 7)                       # n_max above TASC_TOK_MAX_N
    with pytest.raises(b.TascError):
        b.tasc_tok_enrich(t, o, 8, 2, 1)                       # n_max below 2
    bad = torch.tensor([[9, 1, -1, -1, -1, -1]], dtype=torch.int32).cuda()          # constituent 9 = an added token that does not exist yet
    with pytest.raises(b.TascError):
        b.tasc_tok_init_rows(torch.zeros((8, 4), device="cuda"), bad)
    with pytest.raises(b.TascError):
        b.tasc_tok_encode(t, o, 8, bad)
