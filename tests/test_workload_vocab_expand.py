"""Input preparation of configuration 3 (vocabulary expansion): closed forms and brute force on tiny inputs."""
import numpy as np

from workload import vocab_expand as VE
from workload.weights import round_to_bf16


def tiny_corpus():
    docs = [[1, 2, 3, 4, 9], [1, 2, 3, 4], [7, 1, 2, 3], [1, 2, 5], [8, 8, 8, 8, 8], [1, 2]]
    toks = np.array([t for d in docs for t in d], dtype=np.int32)
    offs = np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int64)
    return docs, toks, offs


def brute_counts(docs, n_max):
    c = {}
    for d in docs:
        for n in range(2, n_max + 1):
            for i in range(len(d) - n + 1):
                g = tuple(d[i:i + n])
                c[g] = c.get(g, 0) + 1
    return c


def test_selection_ranks_by_frequency_times_length_minus_one():
    docs, toks, offs = tiny_corpus()
    counts = brute_counts(docs, 4)
    merges = VE.select_merges(toks, offs, 4, n_max=4, vocab=16)
    rewards = sorted(((c * (len(g) - 1), len(g)) for g, c in counts.items()), reverse=True)
    assert [(counts[g] * (len(g) - 1), len(g)) for g in merges] == rewards[:4]
    # reward 6 four ways: (1,2,3) 3*2, (1,2,3,4) 2*3, (8,8,8) 3*2, (8,8,8,8) 2*3 -> longer first, then smaller
    assert merges[:4] == [(1, 2, 3, 4), (8, 8, 8, 8), (1, 2, 3), (8, 8, 8)]
    assert len(set(merges)) == 4


def test_no_merge_crosses_a_document_boundary():
    toks = np.array([1, 2, 1, 2, 1, 2], dtype=np.int32)
    offs = np.array([0, 2, 4, 6], dtype=np.int64)
    merges = VE.select_merges(toks, offs, 8, n_max=3, vocab=4)
    assert merges == [(1, 2)]                      # (2, 1) would need two documents


def test_new_rows_are_the_mean_of_their_constituents():
    r = np.random.default_rng(0)
    emb = round_to_bf16(r.normal(0, 0.02, (32, 8)).astype(np.float32))
    w = {"embed": emb, "lm_head": emb, "layers": [], "final_norm": np.ones(8, np.float32)}
    merges = [(3, 5), (1, 2, 4, 7), (9, 9, 9)]
    e = VE.expand_weights(w, merges)
    assert e["embed"].shape == (35, 8) and e["lm_head"] is e["embed"]
    assert np.array_equal(e["embed"][:32], emb)
    for i, g in enumerate(merges):
        want = np.mean(np.stack([emb[t].astype(np.float64) for t in g]), axis=0)
        assert np.abs(e["embed"][32 + i] - want).max() <= np.abs(want).max() * 2.0 ** -8 + 1e-12    # one bf16 rounding
    f = VE.expand_weights(w, merges, bf16=False)
    assert np.allclose(f["embed"][34], emb[9], rtol=1e-6)                       # mean of three equal rows


def test_retokenize_is_greedy_longest_match_and_invertible():
    merges = [(1, 2), (1, 2, 3), (3, 4)]
    toks = np.array([1, 2, 3, 4, 0, 1, 2, 1, 2, 3], dtype=np.int32)
    offs = np.array([0, 7, 10], dtype=np.int64)
    t2, o2 = VE.retokenize(toks, offs, merges, vocab=10)
    #  doc 0: [1 2 3] 4 0 [1 2]   (the longer match wins over (1, 2) + (3, 4));  doc 1: [1 2 3]
    assert t2.tolist() == [11, 4, 0, 10, 11] and o2.tolist() == [0, 4, 5]
    for d in range(2):
        assert VE.expand_back(t2[o2[d]:o2[d + 1]], merges, vocab=10) == toks[offs[d]:offs[d + 1]].tolist()


def test_expansion_shortens_a_phrase_corpus():
    from workload import configs, corpus
    cfg = configs.get(0)
    toks, offs = corpus.make_corpus(cfg, n_docs=400)
    merges = VE.select_merges(toks, offs, 64, n_max=4, vocab=cfg.model.vocab)
    t2, o2 = VE.retokenize(toks, offs, merges, vocab=cfg.model.vocab)
    assert t2.size < 0.9 * toks.size and t2.max() >= cfg.model.vocab and o2[-1] == t2.size
    assert VE.expand_back(t2[:o2[5]], merges, vocab=cfg.model.vocab) == toks[:offs[5]].tolist()
