"""Pins of the tokenizer-enrichment oracle: a textbook byte-pair example, brute-force recounts, closed forms and
invariants that a wrong reward, a crossed document boundary or a wrong replacement rule breaks."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import tasc_tok as T


def corpus(docs):
    toks = np.array([t for d in docs for t in d], dtype=np.int64)
    offs = np.concatenate([[0], np.cumsum([len(d) for d in docs])]).astype(np.int64)
    return toks, offs


def test_with_bigrams_only_it_is_byte_pair_encoding():
    """n_max = 2 turns Algorithm 1 into the BPE training loop (merge the most frequent pair, replace, repeat).  The
    classic worked example 'aaabdaaabac' (a=0, b=1, c=2, d=3): 'aa' is the most frequent pair; after it 'Za' and 'ab'
    tie at two occurrences and the one that occurs first is taken; three merges leave five symbols."""
    text = [0, 0, 0, 1, 3, 0, 0, 0, 1, 0, 2]
    merges, docs = T.enrich(*corpus([text]), base_vocab=4, budget=3, n_max=2)
    assert merges[0] == (0, 0)
    assert docs == [[6, 3, 6, 0, 2]]                       # X d X a c
    assert merges == [(0, 0), (4, 0), (5, 1)]              # Z = aa, Y = Za, X = Yb
    assert T.expansion(merges, 4, 6) == [0, 0, 0, 1]


def test_reward_prefers_long_frequent_ngrams_and_ties_go_to_the_longer_then_the_earlier():
    # (1,2,3,4) occurs twice: reward 2*3 = 6; (1,2,3) three times: 3*2 = 6; (1,2) four times: 4*1 = 4
    docs = [[1, 2, 3, 4, 9], [1, 2, 3, 4], [7, 1, 2, 3], [1, 2, 5]]
    freq, first = T.collect_ngrams(docs, 4)
    assert freq[(1, 2, 3, 4)] == 2 and freq[(1, 2, 3)] == 3 and freq[(1, 2)] == 4 and first[(1, 2, 3)] == (0, 0)
    assert T.merge_reward(freq[(1, 2, 3, 4)], 4) == T.merge_reward(freq[(1, 2, 3)], 3) == 6
    merges, out = T.enrich(*corpus(docs), base_vocab=16, budget=2, n_max=4)
    assert merges[0] == (1, 2, 3, 4)                       # the longer of the two with reward 6
    # second round, recounted on the new tokenisation [[16 9] [16] [7 1 2 3] [1 2 5]]: the single 4-gram (7,1,2,3) saves
    # three tokens (reward 1 * 3), more than the pair (1,2) that occurs twice (reward 2 * 1)
    assert merges[1] == (7, 1, 2, 3)
    assert out == [[16, 9], [16], [17], [1, 2, 5]]


def test_nothing_crosses_a_document_and_the_loop_stops_when_nothing_is_left():
    merges, docs = T.enrich(*corpus([[1, 2], [1, 2], [1], []]), base_vocab=4, budget=5, n_max=3)
    assert merges == [(1, 2)] and docs == [[4], [4], [1], []]
    merges, _ = T.enrich(*corpus([[1], [2], [1], [2]]), base_vocab=4, budget=5, n_max=3)
    assert merges == []                                    # (1,2) and (2,1) exist only across boundaries


def test_replacement_is_left_to_right_and_non_overlapping():
    assert T.replace_ngram([8, 8, 8, 8, 8], (8, 8), 99) == [99, 99, 8]
    assert T.replace_ngram([1, 2, 1, 2, 1], (1, 2, 1), 99) == [99, 2, 1]
    assert T.replace_ngram([5], (5, 5), 99) == [5]


@settings(max_examples=60, deadline=None)
@given(st.lists(st.lists(st.integers(0, 5), min_size=0, max_size=12), min_size=1, max_size=6), st.integers(2, 4), st.integers(1, 6))
def test_invariants_on_random_corpora(docs, n_max, budget):
    toks, offs = corpus(docs)
    merges, out = T.enrich(toks, offs, base_vocab=6, budget=budget, n_max=n_max)
    # expanding every token gives the original documents back
    assert [[b for t in d for b in T.expansion(merges, 6, t)] for d in out] == docs
    # the chosen n-gram had the largest reward of its round (brute-force recount of that round), and the corpus shrank
    # by (n - 1) per replaced occurrence
    cur = [list(d) for d in docs]
    for i, g in enumerate(merges):
        counts = {}
        for d in cur:
            for n in range(2, n_max + 1):
                for j in range(len(d) - n + 1):
                    counts[tuple(d[j:j + n])] = counts.get(tuple(d[j:j + n]), 0) + 1
        assert counts[g] * (len(g) - 1) == max(c * (len(k) - 1) for k, c in counts.items())
        nxt = [T.replace_ngram(d, g, 6 + i) for d in cur]
        replaced = sum(d.count(6 + i) for d in nxt)
        assert sum(map(len, cur)) - sum(map(len, nxt)) == replaced * (len(g) - 1) and replaced >= 1
        cur = nxt
    assert cur == out
    # encoding the original text with the final vocabulary never yields more tokens than the training-time tokenisation
    # did before the first merge, and expands back to the text
    for d in docs:
        e = T.encode(d, merges, 6)
        assert [b for t in e for b in T.expansion(merges, 6, t)] == d and len(e) <= len(d)


def test_new_rows_are_the_mean_of_the_constituents_at_merge_time():
    E = np.arange(12, dtype=np.float32).reshape(4, 3)       # rows 0..3
    merges = [(1, 3), (4, 0, 2)]                            # token 4 = (1, 3); token 5 = (token 4, 0, 2)
    rows = T.new_rows(E, merges, 4, bf16=False)
    assert np.array_equal(rows[0], (E[1] + E[3]) / 2)
    assert np.array_equal(rows[1], ((rows[0] + E[0]) + E[2]) / np.float32(3))
    # bf16 models: the stored row is the nearest bf16 value of the float32 mean
    import torch
    E2 = np.random.default_rng(0).standard_normal((6, 5)).astype(np.float32)
    r = T.new_rows(E2, [(0, 1, 2), (3, 5)], 6, bf16=True)
    want0 = torch.tensor(((E2[0] + E2[1]) + E2[2]) / np.float32(3)).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r[0], want0)


def test_encoding_prefers_the_longest_added_token():
    merges = [(1, 2), (10, 3), (7, 7)]                      # 10 = (1,2), 11 = (1,2,3), 12 = (7,7)
    assert T.encode([1, 2, 3, 1, 2, 9, 7, 7, 7], merges, 10) == [11, 10, 9, 12, 7]
    assert T.encode([2, 3], merges, 10) == [2, 3]
    assert T.encode([], merges, 10) == []
