"""The model-derived bigram drafter (the comparison drafter of Section 6.2) on the device against the oracle:
the table entry by entry (a device argmax may differ from the oracle's only where the oracle's top-2 logit gap is
below the tolerance), and the drafts of the mixed drafter bit-exact given the same table."""
import numpy as np
import pytest
import torch

from oracle import drafter as D
from oracle import ngrammys as NG
from tests.gpu_harness import make_setup, need_gpu
from workload import configs, corpus
from workload.configs import ModelShape


def device_table(b, s, B):
    pool, bt, kv = s.model.new_kv(B, 16)
    ws = s.model.new_workspace(B, 1)
    table = b.tasc_bigram_table(s.model, kv, B, ws)
    b.tasc_poll_status(ws)
    return table


@pytest.mark.gpu
@pytest.mark.parametrize("which,B", [("f32", 48), ("bf16", 100)])
def test_whole_table_of_a_small_model(which, B):
    b = need_gpu()
    from dataclasses import replace
    cfg = configs.get(0)
    if which == "bf16":
        cfg = replace(cfg, model=ModelShape(n_layers=2, d_model=128, n_q_heads=4, n_kv_heads=2, head_dim=32, d_ff=256,
                                            vocab=512, dtype="bf16"))
    s = make_setup(cfg, build_drafter=False, oracle_ngrams=False, gain_jitter=0.1)
    got = device_table(b, s, B).cpu().numpy()                  # 512 tokens in passes of B: the last pass is ragged
    want, gap = NG.bigram_table(s.oracle)
    tol = 2e-4 if which == "f32" else 1e-2
    differ = np.flatnonzero(got != want)
    assert all(gap[t] < tol for t in differ), [(int(t), int(got[t]), int(want[t]), float(gap[t])) for t in differ[:5]]
    assert len(differ) <= 0.05 * len(want)
    print(f"bigram table ({which}): {len(differ)} of {len(want)} entries differ, all at near-ties")


@pytest.mark.gpu
def test_sampled_entries_of_config1_geometry_and_the_mixed_drafter():
    b = need_gpu()
    cfg = configs.shrunk(configs.get(1), n_layers=2, n_docs=1000)          # vocabulary 49,152, two layers
    s = make_setup(cfg, build_drafter=False, oracle_ngrams=False)
    table = device_table(b, s, 256)
    got = table.cpu().numpy()
    assert got.min() >= 0 and got.max() < cfg.model.vocab
    sample = np.random.default_rng(2).choice(cfg.model.vocab, 300, replace=False)
    want, gap = NG.bigram_table(s.oracle, sample)
    bad = [(int(t), int(got[t]), int(w), float(g)) for t, w, g in zip(sample, want, gap) if got[t] != w and g >= 1e-2]
    assert not bad, bad[:5]
    # the drafter built from the device's table drafts exactly what the oracle drafts from the same table
    dr = b.tasc_drafter_from_bigram(table, cfg.model.vocab)
    ng = NG.as_ngram_model(got)
    ent, fb = dr.export()
    assert fb == 0 and ent.shape[0] == cfg.model.vocab
    assert np.array_equal(ent[:, 0], np.ones(cfg.model.vocab)) and np.array_equal(ent[:, 1], np.arange(cfg.model.vocab))
    assert np.array_equal(ent[:, D.MAX_ORDER + 1], got) and np.array_equal(ent[:, D.MAX_ORDER + 2], np.ones(cfg.model.vocab))
    prompts = corpus.make_prompts(cfg, 12, prompt_len=96)
    tok = np.zeros((12, 128), dtype=np.int32)
    tok[:, :96] = prompts
    ln = np.full(12, 96, dtype=np.int32)
    t_dev, l_dev = torch.from_numpy(tok).cuda(), torch.from_numpy(ln).cuda()
    for num, den in [(1, 1), (1, 256), (1, 4), (3, 4), (0, 1)]:
        have = b.tasc_draft(dr, t_dev, l_dev, 6, num, den).cpu().numpy()
        ref = np.array([D.draft(ng, prompts[i].tolist(), 6, num, den) for i in range(12)], dtype=np.int32)
        assert np.array_equal(have, ref), (num, den)


@pytest.mark.gpu
def test_bigram_drafter_rejects_a_table_outside_the_vocabulary():
    b = need_gpu()
    with pytest.raises(b.TascError) as e:
        b.tasc_drafter_from_bigram(torch.tensor([1, 2, 7], dtype=torch.int32).cuda(), 3)
    assert e.value.code == b.EINVAL
