"""Verify step and generation loop against the oracle, replayed in lock-step (the oracle's committed
state is fed to the device at every step, so one near-tie cannot derail the rest of the comparison)."""
import numpy as np
import pytest
import torch

from oracle import decode as G
from tests.gpu_harness import lockstep, make_setup, need_gpu, record_parity
from workload import configs, corpus

# logits tolerance: float32 model 1e-4 absolute; bf16 models max-abs 2e-2 or relative 1e-2 (an element passes if it is
# within either bound: |err| <= max(2e-2, 1e-2 |ref|)).
# token rule: a device argmax may differ from the oracle's only where the oracle's top-2 gap is below gap_tol.
F32_TOL = dict(logit_atol=1e-4, logit_rtol=0.0, gap_tol=2e-4)
BF16_TOL = dict(logit_atol=2e-2, logit_rtol=1e-2, gap_tol=1e-2)


def check(rep, name, max_near_tie_frac=0.05):
    """Drafts bit-exact, no logit outside the tolerance, no argmax mismatch outside a near-tie, and near-tie
    mismatches on at most 5 % of the compared rows (observed: below 1 %); the counts go to the parity report."""
    record_parity(name, rep)
    print(f"lockstep {name}: steps={rep.steps} rows={rep.rows} near_tie_mismatches={rep.near_tie_mismatches} "
          f"max_logit_err={rep.max_logit_err:.3e} (x{rep.max_err_over_or_bound:.2f} of the either-bound reading)")
    assert rep.steps > 0
    assert rep.draft_mismatches == 0, "drafts must be bit-exact"
    assert not rep.hard_mismatches, rep.hard_mismatches[:5]
    assert rep.accept_mismatches == 0
    assert rep.near_tie_mismatches <= max(1, max_near_tie_frac * rep.rows)


def assert_diverges_only_at_a_near_tie(got, spec, gap_tol, what):
    """A free-running generation may leave the oracle's only at a token whose own logit row had a top-2 gap below
    the tolerance in the oracle (the row that produced the first differing token, not any row anywhere)."""
    want = np.array(spec.tokens)
    if np.array_equal(got, want):
        return None
    first = int(np.argmax(got != want))
    # the oracle step and row that produced generated token `first`: a step commits its accepted drafts
    # (rows 0..a-1 confirmed them) and then the argmax of row a
    g = 0
    for st in spec.steps:
        n = st.n_accepted + 1
        if first < g + n:
            row = first - g
            assert st.gap[row] < gap_tol, f"{what} diverges at token {first} (row {row}, gap {st.gap[row]:.3e}) without a near-tie"
            return first
        g += n
    raise AssertionError(f"{what}: token {first} is beyond the oracle's steps")


@pytest.mark.gpu
def test_config0_lockstep_full():
    cfg = configs.get(0)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 1)
    check(lockstep(s, prompts, cfg.max_new, cfg.k, **F32_TOL), "config0 B=1 full")


@pytest.mark.gpu
def test_config0_batch_with_gain_jitter_and_ragged_prompts():
    cfg = configs.get(0)
    s = make_setup(cfg, gain_jitter=0.2)
    prompts = corpus.make_prompts(cfg, 5, prompt_len=37)          # 37: prefill ends in a ragged chunk
    check(lockstep(s, prompts, 24, 7, **F32_TOL), "config0 B=5 k=7 gain jitter ragged prompts")


@pytest.mark.gpu
def test_config0_teacher_forced_accept_lengths():
    cfg = configs.get(0)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 3)
    for a in (0, 2, cfg.k):
        rep = lockstep(s, prompts, 20, cfg.k, oracle_kwargs=[dict(forced_accept=a)] * 3, forced_mode="accept", **F32_TOL)
        check(rep, f"config0 forced accept {a}")


@pytest.mark.gpu
@pytest.mark.parametrize("side_stream", [False, True])      # a non-default stream makes tasc_generate replay a CUDA graph
def test_config0_generate_matches_oracle_and_plain_greedy(side_stream):
    b = need_gpu()
    cfg = configs.get(0)
    s = make_setup(cfg)
    B = 4
    prompts = corpus.make_prompts(cfg, B)
    P = prompts.shape[1]
    stride = P + cfg.max_new + cfg.k + 1
    tokens = torch.zeros((B, stride), dtype=torch.int32, device="cuda")
    tokens[:, :P] = torch.from_numpy(prompts).cuda()
    length = torch.full((B,), P, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(B, stride + b.MAX_ROWS)
    ws = s.model.new_workspace(B, cfg.k)
    stream = torch.cuda.Stream() if side_stream else torch.cuda.current_stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        out, st = b.tasc_generate(s.model, s.drafter, kv, b.make_seqs(tokens, length), B, cfg.max_new, cfg.k, ws)
    torch.cuda.current_stream().wait_stream(stream)
    out = out.cpu().numpy()
    assert st.steps >= cfg.max_new // (cfg.k + 1) and st.committed >= B * cfg.max_new
    assert sum(st.accepted_hist) > 0 and st.decode_ms > 0
    for i in range(B):
        spec = G.greedy_speculative(s.oracle, s.ngrams, prompts[i], cfg.max_new, cfg.k)
        assert_diverges_only_at_a_near_tie(out[i], spec, F32_TOL["gap_tol"], f"sequence {i}")
    # the committed tokens on the device equal the returned output
    tok = tokens.cpu().numpy()
    assert np.array_equal(tok[:, P:P + cfg.max_new], out)
    assert (length.cpu().numpy() >= P + cfg.max_new).all()


@pytest.mark.gpu
def test_kv_exhaustion_is_reported_not_faulted():
    b = need_gpu()
    cfg = configs.get(0)
    s = make_setup(cfg, build_drafter=False, oracle_ngrams=False)
    B, P, k = 1, 32, 4
    tokens = torch.zeros((B, 64), dtype=torch.int32, device="cuda")
    tokens[:, :P] = torch.from_numpy(corpus.make_prompts(cfg, B)).cuda()
    length = torch.full((B,), P, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(B, 32)           # two pages: positions 0..31 only
    ws = s.model.new_workspace(B, k)
    seqs = b.make_seqs(tokens, length)
    b.tasc_prefill(s.model, kv, seqs, B, P, ws)
    b.tasc_poll_status(ws)
    drafts = torch.zeros((B, k), dtype=torch.int32, device="cuda")
    b.tasc_verify_step(s.model, kv, seqs, drafts, ws)       # rows at positions 31..35: 32.. have no page
    with pytest.raises(b.TascError) as e:
        b.tasc_poll_status(ws)
    assert e.value.code == b.ENOKV
    b.tasc_poll_status(ws)                                  # cleared


@pytest.mark.gpu
def test_verify_rejects_bad_arguments():
    b = need_gpu()
    cfg = configs.get(0)
    s = make_setup(cfg, build_drafter=False, oracle_ngrams=False)
    tokens = torch.zeros((1, 64), dtype=torch.int32, device="cuda")
    length = torch.ones(1, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(1, 64)
    seqs = b.make_seqs(tokens, length)
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.TascError) as e:
        b.tasc_verify_step(s.model, kv, seqs, torch.zeros((1, 4), dtype=torch.int32, device="cuda"), small)
    assert e.value.code == b.EINVAL
    ws = s.model.new_workspace(1, 4)
    with pytest.raises(b.TascError):
        b.tasc_verify_step(s.model, kv, seqs, torch.zeros((1, 16), dtype=torch.int32, device="cuda"), ws)   # k + 1 > 16


# ------------------------------------------------------------------------------------------ bf16 configurations
@pytest.fixture(scope="module")
def setup1():
    return make_setup(configs.get(1))


@pytest.mark.gpu
def test_config1_lockstep_batch1_full(setup1):
    cfg = configs.get(1)
    prompts = corpus.make_prompts(cfg, 1)
    check(lockstep(setup1, prompts, cfg.max_new, cfg.k, **BF16_TOL), "config1 B=1 full depth, 128 tokens")


@pytest.mark.gpu
def test_config1_lockstep_batch16_short(setup1):
    cfg = configs.get(1)
    prompts = corpus.make_prompts(cfg, 16)
    check(lockstep(setup1, prompts, 12, cfg.k, **BF16_TOL), "config1 B=16 full depth, 12 tokens")


@pytest.mark.gpu
def test_config1_teacher_forced_continuation(setup1):
    cfg = configs.get(1)
    prompts = corpus.make_prompts(cfg, 2)
    cont = corpus.make_continuations(cfg, prompts, 40 + cfg.k + 1)
    rep = lockstep(setup1, prompts, 40, cfg.k, oracle_kwargs=[dict(continuation=cont[i]) for i in range(2)],
                   forced_mode="continuation", **BF16_TOL)
    check(rep, "config1 B=2 teacher-forced continuation")


@pytest.mark.gpu
def test_config2_lockstep_short():
    cfg = configs.get(2)
    s = make_setup(cfg, n_docs=20000)
    prompts = corpus.make_prompts(cfg, 2)
    check(lockstep(s, prompts, 18, 8, **BF16_TOL), "config2 B=2 k=8 full depth, 18 tokens")


@pytest.mark.gpu
def test_config3_expanded_vocabulary_lockstep():
    """Configuration 3: 8,192 merged n-gram tokens on top of the 0.5B vocabulary (V = 160,128), embedding rows
    initialised as constituent means, corpus and prompts re-tokenised by greedy longest match.  Two layers and a
    3,000-document corpus keep the oracle quick; the LM head / argmax and the drafter run at the full vocabulary."""
    from dataclasses import replace
    from workload import vocab_expand as VE, weights as W
    cfg3 = configs.get(3)
    base = cfg3.model.vocab
    small = configs.shrunk(cfg3, n_layers=2, n_docs=3000)
    toks, offs = corpus.make_corpus(small)
    merges = VE.select_merges(toks, offs, cfg3.n_merged_tokens, n_max=4, vocab=base)
    assert len(merges) == cfg3.n_merged_tokens
    toks2, offs2 = VE.retokenize(toks, offs, merges, vocab=base)
    host_w = VE.expand_weights(W.make_weights(small.model, small.seed_weights), merges)
    cfg = replace(small, model=replace(small.model, vocab=base + len(merges)))
    s = make_setup(cfg, host_w=host_w, corpus_tokens=(toks2, offs2))
    raw = corpus.make_prompts(small, 2)
    re = [VE.retokenize(raw[i], np.array([0, raw.shape[1]]), merges, vocab=base)[0] for i in range(2)]
    P = min(len(r) for r in re)
    prompts = np.stack([r[:P] for r in re]).astype(np.int32)
    assert prompts.max() >= base                      # merged tokens do occur in the prompts
    check(lockstep(s, prompts, 12, cfg.k, **BF16_TOL), "config3 merged vocabulary, 2 layers, B=2")


@pytest.mark.gpu
def test_config4_shape_long_context_lockstep():
    """Configuration 4's geometry (d_model 1536, 12 query / 2 KV heads of 128, d_ff 8960, n_max 5, k 6, prompts of
    1,024 tokens) with two layers and a 32k vocabulary: 128-wide heads, a context long enough for the key range of a
    (sequence, KV head) to be split over a cluster, and prefill chunks of 96 query rows per KV head."""
    cfg = configs.shrunk(configs.get(4), n_layers=2, vocab=32768, n_docs=20000)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 2)
    check(lockstep(s, prompts, 14, cfg.k, **BF16_TOL), "config4 geometry, 2 layers, B=2")


@pytest.mark.gpu
def test_bf16_prefill_of_ragged_lengths_in_wide_passes():
    """Prompts of 300, 37, 129 and 257 tokens in one batch of configuration 1's geometry (two layers): the bf16
    prefill runs passes of 256 rows per sequence, cut into blocks of 16 rows for the attention, so the batch has
    a sequence that needs a second pass, sequences that end inside a block, and one whose second pass is a single
    row.  The verify step that follows must see the cache the oracle builds token by token."""
    b = need_gpu()
    cfg = configs.shrunk(configs.get(1), n_layers=2, n_docs=2000)
    s = make_setup(cfg, build_drafter=False, oracle_ngrams=False)
    lens = [300, 37, 129, 257]
    B, k = len(lens), cfg.k
    rng = np.random.default_rng(5)
    stride = max(lens) + 4 * (k + 1)
    host = np.zeros((B, stride), dtype=np.int32)
    for i, L in enumerate(lens):
        host[i, :L] = rng.integers(0, cfg.model.vocab, L)
    drafts_h = rng.integers(0, cfg.model.vocab, (B, k)).astype(np.int32)
    tokens = torch.from_numpy(host).cuda()
    length = torch.tensor(lens, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(B, stride + b.MAX_ROWS)
    ws = s.model.new_workspace(B, k)
    seqs = b.make_seqs(tokens, length)
    b.tasc_prefill(s.model, kv, seqs, B, max(lens), ws)
    n_acc, nxt, tgt, logits = b.tasc_verify_step(s.model, kv, seqs, torch.from_numpy(drafts_h).cuda(), ws,
                                                 want_targets=True, want_logits=True)
    b.tasc_poll_status(ws)
    lg, tgt = logits.cpu().numpy(), tgt.cpu().numpy()
    for i, L in enumerate(lens):
        cache = s.oracle.new_cache(L + k + 1)
        s.oracle.prefill(host[i, :L - 1], cache)
        st = G.verify_step(s.oracle, cache, int(host[i, L - 1]), list(map(int, drafts_h[i])), keep_logits=True)
        err = np.abs(lg[i] - st.logits)
        assert (err <= np.maximum(BF16_TOL["logit_atol"], BF16_TOL["logit_rtol"] * np.abs(st.logits))).all(), (i, float(err.max()))
        for r in range(k + 1):
            assert int(tgt[i, r]) == st.y[r] or st.gap[r] < BF16_TOL["gap_tol"], (i, r)


@pytest.mark.gpu
def test_config2_batch32_k3_and_k8_one_step():
    """Batch 32 of configuration 2's geometry at k = 3 (M = 128 rows, one token tile) and k = 8 (M = 288 rows, three
    token tiles of 96), two layers."""
    cfg = configs.shrunk(configs.get(2), n_layers=2, vocab=32768, n_docs=5000)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 32, prompt_len=80)
    for k in (3, 8):
        check(lockstep(s, prompts, k + 1, k, **BF16_TOL), f"config2 geometry, 2 layers, B=32 k={k}")


@pytest.mark.gpu
def test_config1_generate_graph_replay_equals_plain_enqueue(setup1):
    """tasc_generate on a side stream (captured step replayed from a CUDA graph) must produce exactly the tokens and
    statistics of the same call on the default stream (every step enqueued)."""
    b = need_gpu()
    cfg = configs.get(1)
    B, max_new, k = 3, 40, cfg.k
    prompts = corpus.make_prompts(cfg, B)
    P = prompts.shape[1]
    results = []
    for side in (False, True):
        stride = P + max_new + k + 2
        tokens = torch.zeros((B, stride), dtype=torch.int32, device="cuda")
        tokens[:, :P] = torch.from_numpy(prompts).cuda()
        length = torch.full((B,), P, dtype=torch.int32, device="cuda")
        pool, bt, kv = setup1.model.new_kv(B, stride + b.MAX_ROWS)
        ws = setup1.model.new_workspace(B, k)
        stream = torch.cuda.Stream() if side else torch.cuda.current_stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            out, st = b.tasc_generate(setup1.model, setup1.drafter, kv, b.make_seqs(tokens, length), B, max_new, k, ws)
        torch.cuda.current_stream().wait_stream(stream)
        results.append((out.cpu().numpy(), st.steps, list(st.accepted_hist)))
    assert np.array_equal(results[0][0], results[1][0])
    assert results[0][1:] == results[1][1:]


@pytest.mark.gpu
def test_a_wait_that_nothing_ends_times_out_and_leaves_the_context_usable():
    """The library's bounded barrier wait, driven to its limit on purpose by its own self-test kernel: the status word
    reports the time-out, the kernel returns, and the device keeps working (no trap, no hang)."""
    b = need_gpu()
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    b.tasc_selftest_bounded_wait(ws, 200_000)              # ~0.1 ms of SM cycles
    with pytest.raises(b.TascError) as e:
        b.tasc_poll_status(ws)
    assert e.value.code == b.ETIMEOUT
    b.tasc_poll_status(ws)                                 # cleared
    x = torch.ones((8, 64), dtype=torch.bfloat16, device="cuda")
    assert float(b.tasc_gemm_bf16(x, x).sum()) == 8 * 8 * 64
    with pytest.raises(b.TascError):
        b.tasc_selftest_bounded_wait(ws, 0)


# ------------------------------------------------------------------------------------------ widest batch, full depth
@pytest.mark.gpu
def test_config4_geometry_batch64_k6_rows_0_1_63():
    """Configuration 4's geometry at its benchmark batch: 64 sequences x (k + 1 = 7) rows = 448 GEMM rows (four token
    tiles of 112, 224 accumulator columns per tile), prompts of 1,024 tokens, two layers, 32k vocabulary.  The oracle
    runs sequences 0, 1 and 63; the other 61 decode along on the device."""
    cfg = configs.shrunk(configs.get(4), n_layers=2, vocab=32768, n_docs=20000)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 64)
    check(lockstep(s, prompts, 2 * (cfg.k + 1), cfg.k, oracle_rows=[0, 1, 63], **BF16_TOL),
          "config4 geometry, 2 layers, B=64 k=6 (M=448), rows 0/1/63")


@pytest.mark.gpu
@pytest.mark.parametrize("B", [16, 19, 32])
def test_config4_geometry_between_one_and_two_full_token_tiles(B):
    """Configuration 4's geometry (two layers, 32k vocabulary) at 16, 19 and 32 sequences x 7 rows: 112 rows = one token
    tile, where the layers take the few-row kernel (with its additional column finishers) and the LM head the many-row
    kernel; 133 rows = two token tiles of 80 whose second holds 53 rows (a ragged tail in the many-row kernel's last
    tile); 224 rows = two full tiles of 112.  The oracle runs the first and the last sequence."""
    cfg = configs.shrunk(configs.get(4), n_layers=2, vocab=32768, n_docs=20000)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, B, prompt_len=200)
    check(lockstep(s, prompts, cfg.k + 1, cfg.k, oracle_rows=[0, B - 1], **BF16_TOL),
          f"config4 geometry, 2 layers, B={B} k=6 (M={B * 7}), rows 0/{B - 1}")


@pytest.mark.gpu
def test_many_row_kernel_on_every_product_with_64_wide_heads():
    """A one-layer shape whose five weight matrices are all large enough for the many-row GEMM kernel (d_model 2,048,
    32 query / 8 KV heads of 64, d_ff 2,048, vocabulary 8,192: 8 to 34 MB each) at 40 sequences x 7 rows = 280 rows
    (three token tiles of 96) after a prefill in passes of 640 rows: its QKV epilogue with two RoPE halves of 32 per
    head, the split-K clusters of the narrow products, the residual and SiLU epilogues and the row arg-max.  The oracle
    runs sequences 0 and 39."""
    from dataclasses import replace
    base = configs.shrunk(configs.get(2), n_docs=3000)
    shape = replace(base.model, n_layers=1, d_model=2048, n_q_heads=32, n_kv_heads=8, head_dim=64, d_ff=2048, vocab=8192)
    cfg = replace(base, model=shape)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 40, prompt_len=80)
    check(lockstep(s, prompts, 2 * (cfg.k + 1), 6, oracle_rows=[0, 39], **BF16_TOL),
          "many-row kernel, 1 layer, d_model 2048, heads of 64, B=40 k=6 (M=280)")


@pytest.mark.gpu
def test_config4_full_depth_batch1():
    """The 1.5B shape at its full depth (28 layers, vocabulary 151,936, prompt of 1,024 tokens), one sequence,
    four or more steps; the corpus tables come from the first 20,000 documents."""
    cfg = configs.shrunk(configs.get(4), n_docs=20000)
    s = make_setup(cfg)
    prompts = corpus.make_prompts(cfg, 1)
    check(lockstep(s, prompts, 4 * (cfg.k + 1), cfg.k, **BF16_TOL), "config4 full depth (28 layers), B=1, 28 tokens")


@pytest.mark.gpu
def test_config3_full_depth_batch1():
    """The 0.5B shape with the merged vocabulary (V = 160,128) at its full depth of 24 layers, one sequence."""
    from dataclasses import replace
    from workload import vocab_expand as VE, weights as W
    cfg3 = configs.shrunk(configs.get(3), n_docs=5000)
    base = cfg3.model.vocab
    toks, offs = corpus.make_corpus(cfg3)
    merges = VE.select_merges(toks, offs, cfg3.n_merged_tokens, n_max=4, vocab=base)
    toks2, offs2 = VE.retokenize(toks, offs, merges, vocab=base)
    host_w = VE.expand_weights(W.make_weights(cfg3.model, cfg3.seed_weights), merges)
    cfg = replace(cfg3, model=replace(cfg3.model, vocab=base + len(merges)))
    s = make_setup(cfg, host_w=host_w, corpus_tokens=(toks2, offs2))
    raw = corpus.make_prompts(cfg3, 1)
    prompts = VE.retokenize(raw[0], np.array([0, raw.shape[1]]), merges, vocab=base)[0][None, :].astype(np.int32)
    check(lockstep(s, prompts, 4 * (cfg.k + 1), cfg.k, **BF16_TOL), "config3 full depth (24 layers, V=160,128), B=1, 24 tokens")


def one_step_from_prompts(b, s, prompts, drafts_h, k):
    """Prefill + one verify step with the given drafts; returns (logits, targets, n_accepted, next) as numpy."""
    B, P = prompts.shape
    stride = P + 2 * (k + 1)
    tokens = torch.zeros((B, stride), dtype=torch.int32, device="cuda")
    tokens[:, :P] = torch.from_numpy(prompts).cuda()
    length = torch.full((B,), P, dtype=torch.int32, device="cuda")
    pool, bt, kv = s.model.new_kv(B, stride + b.MAX_ROWS)
    ws = s.model.new_workspace(B, k)
    seqs = b.make_seqs(tokens, length)
    b.tasc_prefill(s.model, kv, seqs, B, P, ws)
    n_acc, nxt, tgt, logits = b.tasc_verify_step(s.model, kv, seqs, torch.from_numpy(drafts_h).cuda(), ws,
                                                 want_targets=True, want_logits=True)
    b.tasc_poll_status(ws)
    return logits.cpu().numpy(), tgt.cpu().numpy(), n_acc.cpu().numpy(), nxt.cpu().numpy()


# A sequence's result must not depend on what else is in the batch.  It cannot be bit-identical: the number of
# k-splits of a projection and of key-range splits of the attention is planned from the row count, so float32 sums
# are associated differently at B = 1 and B = 16 / 64, and a K or V element that lands on the other side of a bf16
# rounding boundary moves by 2^-9 of its value.  The bound is a quarter of the tolerance against the oracle.
BATCH_INVARIANCE_ATOL = 5e-3


@pytest.mark.gpu
@pytest.mark.parametrize("which,B,rows", [(1, 16, (0, 7, 15)), (4, 64, (0, 63))])
def test_a_sequence_does_not_depend_on_its_batch(which, B, rows):
    b = need_gpu()
    if which == 1:
        cfg = configs.shrunk(configs.get(1), n_docs=2000)                              # full depth: 30 layers
    else:
        cfg = configs.shrunk(configs.get(4), n_layers=2, vocab=32768, n_docs=2000)
    s = make_setup(cfg, build_drafter=False, oracle_ngrams=False)
    k = cfg.k
    prompts = corpus.make_prompts(cfg, B)
    drafts_h = np.random.default_rng(11).integers(0, cfg.model.vocab, (B, k)).astype(np.int32)
    lg, tgt, n_acc, nxt = one_step_from_prompts(b, s, prompts, drafts_h, k)
    worst = 0.0
    for i in rows:
        lg1, tgt1, n_acc1, nxt1 = one_step_from_prompts(b, s, prompts[i:i + 1], drafts_h[i:i + 1], k)
        diff = float(np.abs(lg[i] - lg1[0]).max())
        worst = max(worst, diff)
        assert diff <= BATCH_INVARIANCE_ATOL, (i, diff)
        top2 = np.sort(lg1[0], axis=-1)[:, -2:]
        gap = top2[:, 1] - top2[:, 0]
        for r in range(k + 1):
            assert tgt[i, r] == tgt1[0, r] or gap[r] <= 2 * diff, (i, r, gap[r], diff)
        if (tgt[i] == tgt1[0]).all():
            assert n_acc[i] == n_acc1[0] and nxt[i] == nxt1[0]
    print(f"batch invariance config {which} B={B}: max |logit difference| {worst:.3e}")


@pytest.mark.gpu
def test_whole_verify_step_is_bitwise_repeatable(setup1):
    """The same step from the same state twice (split-K and the attention merge are reduced in a fixed order, the
    LM-head maximum is order-free): logits, targets and the committed result must be bit-identical."""
    b = need_gpu()
    cfg = configs.get(1)
    B, k = 16, cfg.k
    prompts = corpus.make_prompts(cfg, B)
    drafts_h = np.random.default_rng(3).integers(0, cfg.model.vocab, (B, k)).astype(np.int32)
    first = one_step_from_prompts(b, setup1, prompts, drafts_h, k)
    for _ in range(2):
        again = one_step_from_prompts(b, setup1, prompts, drafts_h, k)
        for x, y in zip(first, again):
            assert np.array_equal(x, y)


@pytest.mark.gpu
def test_config1_generate_against_the_oracle(setup1):
    """tasc_generate (bf16 model, graph-replayed steps) free-running against the oracle's speculative decoding:
    a sequence may leave the oracle's tokens only at a token whose own oracle row was a near-tie."""
    b = need_gpu()
    cfg = configs.get(1)
    B, max_new, k = 2, 48, cfg.k
    prompts = corpus.make_prompts(cfg, B)
    P = prompts.shape[1]
    stride = P + max_new + k + 2
    tokens = torch.zeros((B, stride), dtype=torch.int32, device="cuda")
    tokens[:, :P] = torch.from_numpy(prompts).cuda()
    length = torch.full((B,), P, dtype=torch.int32, device="cuda")
    pool, bt, kv = setup1.model.new_kv(B, stride + b.MAX_ROWS)
    ws = setup1.model.new_workspace(B, k)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        out, st = b.tasc_generate(setup1.model, setup1.drafter, kv, b.make_seqs(tokens, length), B, max_new, k, ws)
    torch.cuda.current_stream().wait_stream(stream)
    out = out.cpu().numpy()
    diverged = []
    for i in range(B):
        spec = G.greedy_speculative(setup1.oracle, setup1.ngrams, prompts[i], max_new, k)
        diverged.append(assert_diverges_only_at_a_near_tie(out[i], spec, BF16_TOL["gap_tol"], f"sequence {i}"))
    print(f"config 1 free-running generation: first divergence per sequence {diverged} (None = identical {max_new} tokens)")
