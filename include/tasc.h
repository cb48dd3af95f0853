/*
 * tasc.h -- C ABI of the B200 (sm_100a) implementation of one batched n-gram
 * speculative-decoding step (TASC-draft; paper Sections 5.1 and 5.2).
 *
 * Conventions
 *   - Plain C.  Every call returns a tasc_status (0 = OK, negative = error);
 *     nothing throws, aborts or traps across this boundary.
 *   - "device" pointers are CUDA global-memory addresses of the current device;
 *     "host" pointers are ordinary process memory.  Each argument says which.
 *   - tasc_stream is a cudaStream_t passed as void* (NULL = the default stream).
 *     Step calls (tasc_draft, tasc_verify_step, tasc_prefill) only enqueue work
 *     on that stream and return; they allocate nothing.  Device-side problems
 *     (a KV position outside the block table, a wait that ran out) are recorded
 *     in a status word inside the caller's workspace and read by
 *     tasc_poll_status, which synchronises the stream.
 *   - The caller owns weights, KV pool, block table, token buffers and the
 *     workspace.  The library owns only what tasc_drafter_build and
 *     tasc_model_create allocate, released by the matching destroy call.
 *   - Token ids are int32, document offsets int64.
 */
#ifndef TASC_H
#define TASC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t tasc_status;
#define TASC_OK          0
#define TASC_EINVAL    (-1)   /* bad argument (null pointer, size out of range, unsupported shape) */
#define TASC_ENOMEM    (-2)   /* device or host allocation failed */
#define TASC_ECUDA     (-3)   /* a CUDA runtime / driver call failed */
#define TASC_ECAPACITY (-4)   /* a hash table or output buffer is too small */
#define TASC_ENOKV     (-5)   /* a KV position falls outside the sequence's block table */
#define TASC_ETIMEOUT  (-6)   /* a bounded device-side wait ran out */

#define TASC_MAX_ORDER   5    /* largest context length n_max of the n-gram models */
#define TASC_MAX_ROWS   16    /* largest k + 1 (rows verified per sequence per step) */
#define TASC_VOCAB_BITS 20    /* token ids must be < 2^20 (six ids + order are packed in 128 bits) */
#define TASC_TOK_MAX_N    6    /* longest n-gram the tokenizer enrichment merges into one token */

#define TASC_F32   0
#define TASC_BF16  1

typedef void* tasc_stream;
typedef struct tasc_drafter tasc_drafter;
typedef struct tasc_model tasc_model;

/* One surviving element of a pruned n-gram model M_n: context of n tokens -> next token, count. */
typedef struct {
    int32_t  n;                      /* context length, 1..n_max */
    int32_t  ctx[TASC_MAX_ORDER];    /* ctx[0..n-1], oldest first; unused slots are -1 */
    int32_t  next;
    uint32_t count;
} tasc_ngram_entry;

/* ------------------------------------------------------------------ drafter */

/*
 * Build the corpus n-gram drafter p_corp (Section 5.2: n-gram models M_n, n <= n_max,
 * from the n-gram frequencies of the task's output corpus, each pruned of elements
 * whose frequency is below p_min; plus the most frequent token as the last resort).
 * n is the context length; n-grams do not cross document boundaries.
 *
 *   corpus_tokens  device, int32[doc_offsets[n_docs]], every id in [0, vocab)
 *   doc_offsets    device, int64[n_docs + 1], non-decreasing, doc_offsets[0] = 0
 *   n_max          1..TASC_MAX_ORDER;  p_min >= 1 (absolute count threshold)
 *   vocab          <= 2^TASC_VOCAB_BITS
 *   out            host; receives a handle owning device tables (tasc_drafter_destroy)
 * Device memory: the tables the handle owns (about 40 bytes per surviving element), and, while the call runs,
 * a counting table of 2^ceil(log2(2 W)) slots of 20 bytes, W = the windows of order 1 (tokens minus documents), plus
 * one byte per token -- about 5.4 GB for a corpus of 110 M tokens; freed before the call returns.
 * Synchronises the stream before returning.  Errors: EINVAL, ENOMEM, ECUDA,
 * ECAPACITY (internal table overflow; not expected for valid input).
 */
tasc_status tasc_drafter_build(const int32_t* corpus_tokens, const int64_t* doc_offsets, int64_t n_docs,
                               int32_t n_max, int32_t p_min, int32_t vocab, tasc_stream stream,
                               tasc_drafter** out);

/*
 * Canonical dump of the pruned models: entries sorted by (n, ctx, next).
 *   out        host, room for cap entries (may be NULL when cap = 0 to query the size)
 *   n_entries  host, receives the total number of entries (even if cap is smaller -> ECAPACITY)
 *   fallback_token  host, receives the most frequent corpus token (smallest id on ties)
 */
tasc_status tasc_drafter_export(const tasc_drafter* d, tasc_ngram_entry* out, int64_t cap, int64_t* n_entries,
                                int32_t* fallback_token);

/*
 * The inverse of tasc_drafter_export: a drafter handle from the surviving elements of the pruned models (any order of
 * the entries; a duplicate (n, ctx, next) is an error the call does not detect) and the last-resort token.  Used to
 * save a built drafter and load it again without the corpus.
 *   entries  host, n_entries of them;  n_max 1..TASC_MAX_ORDER;  every id in [0, vocab), every count >= 1
 *   out      host; receives a handle owning device tables (tasc_drafter_destroy)
 * Synchronises the stream.  Errors: EINVAL, ENOMEM, ECUDA.
 */
tasc_status tasc_drafter_import(const tasc_ngram_entry* entries, int64_t n_entries, int32_t n_max, int32_t vocab,
                                int32_t fallback_token, tasc_stream stream, tasc_drafter** out);

tasc_status tasc_drafter_destroy(tasc_drafter* d);

/*
 * Draft k tokens per sequence from p_mixed = lambda p_corp + (1 - lambda) p_prompt
 * (Section 5.2, mixture equation), lambda = lambda_num / lambda_den, argmax with the
 * smallest token id on ties, evaluated exactly in 64-bit integers.  p_corp: back-off
 * query of M_n in descending n with the last n tokens; p_prompt: the same construction
 * over the sequence's own committed tokens (no pruning).  Drafts already produced in this
 * call extend the query suffix only.  A component with zero weight or without a match at
 * any order takes no part; if neither does, the draft is the most frequent corpus token.
 *
 *   tokens   device, int32[B][stride]: committed tokens of each sequence
 *   len      device, int32[B]: committed length L_b (1 <= L_b <= stride)
 *   drafts   device, int32[B][k] (written)
 *   k        1..TASC_MAX_ROWS-1;  0 <= lambda_num <= lambda_den <= 256
 * Asynchronous on the stream.  Errors: EINVAL (also when stride is too large for the
 * kernel's shared-memory copy of the tokens and successor table: stride <= 12288, which is therefore the
 * longest context -- prompt plus generated tokens plus k + 1 -- the whole path supports).
 */
tasc_status tasc_draft(const tasc_drafter* d, const int32_t* tokens, int64_t stride, const int32_t* len,
                       int32_t B, int32_t k, int32_t lambda_num, int32_t lambda_den, int32_t* drafts,
                       tasc_stream stream);

/*
 * The comparison drafter of Section 6.2 (the "N-Grammys" bigram: for every token of the vocabulary the most probable
 * next token under the target model's own conditional distribution) as a drafter handle: an order-1 model in which
 * context token c has the single successor table[c] with count 1.  tasc_draft then mixes it with the context drafter
 * exactly as it mixes p_corp (a point mass in the place of p_corp: for lambda >= 1/2 it always wins; with a small
 * lambda the context drafter decides wherever it has a match and the bigram elsewhere).  The last-resort token is 0.
 *
 *   table   device, int32[vocab], every entry in [0, vocab) (tasc_bigram_table writes one)
 *   out     host; receives a handle owning device tables (tasc_drafter_destroy)
 * Synchronises the stream.  Errors: EINVAL (also for an entry outside the vocabulary), ENOMEM, ECUDA.
 */
tasc_status tasc_drafter_from_bigram(const int32_t* table, int32_t vocab, tasc_stream stream, tasc_drafter** out);

/*
 * Statistics of the task's output corpus C_task (Section 3: the concentration of the task-conditioned n-gram
 * distribution, Eq. 1-2, reported in Table 1 as the bigram Shannon entropy and the number of distinct bigrams
 * that cover 80 % of the bigram occurrences; Section 4.1 / Appendix "Uniform Information Density": the token
 * entropy divided by log |V|; Section 6.1 / Appendix "Predicting Model Speedup": the Renyi entropy of order 2 of
 * the token distribution, H_2 = -log sum_x p(x)^2).  A bigram is an adjacent token pair inside one document --
 * the windows of the order-1 model before pruning.  Entropies are in bits; typical_set_size = 2^H (Eq. 2).
 */
typedef struct {
    int64_t n_tokens;                 /* tokens of the corpus */
    int64_t n_bigrams;                /* bigram occurrences: sum over documents of max(0, length - 1) */
    int64_t n_unique_tokens;
    int64_t n_unique_bigrams;
    int64_t bigrams_for_cdf;          /* smallest m: the m most frequent bigrams hold >= cdf_num / cdf_den of n_bigrams */
    double  bigram_entropy_bits;
    double  typical_set_size;
    double  token_entropy_bits;
    double  token_entropy_normalised; /* token_entropy_bits / log2(vocab) */
    double  token_renyi2_bits;
} tasc_corpus_statistics;

/*
 *   corpus_tokens, doc_offsets, n_docs, vocab   as for tasc_drafter_build (device pointers)
 *   cdf_num / cdf_den   coverage target of bigrams_for_cdf (the paper's 80 % = 4 / 5); 1 <= cdf_num <= cdf_den <= 65536
 *   out                 host (written)
 * Counting and the reductions run on the device; the integer fields are exact and, like the entropies, do not depend
 * on thread timing.  Allocates transient device memory (about 40 bytes per bigram occurrence plus 8 MiB) and frees it
 * before returning; synchronises the stream.  The corpus must hold fewer than 2^40 tokens.
 * Errors: EINVAL, ENOMEM, ECUDA, ECAPACITY (more than 4,096 distinct bigrams or tokens occurring 2^20 times or more).
 */
tasc_status tasc_corpus_stats(const int32_t* corpus_tokens, const int64_t* doc_offsets, int64_t n_docs, int32_t vocab,
                              int32_t cdf_num, int32_t cdf_den, tasc_stream stream, tasc_corpus_statistics* out);

/* ------------------------------------------------------- tokenizer enrichment */

/*
 * Algorithm 1 of the paper (Section 4.1, "Tokenizer Enrichment"): starting from the base vocabulary, repeat `budget`
 * times: collect the token n-grams (2 <= n <= n_max) of the task corpus as tokenised with the current vocabulary,
 * score each with the merge reward f_merge(t^n) = freq(t^n) * (n - 1), add the argmax as one new token (id
 * base_vocab + i for the i-th addition) and replace its occurrences -- left to right, non-overlapping, inside each
 * document -- before the next round.  freq counts every window; windows do not span documents; argmax ties go to the
 * longer n-gram, then to the one that occurs first.  The prefix-collision test needs token strings and is not applied.
 * Stops early when no n-gram is left.
 *
 *   corpus_tokens, doc_offsets, n_docs   as for tasc_drafter_build (device); ids in [0, base_vocab); fewer than 2^28 tokens
 *   budget        additions M (base_vocab + budget <= 2^TASC_VOCAB_BITS);  n_max  2..TASC_TOK_MAX_N
 *   merges        device, int32[budget][TASC_TOK_MAX_N] (written): the constituents of each added token, ids of the
 *                 vocabulary at the time of the merge (a constituent may be an earlier added token), padded with -1
 *   n_merges      host (written): additions made
 *   tokens_out    device, int32[doc_offsets[n_docs]] (written): the corpus in the enriched vocabulary, compacted
 *   offsets_out   device, int64[n_docs + 1] (written)
 * Every round recounts the whole corpus: the cost is budget x corpus size, so select on a sample of the corpus.
 * Allocates transient device memory (about 50 bytes per n-gram window) and frees it; synchronises the stream.
 * Errors: EINVAL, ENOMEM, ECUDA, ECAPACITY.
 */
tasc_status tasc_tok_enrich(const int32_t* corpus_tokens, const int64_t* doc_offsets, int64_t n_docs, int32_t base_vocab,
                            int32_t budget, int32_t n_max, int32_t* merges, int32_t* n_merges, int32_t* tokens_out,
                            int64_t* offsets_out, tasc_stream stream);

/*
 * Rows of the added tokens for the embedding or the LM-head matrix (Section 4.2): e_new = (1/n) sum_j e_{t_j} over the n
 * constituents, summed in float32 in their order and divided by n, stored in the matrix's type (bf16: nearest even).
 *   matrix   device, [base_vocab][d] in `dtype` (TASC_F32 / TASC_BF16);  merges as written by tasc_tok_enrich
 *   rows_out device, [n_merges][d] in `dtype` (written; also read, for constituents that are added tokens)
 *   device_status  device, int32, zeroed by the caller: TASC_EINVAL if a merge names a token that does not exist yet
 * Asynchronous.  Errors: EINVAL.
 */
tasc_status tasc_tok_init_rows(const void* matrix, int32_t dtype, int32_t base_vocab, int32_t d, const int32_t* merges,
                               int32_t n_merges, void* rows_out, int32_t* device_status, tasc_stream stream);

/*
 * Encode base-token text with the enriched vocabulary (the paper's appendix on byte-pair encoding: the added tokens are
 * queried before the base tokenizer): at every position the added token with the longest expansion into base tokens
 * that matches the upcoming tokens (and ends inside the document) replaces them; elsewhere the base token stays.
 * Two added tokens with the same expansion: the earlier one.
 *   tokens, doc_offsets, n_docs   device, base-vocabulary text;  merges, n_merges as above (device)
 *   tokens_out   device, room for as many tokens as the input (written, compacted);  offsets_out device, int64[n_docs + 1]
 * The trie of the expansions is built on the host from the merge list (expansions of more than 4,096 base tokens:
 * ECAPACITY).  Allocates transient device memory; synchronises the stream.  Errors: EINVAL, ENOMEM, ECUDA, ECAPACITY.
 */
tasc_status tasc_tok_encode(const int32_t* tokens, const int64_t* doc_offsets, int64_t n_docs, int32_t base_vocab,
                            const int32_t* merges, int32_t n_merges, int32_t* tokens_out, int64_t* offsets_out,
                            tasc_stream stream);

/* -------------------------------------------------------------------- model */

/* Decoder shape (pre-norm, RMSNorm, rotate-half RoPE, grouped-query attention, SwiGLU, no biases). */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    int32_t dtype;          /* TASC_F32 or TASC_BF16: type of weight matrices, KV pool and GEMM inputs */
    float   rope_base;      /* e.g. 10000 */
    float   rms_eps;        /* e.g. 1e-6 */
    int32_t max_positions;  /* size of the rotary table: every position must be < max_positions */
    int32_t page_size;      /* tokens per KV page (16) */
} tasc_model_desc;

/*
 * Device pointers to the weights, borrowed for the lifetime of the model handle.
 * Matrices are row-major [out_features][in_features] in the model dtype; norm gains are float32.
 * The per-layer members are HOST arrays of n_layers device pointers.
 */
typedef struct {
    const void*  embed;          /* [vocab][d_model] */
    const void*  lm_head;        /* [vocab][d_model] (may equal embed) */
    const float* final_norm;     /* [d_model] */
    const float* const* attn_norm;   /* each [d_model] */
    const void*  const* wqkv;        /* each [(n_q + 2 n_kv) * head_dim][d_model]: q heads, k heads, v heads */
    const void*  const* wo;          /* each [d_model][n_q * head_dim] */
    const float* const* mlp_norm;    /* each [d_model] */
    const void*  const* w_gate_up;   /* each [2 * d_ff][d_model]: gate rows, then up rows */
    const void*  const* w_down;      /* each [d_model][d_ff] */
} tasc_weights;

/*
 * Paged KV cache, caller-owned.  pool layout (model dtype):
 *   [n_layers][2 (K, V)][n_pages][n_kv_heads][page_size][head_dim]
 * block_table[b][j] is the page holding positions j*page_size .. of sequence b.
 */
typedef struct {
    void*          pool;               /* device */
    int64_t        n_pages;
    const int32_t* block_table;        /* device, int32[B][max_pages_per_seq], every id in [0, n_pages) */
    int32_t        max_pages_per_seq;
} tasc_kv;

/*
 * Committed tokens of the batch.  The KV cache of sequence b holds positions 0 .. len[b]-2:
 * the last committed token has not been through the model yet.
 */
typedef struct {
    int32_t*       tokens;     /* device, int32[B][stride] */
    int64_t        stride;
    int32_t*       len;        /* device, int32[B] */
    const int32_t* stop_len;   /* device, int32[B] or NULL: a sequence with len >= stop_len is skipped */
} tasc_seqs;

/* Validates the shape, builds the rotary table and the weight tensor maps.  Errors: EINVAL, ENOMEM, ECUDA. */
tasc_status tasc_model_create(const tasc_model_desc* desc, const tasc_weights* weights, tasc_model** out);
tasc_status tasc_model_destroy(tasc_model* m);

/* Bytes of workspace that step calls need for up to B_max sequences and k_max drafts.  bf16 models reserve
 * room for at least 2,048 rows in flight, which prefill passes use (up to 256 rows per sequence; 140 MB for the
 * 1.5B shape, tens of MB for the small ones). */
size_t tasc_workspace_bytes(const tasc_model* m, int32_t B_max, int32_t k_max);

/*
 * Run the committed tokens 0 .. len[b]-2 of every sequence through the model to fill the KV
 * cache (no logits).  max_len (host value) >= every len[b]; it fixes the number of passes: a pass
 * carries 16 positions of every sequence (float32 models) or as many as the workspace holds, up to 256
 * per sequence (bf16 models), through the same kernels as a verify step; sequences shorter than a
 * pass's range take no part in it.  Asynchronous.  Errors: EINVAL.
 */
tasc_status tasc_prefill(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, int32_t B, int32_t max_len,
                         void* workspace, size_t workspace_bytes, tasc_stream stream);

/*
 * One verification step (Section 5.1: the target model verifies the drafted tokens in a single
 * forward pass and a prefix is accepted; greedy acceptance, i.e. beam size 1).
 * Rows [last committed token, d_1..d_k] of sequence b run at positions L-1 .. L-1+k (L = len[b]);
 * their K/V are appended to the cache; y_i = argmax of row i's logits (smallest id on ties);
 * a = longest prefix with d_j = y_{j-1}; d_1..d_a and y_a are appended to tokens and len grows by
 * a+1, which also rolls the KV cache back over the rejected rows.
 *
 *   drafts         device, int32[B][k]
 *   forced_targets device, int32[B][k+1] or NULL: replaces y in the accept rule and in what is
 *                  committed (teacher-forced mode); the forward pass still runs in full
 *   n_accepted     device, int32[B] (written): a, 0..k
 *   next_token     device, int32[B] (written): the token committed after the accepted drafts
 *   target_tokens  device, int32[B][k+1] or NULL (written): y
 *   logits_dbg     device, float[B][k+1][vocab] or NULL (written): all logits (debug; large)
 * Asynchronous.  Errors: EINVAL (k+1 > TASC_MAX_ROWS, workspace too small, ...).
 */
tasc_status tasc_verify_step(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, const int32_t* drafts,
                             int32_t B, int32_t k, const int32_t* forced_targets,
                             int32_t* n_accepted, int32_t* next_token, int32_t* target_tokens, float* logits_dbg,
                             void* workspace, size_t workspace_bytes, tasc_stream stream);

/* How tasc_generate chooses the targets of each step. */
#define TASC_MODE_GREEDY        0   /* targets = the model's own argmax */
#define TASC_MODE_CONTINUATION  1   /* teacher-forced: targets = continuation[b][g .. g+k], g = tokens generated so far */
#define TASC_MODE_FORCED_ACCEPT 2   /* teacher-forced: exactly forced_accept drafts are accepted every step */

typedef struct {
    int32_t k;
    int32_t lambda_num, lambda_den;
    int32_t mode;
    int32_t forced_accept;              /* TASC_MODE_FORCED_ACCEPT: 0..k */
    const int32_t* continuation;        /* TASC_MODE_CONTINUATION: device, int32[B][continuation_stride] */
    int64_t continuation_stride;        /* >= max_new + k + 1 */
} tasc_draft_params;

typedef struct {
    int64_t steps;                      /* speculative steps enqueued */
    int64_t committed;                  /* tokens committed over all sequences (before truncation to max_new) */
    int64_t accepted_hist[TASC_MAX_ROWS]; /* accepted_hist[a] = sequence-steps that accepted exactly a drafts */
    float   prefill_ms, decode_ms;      /* device time of the two phases */
} tasc_stats;

/*
 * Prefill, then repeat [draft k tokens -> verify step] until every sequence has generated max_new
 * tokens.  On entry seqs holds the prompts (len = prompt lengths, stride >= prompt + max_new + k + 1);
 * on return tokens/len hold prompt + generated tokens (a sequence may overshoot max_new by up to k).
 *   out    device, int32[B][max_new] (written): the first max_new generated tokens
 *   stats  host (written), may be NULL
 * On a stream other than the legacy default stream the step is captured once into a CUDA graph (after a first
 * plainly enqueued step) and replayed, which allocates the graph's resources for the duration of the call.
 * Synchronises the stream.  Errors: EINVAL, ECUDA, and device-side statuses (ENOKV, ETIMEOUT).
 */
tasc_status tasc_generate(const tasc_model* m, const tasc_drafter* d, const tasc_kv* kv, const tasc_seqs* seqs,
                          int32_t B, int32_t max_new, const tasc_draft_params* params, int32_t* out,
                          tasc_stats* stats, void* workspace, size_t workspace_bytes, tasc_stream stream);

/*
 * The bigram table of the comparison drafter of Section 6.2 ("N-Grammys": a bigram model obtained by taking the target
 * model's conditional distribution for each element of the vocabulary): table[t] = argmax over x of the model's logits
 * for the single-token context t (position 0, no earlier keys), smallest id on ties.  The vocabulary runs through the
 * verify forward (every layer, LM head, row argmax) as passes of B one-row sequences.
 *
 *   kv         a pool in which each of the B sequences has at least one page (block_table as for tasc_verify_step);
 *              its contents are overwritten
 *   B          single-token sequences per pass (1 .. as many as workspace and kv were sized for)
 *   table      device, int32[vocab] (written)
 *   workspace  at least tasc_workspace_bytes(m, B, 1) bytes
 * Asynchronous (ceil(vocab / B) forward passes are enqueued).  Errors: EINVAL; device-side statuses via tasc_poll_status.
 */
tasc_status tasc_bigram_table(const tasc_model* m, const tasc_kv* kv, int32_t B, int32_t* table, void* workspace,
                              size_t workspace_bytes, tasc_stream stream);

/* Synchronise the stream and return the device status word of the workspace (TASC_OK if clean); clears it. */
tasc_status tasc_poll_status(void* workspace, tasc_stream stream);

/*
 * Failure-path self-test.  Every device-side wait of the library (TMA arrival, MMA completion, ring slots) is
 * bounded: when the budget runs out the kernel records TASC_ETIMEOUT in the status word, gives up the wait and
 * returns normally, so the context stays usable.  This call launches a one-thread kernel that waits, through the
 * same routine, on a barrier that nothing will ever signal, for budget_cycles SM clock cycles (1 .. 2e9); a following
 * tasc_poll_status(workspace) must then report TASC_ETIMEOUT.  Nothing faults or hangs.
 *   workspace  device, at least 4 bytes: the status word
 * Asynchronous.  Errors: EINVAL.
 */
tasc_status tasc_selftest_bounded_wait(void* workspace, int64_t budget_cycles, tasc_stream stream);

/*
 * Y[M][N] (float32) = X[M][K] * W[N][K]^T for bf16 X and W on the tensor cores, the building block of
 * every projection of the verify forward (exported for unit tests and profiling).
 *   x, w       device, bf16, row-major, 16-byte aligned; K a multiple of 8
 *   y          device, float32[M][N]
 *   workspace  device, at least tasc_gemm_workspace_bytes(M, N, K) bytes (split-K partial sums)
 * Asynchronous.  Errors: EINVAL, ECUDA.
 */
tasc_status tasc_gemm_bf16(const void* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                           void* workspace, size_t workspace_bytes, tasc_stream stream);
/*
 * Same product for float32 X: every x is carried through the bf16 tensor cores as the pair
 * hi = bf16(x), lo = bf16(x - hi), and the two partial products are added in float32.  This is how
 * the verify forward feeds its activations to the projections, so that only the weights and the
 * KV cache are rounded to bf16.   x: device, float32[M][K].  Other arguments as tasc_gemm_bf16.
 */
tasc_status tasc_gemm_bf16x2(const float* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                             void* workspace, size_t workspace_bytes, tasc_stream stream);
size_t tasc_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K);

/*
 * The product of tasc_gemm_bf16 for callers that cannot allocate.  (The paper has no counterpart: this is
 * a service entry point of the library, not a step of the method.)
 *
 * Who needs it: code that runs where device memory can no longer be requested -- inside a serving process
 * whose memory pool was fixed at start-up, under a host that forbids cudaMalloc once initialisation is over,
 * or anywhere no allocator is at hand to provide the split-K workspace that tasc_gemm_bf16 demands.  Here
 * the partial sums go to a fixed 8 MiB device array that is part of the library image, so every GPU that
 * loads the library holds those 8 MiB until the process exits.  The call itself requests no memory of any
 * kind (no cudaMalloc / cudaFree, no allocating library routine); the caller passes inputs and output.
 * (If launch timing was switched on with tasc_profile_enable, the accounting creates CUDA events as usual.)
 *
 *   x, w, y, M, N, K   as tasc_gemm_bf16
 *   device_status      device, int32, or NULL: receives a device-side error code of this call (0 = none),
 *                      cleared at the start of the call.  With NULL the word lives inside the shared array
 *                      where no call can read it back: a device-side error (a bounded wait that ran out,
 *                      TASC_ETIMEOUT) then goes unreported and y holds zeros for the affected tiles -- pass
 *                      a status word if the result must be trusted.
 * Limits and rules:
 *   - the float32 partial sums (k-splits * M * N * 4 bytes) must fit in 8 MiB minus 256 bytes; the call takes
 *     fewer k-splits than tasc_gemm_bf16 if that makes them fit (only the summation order changes) and
 *     returns TASC_ECAPACITY when even one split does not (M * N * 4 > 8 MiB - 256);
 *   - the first call on each device looks up the array's device address (that device must be current, as
 *     for every call) -- make that first call before starting any stream capture;
 *   - all calls share the array and it keeps the previous call's contents; the kernel overwrites everything
 *     it later reads, so calls that follow each other on one stream are safe, but calls that overlap on the
 *     GPU (different streams or threads) race on it and corrupt each other's results.
 * Asynchronous on the stream.  Errors: EINVAL, ECAPACITY, ECUDA.
 */
tasc_status tasc_gemm_bf16_static(const void* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                                  int32_t* device_status, tasc_stream stream);

/*
 * Launch accounting.  Kernel launches are counted per kind for the life of the process
 * (tasc_launch_counts).  With timing enabled, every launch is additionally bracketed by CUDA events
 * on its own stream; tasc_profile_read synchronises the device, returns the summed milliseconds and
 * the number of timed launches per kind since the last read, and forgets them.  Timing adds event
 * records between kernels, so it belongs in a separate, untimed pass.
 *   arrays: host, n >= tasc_profile_kinds() elements.
 */
int32_t     tasc_profile_kinds(void);
const char* tasc_profile_kind_name(int32_t kind);
tasc_status tasc_profile_enable(int32_t on);
tasc_status tasc_profile_read(double* ms_by_kind, int64_t* timed_launches_by_kind, int32_t n);
tasc_status tasc_launch_counts(int64_t* launches_by_kind, int32_t n);

const char* tasc_status_string(tasc_status s);
/* Text of the most recent failing CUDA runtime call behind a TASC_ECUDA (name, message, source location), or "". */
const char* tasc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TASC_H */
