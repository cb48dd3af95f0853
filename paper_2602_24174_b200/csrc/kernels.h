// Internal launch interface between the C-ABI layer (api.cu) and the kernel files.
#pragma once

#include "common.cuh"

namespace tasc {

// ------------------------------------------------------------------ launch accounting (profile.cu)
enum Kind { K_DRAFT, K_ROWS, K_EMBED, K_GEMM, K_GEMM_LM, K_QKV_ROPE, K_ATT_SPLIT, K_ATT_COMBINE, K_RESNORM, K_SILU,
            K_ACCEPT, K_OTHER, K_COUNT };
void prof_begin(int kind, cudaStream_t s);     // counts the launch; records an event when timing is enabled
void prof_end(int kind, cudaStream_t s);
bool profiling_enabled();                      // per-launch event timing is on (tasc_profile_enable)
struct ProfScope {
    int kind; cudaStream_t s;
    ProfScope(int k, cudaStream_t st) : kind(k), s(st) { prof_begin(kind, s); }
    ~ProfScope() { prof_end(kind, s); }
};

// ------------------------------------------------------------------ tensor-core GEMM with split-K partial sums in global memory (gemm_tcgen05.cu)
// The exported building block tasc_gemm_bf16 / tasc_gemm_bf16_static; the forward uses gemm_fused.cu.
// Computes partial sums P[s][m][n] = sum over the k-range of split s of X[m][k] * W[n][k]
// (bf16 inputs, float32 accumulation in TMEM).  Consumers add the `splits` slices in order.
struct GemmPlan {
    int pair;        // 1: activations are (hi, lo) bf16 row pairs, see gemm_tcgen05.cu
    int TB;          // tokens per CTA tile, multiple of 16
    int BN;          // activation rows per CTA tile (UMMA N) = TB, or 2 * TB in paired mode; 16..256
    int m_tiles;     // ceil(M / TB)
    int out_tiles;   // ceil(N / 128): weight rows per CTA tile = UMMA M = 128
    int splits;      // split-K factor
    int stages;      // TMA -> MMA pipeline depth
    int smem_bytes;
};
GemmPlan plan_gemm(int M, int N, int K, size_t max_partial_bytes, bool pair);
// TB for M token rows.  few_tiles (1..3): how many token tiles 49..128 paired rows are cut into at least (see gemm_token_tile).
int gemm_token_tile(int M, bool pair, int few_tiles = 3, bool many_rows = false);
inline size_t gemm_partial_bytes(const GemmPlan& p, int M, int N) { return (size_t)p.splits * M * N * sizeof(float); }

// rows x cols bf16 row-major matrix, box = {64 cols, box_rows}, 128-byte swizzle.
tasc_status encode_tmap_bf16(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows);
// One layer's K (or V) pages seen as a rows x head_dim bf16 matrix (rows = pages * kv_heads * 16): box = one page of
// one KV head, {min(head_dim, 64) columns, 16 rows}, 128-byte swizzle (64-byte for head_dim 32).
tasc_status encode_tmap_kv(CUtensorMap* map, const void* ptr, uint64_t rows, int hd);

tasc_status launch_gemm_bf16(const CUtensorMap* tmW, const CUtensorMap* tmX, float* partials, int M, int N, int K,
                             const GemmPlan& plan, int* status, cudaStream_t stream);
tasc_status gemm_set_attributes();

// ------------------------------------------------------------------ fused projection GEMMs (gemm_fused.cu)
// What happens to the reduced output tile before anything is written to global memory.
enum Epi {
    EPI_PLAIN,    // y[m][f] = acc (times the row's RMS factor when ssq_in is given)
    EPI_QKV,      // acc * rms factor; RoPE on q and k heads; q -> qbuf, k and v -> KV pages
    EPI_RESID,    // x[m][f] += acc; a_out = (hi, lo) of x * gain; ssq_out[m][tile] = sum over the tile of x^2
    EPI_SWIGLU,   // tile = 64 gate rows + the 64 matching up rows; a_out = (hi, lo) of SiLU(gate) * up, both times the rms factor
    EPI_LM        // per token row an atomic max of (value, id) in argmax[m]; logits (nullable) get the scaled rows
};
struct FusedArgs {
    int M, N, K;                       // token rows, output features (EPI_SWIGLU: d_ff), reduction length
    int num_kb, BN, TB, TBL, stages, pair, data_bytes; // filled in by launch_gemm_fused from the plan
    int BNW, n_ft, n_tt;               // many-row kernel (gemm_wide.cu): features per MMA, feature tiles, token tiles
    int early;                         // the epilogue's global operands were complete before the preceding grid began
    const float* ssq_in;               // [M][ssq_slots] partial sums of squares of the input rows (null: no scaling)
    int ssq_slots;
    float inv_d, eps;                  // rms factor = 1 / sqrt(sum(ssq) * inv_d + eps)
    float* y;                          // EPI_PLAIN
    const int* row_pos;                // EPI_QKV: position of each row, -1 = unused
    const float2* rope;
    float* qbuf;
    __nv_bfloat16 *k_pages, *v_pages;
    const int32_t* block_table;
    int max_pages, page_size;
    long long n_pages;
    int R, n_q, n_kv, hd, max_positions;
    float* x;                          // EPI_RESID
    const float* gain;
    float* ssq_out;
    int ssq_out_slots;                 // slots per row; ssq_sub of them per 128 features (the many-row kernel writes one per 32 features)
    int ssq_sub;
    __nv_bfloat16* a_out;              // EPI_RESID / EPI_SWIGLU: activation buffer of the next GEMM, [tiles][2 TB][N]
    unsigned long long* argmax;        // EPI_LM
    float* logits;
    int* status;
};
struct FusedPlan {
    int TBL;           // tokens per tile of the activation layout
    int TB, BN, m_tiles, out_tiles, num_kb;   // TB: tokens per CTA (a multiple of TBL); BN = 2 TB; m_tiles: CTAs along the tokens
    int S;             // cluster size = k-splits
    int stages, data_bytes, smem_bytes;
    int wide;          // 1: the many-row kernel of gemm_wide.cu (M > 128) with BNW weight rows per MMA and `grid` persistent CTAs
    int BNW, grid;
    int threads;       // few-row kernel: 192, or 384 (six more warps that only finish columns) where a CTA finishes many token columns
};
// hd: head_dim, for EPI_QKV.  wide_min_mb: < 0 for a pass whose products all take the few-row kernel; otherwise the
// pass lays its activations out for the many-row kernel (gemm_token_tile with many_rows) and a product takes that
// kernel if its weight matrix has at least this many MB.
FusedPlan plan_fused(int M, int N, int K, int epi, int few_tiles = 3, int hd = 0, double wide_min_mb = -1.0);
// The many-row variant (gemm_wide.cu): fills `p` and returns true where it applies (M > 128, N a multiple of 32).
// token_tile > 0: the pass's token tile is given (its other products take the few-row kernel), any M.
bool plan_wide(int M, int N, int K, int epi, int hd, FusedPlan& p, int token_tile = 0);
tasc_status launch_gemm_wide(int epi, const CUtensorMap* tmW, const CUtensorMap* tmX, FusedArgs a, const FusedPlan& p,
                             cudaStream_t stream);
// tmW: weight map with box rows 128 (64 for EPI_SWIGLU); tmX: (hi, lo) activation map with box rows BN = 2 TB.
tasc_status launch_gemm_fused(int epi, const CUtensorMap* tmW, const CUtensorMap* tmX, FusedArgs a, const FusedPlan& p,
                              cudaStream_t stream);

// ------------------------------------------------------------------ float32 GEMM for the f32 model (gemm_simt.cu)
// Same contract with splits = 1: P[0][m][n].
void launch_gemm_f32(const float* X, const float* W, float* partials, int M, int N, int K,
                     unsigned long long* argmax, float* logits, cudaStream_t stream);

// ------------------------------------------------------------------ layer kernels (layers.cu)
struct RowPlan {              // per-step row bookkeeping, all device pointers into the workspace
    int* row_tok;             // [M] token id of each row
    int* row_pos;             // [M] position of each row, -1 = row not in use
    int* seq_pos0;            // [B] position of the sequence's first row
    int* seq_rows;            // [B] rows in use (0 = sequence skipped)
};
// Rows of a verify step: [last committed token, drafts] at positions len-1 ..; skipped when len >= stop_len.
void launch_rows_verify(const RowPlan& rp, const int32_t* tokens, int64_t stride, const int32_t* len,
                        const int32_t* stop_len, const int32_t* drafts, int B, int R, int vocab, int* status,
                        cudaStream_t stream);
// Rows of prefill chunk c: committed tokens c*R .. c*R+R-1, limited to positions <= len-2.
void launch_rows_prefill(const RowPlan& rp, const int32_t* tokens, int64_t stride, const int32_t* len, int B, int R,
                         int chunk, int vocab, int* status, cudaStream_t stream);

// float32 model: x[m] = embed[tok]; h[m] = RMSNorm(x[m]) * gain
template <typename T>
void launch_embed_norm(const T* embed, const int* row_tok, const float* gain, float eps, float* x, T* h, int M, int d,
                       int TB, cudaStream_t stream);
// bf16 model, first launch of a forward: row plan (chunk < 0: verify step, else prefill chunk) + embedding:
// x[m] = embed[tok]; a_out = (hi, lo) of x * gain; ssq[m][0] = sum x^2, other slots 0; argmax[m] = 0 (if given).
void launch_rows_embed(const RowPlan& rp, const int32_t* tokens, int64_t stride, const int32_t* len, const int32_t* stop_len,
                       const int32_t* drafts, int B, int R, int chunk, int vocab, int* status, const __nv_bfloat16* embed,
                       const float* gain, float* x, __nv_bfloat16* a_out, float* ssq, int ssq_slots, unsigned long long* argmax,
                       int d, int TB, cudaStream_t stream);
// x += sum_s P[s]; h = RMSNorm(x) * gain  (gain == null: only the residual update)
template <typename T>
void launch_residual_norm(const float* partials, int splits, float* x, const float* gain, float eps, T* h, int M, int d,
                          int TB, cudaStream_t stream);
// qkv = sum_s P[s]; RoPE on q and k; q -> qbuf [M][n_q*hd] (float32); k, v -> KV pages of the layer.
template <typename T>
void launch_qkv_rope_append(const float* partials, int splits, const RowPlan& rp, const float2* rope, float* qbuf,
                            T* k_pages, T* v_pages, const int32_t* block_table, int max_pages, int page_size,
                            long long n_pages, int M, int R, int n_q, int n_kv, int hd, int max_positions, int* status,
                            cudaStream_t stream);
// act = SiLU(gate) * up with gate = sum_s P[s][:, :dff], up = sum_s P[s][:, dff:]
template <typename T>
void launch_silu_mul(const float* partials, int splits, T* act, int M, int dff, int TB, cudaStream_t stream);
// float32 rows -> (hi, lo) bf16 row pairs in the tile-local layout of the paired GEMM
void launch_split_rows(const float* x, __nv_bfloat16* buf, int M, int K, int TB, cudaStream_t stream);
// y[M][N] = sum_s P[s]
void launch_sum_partials(const float* partials, int splits, float* y, size_t n, cudaStream_t stream);
void launch_fill_u64(unsigned long long* p, unsigned long long v, int n, cudaStream_t stream);
// Greedy acceptance, commit and bookkeeping (one thread per sequence).
void launch_accept(const unsigned long long* argmax, const RowPlan& rp, const int32_t* drafts,
                   const int32_t* forced_targets, int32_t* tokens, int64_t stride, int32_t* len, int B, int R,
                   int32_t* n_accepted, int32_t* next_token, int32_t* target_tokens, long long* hist,
                   cudaStream_t stream);
void launch_rope_table(float2* table, int max_positions, int hd, float base, cudaStream_t stream);
void launch_wait_selftest(long long budget_cycles, int* status, cudaStream_t stream);
// Teacher-forced targets built on the device from the drafts (see TASC_MODE_*).
void launch_forced_targets(int mode, const int32_t* drafts, const int32_t* continuation, int64_t cont_stride,
                           const int32_t* len, const int32_t* prompt_len, int forced_accept, int vocab, int B, int k,
                           int32_t* targets, cudaStream_t stream);
void launch_gather_output(const int32_t* tokens, int64_t stride, const int32_t* prompt_len, int B, int max_new,
                          int32_t* out, cudaStream_t stream);
void launch_min_generated(const int32_t* len, const int32_t* prompt_len, int B, int* out_min, cudaStream_t stream);
// Model-derived bigram table: B single-token sequences t0 .. t0 + B - 1, and table[t0 + b] = argmax of row b.
void launch_bigram_rows(int32_t* tokens, int32_t* len, int t0, int vocab, int B, cudaStream_t stream);
void launch_bigram_store(const unsigned long long* argmax, int32_t* table, int t0, int vocab, int B, cudaStream_t stream);

// ------------------------------------------------------------------ attention (attention.cu)
// Verify attention of R query rows per sequence over the paged KV cache (grouped-query, causal within the rows).
template <typename T>
void launch_attention(const float* qbuf, const T* k_pages, const T* v_pages, const int32_t* block_table, int max_pages,
                      int page_size, long long n_pages, const RowPlan& rp, T* out, int TB, float* scratch, int B, int R,
                      int n_q, int n_kv, int hd, int n_splits, cudaStream_t stream);
size_t attention_scratch_bytes(int B, int R, int n_q, int hd, int n_splits);
int attention_splits(int B, int n_kv, int max_ctx);


// ------------------------------------------------------------------ tensor-core attention for bf16 models (attention_mma.cu)
struct AttnPlan {
    int splits;      // key-range splits per (sequence, head group) = cluster size, 1..8
    int stages;      // depth of the K/V tile ring
    int heads;       // query heads per CTA: a divisor of n_q / n_kv (the heads sharing a KV head are dealt out to several CTAs)
};
// Same contract as launch_attention; the result goes to `out` as (hi, lo) bf16 rows; needs no scratch memory.
tasc_status launch_attention_mma(const float* qbuf, const __nv_bfloat16* k_pages, const __nv_bfloat16* v_pages,
                                 const int32_t* block_table, int max_pages, int page_size, long long n_pages,
                                 const RowPlan& rp, __nv_bfloat16* out, int TB, int B, int R, int n_q, int n_kv, int hd,
                                 const AttnPlan& plan, int* status, cudaStream_t stream);
// B sequences (or sequence blocks), g = n_q / n_kv query heads per KV head, `rows` query rows per sequence block
AttnPlan plan_attention_mma(int B, int n_kv, int hd, int g, int rows, int max_ctx);

}  // namespace tasc
