// C-ABI layer: model handle, workspace layout, the verify forward as a sequence of kernel launches,
// prefill, the speculative step and the generation loop.  Argument checking and launch order only;
// all arithmetic is in the kernel files.
#include "kernels.h"

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

// Launch shapes and activation tensor maps of one forward of a bf16 model, which depend only on the row counts, the
// cache capacity and the workspace address: planned once and reused by every later step on the same buffers.
struct StepPlans {
    int B, R, max_ctx;
    const void* ws_h;
    tasc::AttnPlan att;
    int TB;
    uint64_t rows;
    CUtensorMap tm_h, tm_o, tm_act, tm_h_lm;
    tasc::FusedPlan p_qkv, p_o, p_gu, p_down, p_lm;
};

struct tasc_model {
    tasc_model_desc desc;
    const void* embed;
    const void* lm_head;
    const float* final_norm;
    std::vector<const float*> attn_norm, mlp_norm;
    std::vector<const void*> wqkv, wo, w_gate_up, w_down;
    float2* rope;                                   // [max_positions][head_dim / 2] (cos, sin), library-owned
    // tensor maps of the weight matrices (bf16 models): box = 64 columns x 128 rows (gate/up: 64 rows, see EPI_SWIGLU)
    std::vector<CUtensorMap> tm_qkv, tm_o, tm_gu, tm_down;
    CUtensorMap tm_lm;
    int qkv_rows, q_dim, kv_dim;
    int few_tiles;                                  // token tiles for 49..128 rows (see gemm_token_tile), from the layer's weight bytes
    double layer_mb;                                // projection weights of one layer, MB
    mutable std::mutex plan_mu;
    mutable std::vector<StepPlans> plans;           // most recently used last; a handful of (B, k, workspace) combinations
};

namespace tasc {
namespace {

constexpr size_t ALIGN = 256;
constexpr size_t MIN_PARTIAL_BYTES = 64ull << 20;

struct Layout {
    size_t off = 0;
    template <typename U> U* take(uint8_t* base, size_t count) {
        U* p = reinterpret_cast<U*>(base + off);
        off += (count * sizeof(U) + ALIGN - 1) / ALIGN * ALIGN;
        return p;
    }
};

struct Workspace {
    int* status;
    long long* hist;              // [TASC_MAX_ROWS]
    int* min_gen;
    RowPlan rp;
    unsigned long long* argmax;   // [M]
    int32_t *drafts, *targets, *n_accepted, *next_token, *prompt_len, *stop_len;
    float* x;                     // [M][d] residual stream
    void *h, *o, *act;            // GEMM inputs: float rows, or (hi, lo) bf16 row pairs
    float* q;                     // [M][n_q * hd]
    float* partials;
    size_t partial_bytes;
    float* att_scratch;
    float* ssq;                   // [M][ceil(d / 128)] partial sums of squares of the residual rows (bf16 models)
    int ssq_slots;
    size_t bytes;
};

// Rows a pass may carry: TASC_MAX_ROWS per sequence for a verify step, and for bf16 models at least PREFILL_ROWS
// in all, so that a prefill of few sequences still runs passes of hundreds of rows (weights are read once per pass).
constexpr int PREFILL_ROWS = 2048;
constexpr int PREFILL_ROWS_PER_SEQ = 256;
size_t workspace_rows(const tasc_model* m, int B) {
    const size_t verify = (size_t)B * TASC_MAX_ROWS;
    return m->desc.dtype == TASC_F32 ? verify : std::max<size_t>(verify, PREFILL_ROWS);
}
// Rows per sequence of one prefill pass: a multiple of 16 that fits the workspace.
int prefill_rows(const tasc_model* m, int B) {
    if (m->desc.dtype == TASC_F32) return TASC_MAX_ROWS;
    const int per = (int)(workspace_rows(m, B) / (size_t)B) / 16 * 16;
    return std::max(TASC_MAX_ROWS, std::min(per, PREFILL_ROWS_PER_SEQ));
}

// The layout is always made for workspace_rows() rows so that every call agrees on it.
Workspace layout_workspace(const tasc_model* m, int B, void* base_) {
    const tasc_model_desc& d = m->desc;
    uint8_t* base = static_cast<uint8_t*>(base_);
    const size_t M = workspace_rows(m, B);
    const size_t esz = d.dtype == TASC_F32 ? 4 : 2;
    Layout L;
    Workspace w;
    w.status = L.take<int>(base, 64);
    w.hist = L.take<long long>(base, TASC_MAX_ROWS);
    w.min_gen = L.take<int>(base, 64);
    w.rp.row_tok = L.take<int>(base, M);
    w.rp.row_pos = L.take<int>(base, M);
    w.rp.seq_pos0 = L.take<int>(base, B);
    w.rp.seq_rows = L.take<int>(base, B);
    w.argmax = L.take<unsigned long long>(base, M);
    w.drafts = L.take<int32_t>(base, M);
    w.targets = L.take<int32_t>(base, M);
    w.n_accepted = L.take<int32_t>(base, B);
    w.next_token = L.take<int32_t>(base, B);
    w.prompt_len = L.take<int32_t>(base, B);
    w.stop_len = L.take<int32_t>(base, B);
    w.x = L.take<float>(base, M * d.d_model);
    // (hi, lo) rows of every token tile, each tile padded to a multiple of 16 tokens (at most max(3, M / 128 + 1) tiles)
    const size_t act_rows = d.dtype == TASC_F32 ? M : 2 * (M + 16 * (size_t)std::max<long long>(3, (long long)(M / 128 + 1)));
    w.h = L.take<uint8_t>(base, act_rows * d.d_model * esz);
    w.q = L.take<float>(base, M * m->q_dim);
    w.o = L.take<uint8_t>(base, act_rows * m->q_dim * esz);
    w.act = L.take<uint8_t>(base, act_rows * d.d_ff * esz);
    const size_t n_max = std::max<size_t>({(size_t)m->qkv_rows, (size_t)2 * d.d_ff, (size_t)d.d_model});
    // split-K partial sums in global memory are used by the float32 model only
    w.partial_bytes = d.dtype == TASC_F32 ? std::max(MIN_PARTIAL_BYTES, M * n_max * sizeof(float)) : ALIGN;
    w.partials = L.take<float>(base, w.partial_bytes / sizeof(float));
    const int splits_max = attention_splits(B, d.n_kv_heads, 1 << 30);
    // split partials in global memory are used by the float32 model only
    const size_t att_bytes = d.dtype == TASC_F32 ? attention_scratch_bytes(B, TASC_MAX_ROWS, d.n_q_heads, d.head_dim, splits_max) : ALIGN;
    w.att_scratch = L.take<float>(base, att_bytes / sizeof(float));
    w.ssq_slots = (d.d_model + 127) / 128;
    w.ssq = L.take<float>(base, M * w.ssq_slots * 4);      // passes of more than 128 rows keep four slots per 128 features
    w.bytes = L.off;
    return w;
}

__global__ void init_generate_kernel(const int32_t* len, int32_t* prompt_len, int32_t* stop_len, int B, int max_new) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    prompt_len[b] = len[b];
    stop_len[b] = len[b] + max_new;
}

struct KvView {
    void* k; void* v;
};
KvView layer_kv(const tasc_model* m, const tasc_kv* kv, int layer) {
    const tasc_model_desc& d = m->desc;
    const size_t esz = d.dtype == TASC_F32 ? 4 : 2;
    const size_t per = (size_t)kv->n_pages * d.n_kv_heads * d.page_size * d.head_dim * esz;
    uint8_t* base = static_cast<uint8_t*>(kv->pool) + (size_t)layer * 2 * per;
    return KvView{base, base + per};
}

// Where the rows of a forward come from: a verify step (chunk < 0: last committed token + drafts) or prefill chunk `chunk`.
// Which passes and products take the many-row kernel (gemm_wide.cu); see plan_fused.  Measured on the 135M, 0.5B and
// 1.5B shapes at 192 .. 1,024 rows: a product gains from it once its weight matrix has about 7 MB (gate/up, down and
// the LM head of the larger shapes; the narrow QKV and O matrices stay with the few-row kernel and its 128-row weight
// tiles), and a pass of 129 .. 255 rows only on layers of 60 MB and more (its two token tiles fill three quarters of
// the MMA's rows or less, and the few-row kernel then prefers three narrower tiles).
constexpr double WIDE_MATRIX_MB = 7.0;
constexpr double WIDE_LAYER_MB = 60.0;
constexpr int WIDE_ROWS = 256;

struct RowSource {
    const tasc_seqs* seqs;
    const int32_t* drafts;
    int chunk;
};

// float32 model (the tiny configuration): one launch per stage, float32 SIMT kernels.
tasc_status forward_f32(const tasc_model* m, const tasc_kv* kv, const Workspace& w, const RowSource& src, int B, int R, bool lm_head,
                        float* logits, cudaStream_t s) {
    const tasc_model_desc& d = m->desc;
    const int M = B * R;
    const tasc_seqs* sq = src.seqs;
    if (src.chunk < 0) launch_rows_verify(w.rp, sq->tokens, sq->stride, sq->len, sq->stop_len, src.drafts, B, R, d.vocab, w.status, s);
    else launch_rows_prefill(w.rp, sq->tokens, sq->stride, sq->len, B, R, src.chunk, d.vocab, w.status, s);
    const int max_ctx = kv->max_pages_per_seq * d.page_size;
    const int att_splits = attention_splits(B, d.n_kv_heads, max_ctx);
    float* h = static_cast<float*>(w.h);
    float* q = w.q;
    float* o = static_cast<float*>(w.o);
    float* act = static_cast<float*>(w.act);
    auto gemm = [&](const float* X, const void* W, int N, int K, unsigned long long* argmax, float* lg) {
        launch_gemm_f32(X, static_cast<const float*>(W), w.partials, M, N, K, argmax, lg, s);
    };
    launch_embed_norm<float>(static_cast<const float*>(m->embed), w.rp.row_tok, m->attn_norm[0], d.rms_eps, w.x, h, M, d.d_model, 0, s);
    for (int l = 0; l < d.n_layers; ++l) {
        const KvView kvl = layer_kv(m, kv, l);
        gemm(h, m->wqkv[l], m->qkv_rows, d.d_model, nullptr, nullptr);
        launch_qkv_rope_append<float>(w.partials, 1, w.rp, m->rope, q, static_cast<float*>(kvl.k), static_cast<float*>(kvl.v),
                                      kv->block_table, kv->max_pages_per_seq, d.page_size, kv->n_pages, M, R, d.n_q_heads,
                                      d.n_kv_heads, d.head_dim, d.max_positions, w.status, s);
        launch_attention<float>(q, static_cast<const float*>(kvl.k), static_cast<const float*>(kvl.v), kv->block_table,
                                kv->max_pages_per_seq, d.page_size, kv->n_pages, w.rp, o, 0, w.att_scratch, B, R, d.n_q_heads,
                                d.n_kv_heads, d.head_dim, att_splits, s);
        gemm(o, m->wo[l], d.d_model, m->q_dim, nullptr, nullptr);
        launch_residual_norm<float>(w.partials, 1, w.x, m->mlp_norm[l], d.rms_eps, h, M, d.d_model, 0, s);
        gemm(h, m->w_gate_up[l], 2 * d.d_ff, d.d_model, nullptr, nullptr);
        launch_silu_mul<float>(w.partials, 1, act, M, d.d_ff, 0, s);
        gemm(act, m->w_down[l], d.d_model, d.d_ff, nullptr, nullptr);
        const float* next_gain = l + 1 < d.n_layers ? m->attn_norm[l + 1] : m->final_norm;
        launch_residual_norm<float>(w.partials, 1, w.x, next_gain, d.rms_eps, h, M, d.d_model, 0, s);
    }
    if (lm_head) {
        launch_fill_u64(w.argmax, 0ull, M, s);
        gemm(h, m->lm_head, d.vocab, d.d_model, w.argmax, logits);
    }
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

// bf16 models: five launches per layer (QKV+RoPE+KV append, attention, O+residual, gate/up+SiLU*mul, down+residual),
// each with programmatic stream serialisation; see gemm_fused.cu and attention_mma.cu.
tasc_status forward_bf16(const tasc_model* m, const tasc_kv* kv, const Workspace& w, const RowSource& src, int B, int R,
                         bool lm_head, float* logits, cudaStream_t s) {
    const tasc_model_desc& d = m->desc;
    const int M = B * R;
    const int max_ctx = kv->max_pages_per_seq * d.page_size;
    tasc_status st;
    StepPlans sp;
    {
        std::lock_guard<std::mutex> lk(m->plan_mu);
        auto it = std::find_if(m->plans.begin(), m->plans.end(), [&](const StepPlans& c) {
            return c.B == B && c.R == R && c.max_ctx == max_ctx && c.ws_h == w.h; });
        if (it != m->plans.end()) {
            sp = *it;
        } else {
            sp.B = B; sp.R = R; sp.max_ctx = max_ctx; sp.ws_h = w.h;
            // attention works on blocks of at most 16 rows per sequence (one block in a verify step, several in a prefill pass)
            const int att_rows = R <= 16 ? R : 16;
            sp.att = plan_attention_mma(B * (R / att_rows), d.n_kv_heads, d.head_dim, d.n_q_heads / d.n_kv_heads, att_rows, max_ctx);
            // passes of more than 128 rows: the products with large weight matrices take the many-row kernel
            const double big_mb = 2.0 * 2.0 * (double)d.d_ff * d.d_model / 1e6;      // the largest matrix of a layer (gate/up)
            const bool wide_pass = M > 128 && big_mb >= WIDE_MATRIX_MB && (M >= WIDE_ROWS || m->layer_mb >= WIDE_LAYER_MB);
            const double wide_min_mb = wide_pass ? WIDE_MATRIX_MB : -1.0;
            sp.TB = gemm_token_tile(M, true, m->few_tiles, wide_min_mb >= 0.0);
            sp.rows = (uint64_t)((M + sp.TB - 1) / sp.TB) * 2 * sp.TB;
            if ((st = encode_tmap_bf16(&sp.tm_h, w.h, sp.rows, d.d_model, 2 * sp.TB)) != TASC_OK) return st;
            if ((st = encode_tmap_bf16(&sp.tm_o, w.o, sp.rows, m->q_dim, 2 * sp.TB)) != TASC_OK) return st;
            if ((st = encode_tmap_bf16(&sp.tm_act, w.act, sp.rows, d.d_ff, 2 * sp.TB)) != TASC_OK) return st;
            sp.p_qkv = plan_fused(M, m->qkv_rows, d.d_model, EPI_QKV, m->few_tiles, d.head_dim, wide_min_mb);
            sp.p_o = plan_fused(M, d.d_model, m->q_dim, EPI_RESID, m->few_tiles, 0, wide_min_mb);
            sp.p_gu = plan_fused(M, d.d_ff, d.d_model, EPI_SWIGLU, m->few_tiles, 0, wide_min_mb);
            sp.p_down = plan_fused(M, d.d_model, d.d_ff, EPI_RESID, m->few_tiles, 0, wide_min_mb);
            sp.p_lm = plan_fused(M, d.vocab, d.d_model, EPI_LM, m->few_tiles, 0, wide_min_mb);
            // the LM head's CTAs take several layout tiles at once
            if ((st = encode_tmap_bf16(&sp.tm_h_lm, w.h, sp.rows, d.d_model, sp.p_lm.BN)) != TASC_OK) return st;
            if (m->plans.size() >= 16) m->plans.erase(m->plans.begin());
            m->plans.push_back(sp);
        }
    }
    const AttnPlan& att_plan = sp.att;
    const int TB = sp.TB;
    const CUtensorMap &tm_h = sp.tm_h, &tm_o = sp.tm_o, &tm_act = sp.tm_act;
    const FusedPlan &p_qkv = sp.p_qkv, &p_o = sp.p_o, &p_gu = sp.p_gu, &p_down = sp.p_down;
    __nv_bfloat16* h = static_cast<__nv_bfloat16*>(w.h);
    __nv_bfloat16* o = static_cast<__nv_bfloat16*>(w.o);
    __nv_bfloat16* act = static_cast<__nv_bfloat16*>(w.act);

    FusedArgs base = {};
    base.M = M;
    const int ssq_sub = M > 128 ? 4 : 1;
    const int ssq_slots = w.ssq_slots * ssq_sub;
    base.ssq_slots = ssq_slots;
    base.ssq_sub = ssq_sub;
    base.inv_d = 1.0f / (float)d.d_model;
    base.eps = d.rms_eps;
    base.status = w.status;

    launch_rows_embed(w.rp, src.seqs->tokens, src.seqs->stride, src.seqs->len, src.seqs->stop_len, src.drafts, B, R, src.chunk,
                      d.vocab, w.status, static_cast<const __nv_bfloat16*>(m->embed), m->attn_norm[0], w.x, h, w.ssq, ssq_slots,
                      lm_head ? w.argmax : nullptr, d.d_model, TB, s);
    for (int l = 0; l < d.n_layers; ++l) {
        const KvView kvl = layer_kv(m, kv, l);
        FusedArgs a = base;
        a.N = m->qkv_rows; a.K = d.d_model; a.ssq_in = w.ssq;
        a.row_pos = w.rp.row_pos; a.rope = m->rope; a.qbuf = w.q;
        a.k_pages = static_cast<__nv_bfloat16*>(kvl.k); a.v_pages = static_cast<__nv_bfloat16*>(kvl.v);
        a.block_table = kv->block_table; a.max_pages = kv->max_pages_per_seq; a.page_size = d.page_size; a.n_pages = kv->n_pages;
        a.R = R; a.n_q = d.n_q_heads; a.n_kv = d.n_kv_heads; a.hd = d.head_dim; a.max_positions = d.max_positions;
        a.early = l > 0;               // layer 0 follows the kernel that writes the row plan
        if ((st = launch_gemm_fused(EPI_QKV, &m->tm_qkv[l], &tm_h, a, p_qkv, s)) != TASC_OK) return st;

        st = launch_attention_mma(w.q, static_cast<const __nv_bfloat16*>(kvl.k), static_cast<const __nv_bfloat16*>(kvl.v),
                                  kv->block_table, kv->max_pages_per_seq, d.page_size, kv->n_pages, w.rp, o, TB, B, R,
                                  d.n_q_heads, d.n_kv_heads, d.head_dim, att_plan, w.status, s);
        if (st != TASC_OK) return st;

        a = base;
        a.N = d.d_model; a.K = m->q_dim; a.x = w.x; a.gain = m->mlp_norm[l]; a.a_out = h; a.ssq_out = w.ssq; a.ssq_out_slots = ssq_slots;
        a.early = 1;                   // x was last written three launches back
        if ((st = launch_gemm_fused(EPI_RESID, &m->tm_o[l], &tm_o, a, p_o, s)) != TASC_OK) return st;

        a = base;
        a.N = d.d_ff; a.K = d.d_model; a.ssq_in = w.ssq; a.a_out = act;
        if ((st = launch_gemm_fused(EPI_SWIGLU, &m->tm_gu[l], &tm_h, a, p_gu, s)) != TASC_OK) return st;

        a = base;
        a.N = d.d_model; a.K = d.d_ff; a.x = w.x; a.gain = l + 1 < d.n_layers ? m->attn_norm[l + 1] : m->final_norm;
        a.a_out = h; a.ssq_out = w.ssq; a.ssq_out_slots = ssq_slots;
        a.early = 1;                   // x was last written two launches back
        if ((st = launch_gemm_fused(EPI_RESID, &m->tm_down[l], &tm_act, a, p_down, s)) != TASC_OK) return st;
    }
    if (lm_head) {
        const FusedPlan& p_lm = sp.p_lm;
        const CUtensorMap& tm_h_lm = sp.tm_h_lm;
        FusedArgs a = base;
        a.N = d.vocab; a.K = d.d_model; a.ssq_in = w.ssq; a.argmax = w.argmax; a.logits = logits;
        if ((st = launch_gemm_fused(EPI_LM, &m->tm_lm, &tm_h_lm, a, p_lm, s)) != TASC_OK) return st;
    }
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

tasc_status forward_any(const tasc_model* m, const tasc_kv* kv, const Workspace& w, const RowSource& src, int B, int R,
                        bool lm_head, float* logits, cudaStream_t s) {
    return m->desc.dtype == TASC_F32 ? forward_f32(m, kv, w, src, B, R, lm_head, logits, s)
                                     : forward_bf16(m, kv, w, src, B, R, lm_head, logits, s);
}

bool check_common(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, int B, void* ws, size_t ws_bytes) {
    if (!m || !kv || !seqs || !ws || B < 1) return false;
    if (!kv->pool || !kv->block_table || kv->n_pages < 1 || kv->max_pages_per_seq < 1) return false;
    if (!seqs->tokens || !seqs->len || seqs->stride < 1) return false;
    if (reinterpret_cast<uintptr_t>(ws) % ALIGN) return false;
    return ws_bytes >= layout_workspace(m, B, ws).bytes;
}

tasc_status verify_enqueue(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, const Workspace& w,
                           const int32_t* drafts, int B, int k, const int32_t* forced, int32_t* n_accepted,
                           int32_t* next_token, int32_t* target_tokens, float* logits, cudaStream_t s) {
    const int R = k + 1;
    tasc_status st = forward_any(m, kv, w, RowSource{seqs, drafts, -1}, B, R, true, logits, s);
    if (st != TASC_OK) return st;
    launch_accept(w.argmax, w.rp, drafts, forced, seqs->tokens, seqs->stride, seqs->len, B, R, n_accepted, next_token,
                  target_tokens, w.hist, s);
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

tasc_status prefill_enqueue(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, const Workspace& w, int B,
                            int max_len, cudaStream_t s) {
    const int R = prefill_rows(m, B);
    const int chunks = (std::max(max_len - 1, 0) + R - 1) / R;
    for (int c = 0; c < chunks; ++c) {
        tasc_status st = forward_any(m, kv, w, RowSource{seqs, nullptr, c}, B, R, false, nullptr, s);
        if (st != TASC_OK) return st;
    }
    return TASC_OK;
}

}  // namespace
}  // namespace tasc

using namespace tasc;

extern "C" tasc_status tasc_model_create(const tasc_model_desc* desc, const tasc_weights* wt, tasc_model** out) {
    if (!out) return TASC_EINVAL;
    *out = nullptr;
    if (!desc || !wt) return TASC_EINVAL;
    const tasc_model_desc& d = *desc;
    if (d.n_layers < 1 || d.d_model < 8 || d.n_q_heads < 1 || d.n_kv_heads < 1 || d.n_q_heads % d.n_kv_heads ||
        d.head_dim < 8 || d.head_dim > 256 || d.head_dim % 8 || d.d_ff < 8 || d.vocab < 2 ||
        d.vocab > (1 << TASC_VOCAB_BITS) || (d.dtype != TASC_F32 && d.dtype != TASC_BF16) || d.max_positions < 1 ||
        d.page_size < 1 || d.d_model % 8 || d.d_ff % 8 || !(d.rope_base > 0.f) || !(d.rms_eps >= 0.f))
        return TASC_EINVAL;
    if (!wt->embed || !wt->lm_head || !wt->final_norm || !wt->attn_norm || !wt->wqkv || !wt->wo || !wt->mlp_norm ||
        !wt->w_gate_up || !wt->w_down)
        return TASC_EINVAL;
    if (d.dtype == TASC_BF16) {
        // tensor-core attention: head_dim 32, 64 or 128 and at most 128 query rows per KV head in a prefill chunk
        if (d.head_dim != 32 && d.head_dim != 64 && d.head_dim != 128) return TASC_EINVAL;
        if ((d.n_q_heads / d.n_kv_heads) * TASC_MAX_ROWS > 128) return TASC_EINVAL;
    }
    tasc_model* m = new (std::nothrow) tasc_model();
    if (!m) return TASC_ENOMEM;
    m->desc = d;
    m->embed = wt->embed; m->lm_head = wt->lm_head; m->final_norm = wt->final_norm;
    m->q_dim = d.n_q_heads * d.head_dim;
    m->kv_dim = d.n_kv_heads * d.head_dim;
    m->qkv_rows = m->q_dim + 2 * m->kv_dim;
    {
        // every extra token tile streams the layer's weights once more (about 0.15 us per MB) and saves about 7 us of
        // exchange and epilogue time per layer: below 24 MB three tiles, below 60 MB two, above that one
        const double layer_mb = 2.0 * ((double)m->qkv_rows * d.d_model + (double)d.d_model * m->q_dim + 3.0 * d.d_ff * d.d_model) / 1e6;
        m->few_tiles = layer_mb < 24.0 ? 3 : (layer_mb < 60.0 ? 2 : 1);
        m->layer_mb = layer_mb;
    }
    m->rope = nullptr;
    for (int l = 0; l < d.n_layers; ++l) {
        if (!wt->attn_norm[l] || !wt->wqkv[l] || !wt->wo[l] || !wt->mlp_norm[l] || !wt->w_gate_up[l] || !wt->w_down[l]) {
            delete m;
            return TASC_EINVAL;
        }
        m->attn_norm.push_back(wt->attn_norm[l]); m->mlp_norm.push_back(wt->mlp_norm[l]);
        m->wqkv.push_back(wt->wqkv[l]); m->wo.push_back(wt->wo[l]);
        m->w_gate_up.push_back(wt->w_gate_up[l]); m->w_down.push_back(wt->w_down[l]);
    }
    tasc_status st = TASC_OK;
    if (d.dtype == TASC_BF16) {
        m->tm_qkv.resize(d.n_layers); m->tm_o.resize(d.n_layers); m->tm_gu.resize(d.n_layers); m->tm_down.resize(d.n_layers);
        st = gemm_set_attributes();
        for (int l = 0; l < d.n_layers && st == TASC_OK; ++l) {
            st = encode_tmap_bf16(&m->tm_qkv[l], m->wqkv[l], m->qkv_rows, d.d_model, 128);
            if (st == TASC_OK) st = encode_tmap_bf16(&m->tm_o[l], m->wo[l], d.d_model, m->q_dim, 128);
            if (st == TASC_OK) st = encode_tmap_bf16(&m->tm_gu[l], m->w_gate_up[l], 2 * (uint64_t)d.d_ff, d.d_model, 64);
            if (st == TASC_OK) st = encode_tmap_bf16(&m->tm_down[l], m->w_down[l], d.d_model, d.d_ff, 128);
        }
        if (st == TASC_OK) st = encode_tmap_bf16(&m->tm_lm, m->lm_head, d.vocab, d.d_model, 128);
    }
    if (st == TASC_OK) {
        const size_t n = (size_t)d.max_positions * (d.head_dim / 2);
        if (cudaMalloc(reinterpret_cast<void**>(&m->rope), n * sizeof(float2)) != cudaSuccess) {
            (void)cudaGetLastError();
            st = TASC_ENOMEM;
        } else {
            launch_rope_table(m->rope, d.max_positions, d.head_dim, d.rope_base, nullptr);
            if (cudaDeviceSynchronize() != cudaSuccess) { (void)cudaGetLastError(); st = TASC_ECUDA; }
        }
    }
    if (st != TASC_OK) {
        if (m->rope) cudaFree(m->rope);
        delete m;
        return st;
    }
    *out = m;
    return TASC_OK;
}

extern "C" tasc_status tasc_model_destroy(tasc_model* m) {
    if (!m) return TASC_EINVAL;
    if (m->rope) cudaFree(m->rope);
    delete m;
    return TASC_OK;
}

extern "C" size_t tasc_workspace_bytes(const tasc_model* m, int32_t B_max, int32_t k_max) {
    if (!m || B_max < 1 || k_max < 1 || k_max > TASC_MAX_ROWS - 1) return 0;
    return layout_workspace(m, B_max, nullptr).bytes;
}

extern "C" tasc_status tasc_prefill(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, int32_t B, int32_t max_len,
                                    void* workspace, size_t workspace_bytes, tasc_stream stream) {
    if (!check_common(m, kv, seqs, B, workspace, workspace_bytes) || max_len < 1 || max_len > seqs->stride) return TASC_EINVAL;
    const Workspace w = layout_workspace(m, B, workspace);
    return prefill_enqueue(m, kv, seqs, w, B, max_len, static_cast<cudaStream_t>(stream));
}

extern "C" tasc_status tasc_verify_step(const tasc_model* m, const tasc_kv* kv, const tasc_seqs* seqs, const int32_t* drafts,
                                        int32_t B, int32_t k, const int32_t* forced_targets, int32_t* n_accepted,
                                        int32_t* next_token, int32_t* target_tokens, float* logits_dbg, void* workspace,
                                        size_t workspace_bytes, tasc_stream stream) {
    if (!check_common(m, kv, seqs, B, workspace, workspace_bytes) || !drafts || !n_accepted || !next_token || k < 1 ||
        k > TASC_MAX_ROWS - 1)
        return TASC_EINVAL;
    const Workspace w = layout_workspace(m, B, workspace);
    return verify_enqueue(m, kv, seqs, w, drafts, B, k, forced_targets, n_accepted, next_token, target_tokens, logits_dbg,
                          static_cast<cudaStream_t>(stream));
}

extern "C" tasc_status tasc_generate(const tasc_model* m, const tasc_drafter* dr, const tasc_kv* kv, const tasc_seqs* seqs_in,
                                     int32_t B, int32_t max_new, const tasc_draft_params* p, int32_t* out, tasc_stats* stats,
                                     void* workspace, size_t workspace_bytes, tasc_stream stream) {
    if (!check_common(m, kv, seqs_in, B, workspace, workspace_bytes) || !dr || !p || !out || max_new < 1) return TASC_EINVAL;
    const int k = p->k;
    if (k < 1 || k > TASC_MAX_ROWS - 1) return TASC_EINVAL;
    if (p->mode < TASC_MODE_GREEDY || p->mode > TASC_MODE_FORCED_ACCEPT) return TASC_EINVAL;
    if (p->mode == TASC_MODE_CONTINUATION && (!p->continuation || p->continuation_stride < (int64_t)max_new + k + 1)) return TASC_EINVAL;
    if (p->mode == TASC_MODE_FORCED_ACCEPT && (p->forced_accept < 0 || p->forced_accept > k)) return TASC_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const Workspace w = layout_workspace(m, B, workspace);

    std::vector<int32_t> plen(B);
    TASC_CUDA_TRY(cudaMemcpyAsync(plen.data(), seqs_in->len, B * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    TASC_CUDA_TRY(cudaStreamSynchronize(s));
    int max_len = 0;
    for (int b = 0; b < B; ++b) {
        if (plen[b] < 1 || (int64_t)plen[b] + max_new + k > seqs_in->stride) return TASC_EINVAL;
        max_len = std::max(max_len, plen[b]);
    }
    init_generate_kernel<<<(B + 127) / 128, 128, 0, s>>>(seqs_in->len, w.prompt_len, w.stop_len, B, max_new);
    TASC_CUDA_TRY(cudaMemsetAsync(w.hist, 0, TASC_MAX_ROWS * sizeof(long long), s));
    tasc_seqs seqs = *seqs_in;
    seqs.stop_len = w.stop_len;

    cudaEvent_t ev[3];
    for (auto& e : ev) TASC_CUDA_TRY(cudaEventCreate(&e));
    tasc_status st = TASC_OK;
    cudaEventRecord(ev[0], s);
    st = prefill_enqueue(m, kv, &seqs, w, B, max_len, s);
    cudaEventRecord(ev[1], s);
    int64_t steps = 0;
    int min_gen = 0;
    const bool forced = p->mode != TASC_MODE_GREEDY;
    auto enqueue_step = [&]() -> tasc_status {
        tasc_status e = tasc_draft(dr, seqs.tokens, seqs.stride, seqs.len, B, k, p->lambda_num, p->lambda_den, w.drafts, s);
        if (e != TASC_OK) return e;
        if (forced)
            launch_forced_targets(p->mode, w.drafts, p->continuation, p->continuation_stride, seqs.len, w.prompt_len,
                                  p->forced_accept, m->desc.vocab, B, k, w.targets, s);
        return verify_enqueue(m, kv, &seqs, w, w.drafts, B, k, forced ? w.targets : nullptr, w.n_accepted, w.next_token,
                              nullptr, nullptr, s);
    };
    // Every step enqueues the same ~5 launches per layer on the same buffers, so after a first plain step the step
    // is captured once into a CUDA graph and replayed: the host then costs one launch per step instead of ~150.
    // (Not possible on the legacy default stream, and not while launch timing is on: then every step is enqueued.)
    cudaGraphExec_t step_graph = nullptr;
    auto capture_step = [&]() {
        if (s == nullptr || s == cudaStreamLegacy || profiling_enabled()) return;
        if (cudaStreamBeginCapture(s, cudaStreamCaptureModeRelaxed) != cudaSuccess) { (void)cudaGetLastError(); return; }
        const tasc_status e = enqueue_step();
        cudaGraph_t g = nullptr;
        if (cudaStreamEndCapture(s, &g) != cudaSuccess || e != TASC_OK || !g) { (void)cudaGetLastError(); if (g) cudaGraphDestroy(g); return; }
        if (cudaGraphInstantiate(&step_graph, g, 0) != cudaSuccess) { (void)cudaGetLastError(); step_graph = nullptr; }
        cudaGraphDestroy(g);
    };
    while (st == TASC_OK && min_gen < max_new) {
        const int todo = (max_new - min_gen + k) / (k + 1);      // the slowest sequence needs at least this many steps
        for (int i = 0; i < todo && st == TASC_OK; ++i) {
            if (steps == 1 && !step_graph) capture_step();       // step 0 ran plainly (first-use set-up happens outside a capture)
            if (step_graph && steps >= 1) {
                if (cudaGraphLaunch(step_graph, s) != cudaSuccess) { (void)cudaGetLastError(); st = TASC_ECUDA; }
            } else {
                st = enqueue_step();
            }
            ++steps;
        }
        if (st != TASC_OK) break;
        launch_min_generated(seqs.len, w.prompt_len, B, w.min_gen, s);
        if (cudaMemcpyAsync(&min_gen, w.min_gen, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess) { (void)cudaGetLastError(); st = TASC_ECUDA; break; }
        int dev_status = 0;
        if (cudaMemcpy(&dev_status, w.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { (void)cudaGetLastError(); st = TASC_ECUDA; break; }
        if (dev_status != 0) { st = dev_status; break; }
    }
    if (step_graph) cudaGraphExecDestroy(step_graph);
    cudaEventRecord(ev[2], s);
    if (st == TASC_OK) {
        launch_gather_output(seqs.tokens, seqs.stride, w.prompt_len, B, max_new, out, s);
        if (cudaStreamSynchronize(s) != cudaSuccess) { (void)cudaGetLastError(); st = TASC_ECUDA; }
    } else {
        cudaStreamSynchronize(s);
        (void)cudaGetLastError();
    }
    if (stats) {
        long long hist[TASC_MAX_ROWS] = {0};
        if (st == TASC_OK && cudaMemcpy(hist, w.hist, sizeof(hist), cudaMemcpyDeviceToHost) != cudaSuccess) { (void)cudaGetLastError(); st = TASC_ECUDA; }
        stats->steps = steps;
        stats->committed = 0;
        for (int a = 0; a < TASC_MAX_ROWS; ++a) { stats->accepted_hist[a] = hist[a]; stats->committed += hist[a] * (a + 1); }
        stats->prefill_ms = stats->decode_ms = 0.f;
        if (st == TASC_OK) {
            cudaEventElapsedTime(&stats->prefill_ms, ev[0], ev[1]);
            cudaEventElapsedTime(&stats->decode_ms, ev[1], ev[2]);
        }
    }
    for (auto& e : ev) cudaEventDestroy(e);
    return st;
}

extern "C" tasc_status tasc_bigram_table(const tasc_model* m, const tasc_kv* kv, int32_t B, int32_t* table, void* workspace,
                                         size_t workspace_bytes, tasc_stream stream) {
    if (!m || !kv || !table || !workspace || B < 1) return TASC_EINVAL;
    if (!kv->pool || !kv->block_table || kv->n_pages < 1 || kv->max_pages_per_seq < 1) return TASC_EINVAL;
    if (reinterpret_cast<uintptr_t>(workspace) % ALIGN || workspace_bytes < layout_workspace(m, B, workspace).bytes) return TASC_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const Workspace w = layout_workspace(m, B, workspace);
    const int V = m->desc.vocab;
    // B single-token sequences per pass: each row is the whole context of its sequence (position 0, its own key only)
    tasc_seqs seqs;
    seqs.tokens = w.targets; seqs.stride = 1; seqs.len = w.n_accepted; seqs.stop_len = nullptr;
    for (int t0 = 0; t0 < V; t0 += B) {
        launch_bigram_rows(w.targets, w.n_accepted, t0, V, B, s);
        tasc_status st = forward_any(m, kv, w, RowSource{&seqs, nullptr, -1}, B, 1, true, nullptr, s);
        if (st != TASC_OK) return st;
        launch_bigram_store(w.argmax, table, t0, V, B, s);
    }
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

extern "C" tasc_status tasc_poll_status(void* workspace, tasc_stream stream) {
    if (!workspace) return TASC_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int v = 0;
    TASC_CUDA_TRY(cudaStreamSynchronize(s));
    TASC_CUDA_TRY(cudaMemcpy(&v, workspace, sizeof(int), cudaMemcpyDeviceToHost));
    if (v != 0) TASC_CUDA_TRY(cudaMemset(workspace, 0, sizeof(int)));
    return v;
}

extern "C" tasc_status tasc_selftest_bounded_wait(void* workspace, int64_t budget_cycles, tasc_stream stream) {
    if (!workspace || budget_cycles < 1 || budget_cycles > 2000000000ll) return TASC_EINVAL;
    launch_wait_selftest(budget_cycles, static_cast<int*>(workspace), static_cast<cudaStream_t>(stream));
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

extern "C" size_t tasc_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K) {
    if (M < 1 || N < 1 || K < 1) return 0;
    const GemmPlan p = plan_gemm(M, N, K, (size_t)1 << 40, false);
    const GemmPlan p2 = plan_gemm(M, N, K, (size_t)1 << 40, true);
    const size_t split_rows = (size_t)p2.m_tiles * p2.BN * K * 2;      // (hi, lo) copy of X for tasc_gemm_bf16x2
    return 256 + std::max(gemm_partial_bytes(p, M, N), gemm_partial_bytes(p2, M, N)) + 256 + split_rows;
}

extern "C" tasc_status tasc_gemm_bf16(const void* x, const void* wt, float* y, int32_t M, int32_t N, int32_t K, void* workspace,
                                      size_t workspace_bytes, tasc_stream stream) {
    if (!x || !wt || !y || !workspace || M < 1 || N < 1 || K < 8 || K % 8) return TASC_EINVAL;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return TASC_EINVAL;
    const size_t need = tasc_gemm_workspace_bytes(M, N, K);
    if (workspace_bytes < need) return TASC_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const GemmPlan p = plan_gemm(M, N, K, (size_t)1 << 40, false);
    tasc_status st = gemm_set_attributes();
    if (st != TASC_OK) return st;
    CUtensorMap tmW, tmX;
    if ((st = encode_tmap_bf16(&tmW, wt, N, K, 128)) != TASC_OK) return st;
    if ((st = encode_tmap_bf16(&tmX, x, M, K, p.BN)) != TASC_OK) return st;
    int* status = static_cast<int*>(workspace);
    TASC_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int), s));          // a reused workspace must not report an old error
    float* partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + 256);
    if ((st = launch_gemm_bf16(&tmW, &tmX, partials, M, N, K, p, status, s)) != TASC_OK) return st;
    launch_sum_partials(partials, p.splits, y, (size_t)M * N, s);
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

extern "C" tasc_status tasc_gemm_bf16x2(const float* x, const void* wt, float* y, int32_t M, int32_t N, int32_t K,
                                        void* workspace, size_t workspace_bytes, tasc_stream stream) {
    if (!x || !wt || !y || !workspace || M < 1 || N < 1 || K < 8 || K % 8) return TASC_EINVAL;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return TASC_EINVAL;
    if (workspace_bytes < tasc_gemm_workspace_bytes(M, N, K)) return TASC_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the forward's kernel with the plain epilogue: split-K inside a cluster, no partial sums in global memory
    const FusedPlan p = plan_fused(M, N, K, EPI_PLAIN);
    int* status = static_cast<int*>(workspace);
    TASC_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int), s));
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(workspace) + 256);
    const uint64_t rows = (uint64_t)p.m_tiles * p.BN;
    TASC_CUDA_TRY(cudaMemsetAsync(xs, 0, rows * K * 2, s));
    launch_split_rows(x, xs, M, K, p.TBL, s);
    CUtensorMap tmW, tmX;
    tasc_status st;
    if ((st = encode_tmap_bf16(&tmW, wt, N, K, 128)) != TASC_OK) return st;
    if ((st = encode_tmap_bf16(&tmX, xs, rows, K, p.BN)) != TASC_OK) return st;
    FusedArgs a = {};
    a.M = M; a.N = N; a.K = K; a.y = y; a.status = status;
    if ((st = launch_gemm_fused(EPI_PLAIN, &tmW, &tmX, a, p, s)) != TASC_OK) return st;
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

extern "C" const char* tasc_status_string(tasc_status s) {
    switch (s) {
        case TASC_OK: return "ok";
        case TASC_EINVAL: return "invalid argument";
        case TASC_ENOMEM: return "out of memory";
        case TASC_ECUDA: return "CUDA call failed";
        case TASC_ECAPACITY: return "capacity exceeded";
        case TASC_ENOKV: return "KV position outside the block table";
        case TASC_ETIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}
