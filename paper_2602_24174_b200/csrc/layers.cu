// Row bookkeeping and the fused element-wise stages of the verify forward: embedding gather + RMSNorm,
// split-K reduction fused with (residual add + RMSNorm), (RoPE + KV page append), (SiLU * up), and the
// greedy acceptance / commit step.  All float math is float32; T is the model's storage type.
#include "kernels.h"

namespace tasc {

namespace {

__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nw; ++i) t += red[i];     // same order in every thread
    __syncthreads();
    return t;
}

__global__ void rows_verify_kernel(RowPlan rp, const int32_t* tokens, int64_t stride, const int32_t* len,
                                   const int32_t* stop_len, const int32_t* drafts, int B, int R, int vocab, int* status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * R) return;
    const int b = i / R, r = i % R;
    const int L = len[b];
    bool active = L >= 1 && L <= stride && !(stop_len && L >= stop_len[b]);
    if (L < 1 || L > stride) set_status(status, TASC_EINVAL);
    int tok = 0;
    if (active) {
        tok = r == 0 ? tokens[(int64_t)b * stride + L - 1] : drafts[b * (R - 1) + r - 1];
        if (tok < 0 || tok >= vocab) { set_status(status, TASC_EINVAL); tok = 0; }
    }
    rp.row_tok[i] = tok;
    rp.row_pos[i] = active ? L - 1 + r : -1;
    if (r == 0) {
        rp.seq_pos0[b] = active ? L - 1 : 0;
        rp.seq_rows[b] = active ? R : 0;
    }
}

__global__ void rows_prefill_kernel(RowPlan rp, const int32_t* tokens, int64_t stride, const int32_t* len, int B, int R,
                                    int chunk, int vocab, int* status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * R) return;
    const int b = i / R, r = i % R;
    const int L = len[b];
    if (L < 1 || L > stride) set_status(status, TASC_EINVAL);
    const int pos0 = chunk * R;
    int rows = L - 1 - pos0;
    rows = rows < 0 ? 0 : (rows > R ? R : rows);
    if (L < 1 || L > stride) rows = 0;
    int tok = 0;
    if (r < rows) {
        tok = tokens[(int64_t)b * stride + pos0 + r];
        if (tok < 0 || tok >= vocab) { set_status(status, TASC_EINVAL); tok = 0; }
    }
    rp.row_tok[i] = tok;
    rp.row_pos[i] = r < rows ? pos0 + r : -1;
    if (r == 0) {
        rp.seq_pos0[b] = pos0;
        rp.seq_rows[b] = rows;
    }
}

// x[m] = embed[tok]; h[m] = RMSNorm(x[m]) * gain
template <typename T>
__global__ void __launch_bounds__(128)
embed_norm_kernel(const T* __restrict__ embed, const int* __restrict__ row_tok, const float* __restrict__ gain, float eps,
                  float* __restrict__ x, T* __restrict__ h, int d, int TB) {
    __shared__ float red[4];
    const int m = blockIdx.x;
    const T* e = embed + (size_t)row_tok[m] * d;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = Num<T>::to_f(e[j]);
        x[(size_t)m * d + j] = v;
        ss += v * v;
    }
    const float inv = 1.0f / sqrtf(block_sum(ss, red) / (float)d + eps);
    for (int j = threadIdx.x; j < d; j += blockDim.x)
        ActStore<T>::put(h, m, j, d, TB, x[(size_t)m * d + j] * inv * gain[j]);
}

// bf16 model, first launch of a forward: the row plan of a verify step (chunk < 0: rows = [last committed token,
// drafts] at positions len-1 ..; skipped when len >= stop_len) or of prefill chunk `chunk` (committed tokens
// chunk*R .. limited to positions <= len-2), and the embedding of every row.  The RMS factor is applied by the
// consumer GEMM, so the row leaves here as x * gain (hi, lo) plus its sum of squares.
__global__ void __launch_bounds__(128)
rows_embed_kernel(RowPlan rp, const int32_t* __restrict__ tokens, int64_t stride, const int32_t* __restrict__ len,
                  const int32_t* __restrict__ stop_len, const int32_t* __restrict__ drafts, int R, int chunk, int vocab,
                  int* status, const __nv_bfloat16* __restrict__ embed, const float* __restrict__ gain, float* __restrict__ x,
                  __nv_bfloat16* __restrict__ a_out, float* __restrict__ ssq, int ssq_slots, unsigned long long* argmax, int d,
                  int TB) {
    __shared__ float red[4];
    __shared__ int s_tok;
    const int m = blockIdx.x;
    if (threadIdx.x == 0) {
        const int b = m / R, r = m % R;
        const int L = len[b];
        const bool len_ok = L >= 1 && L <= stride;
        if (!len_ok) set_status(status, TASC_EINVAL);
        int tok = 0, pos = -1, pos0 = 0, rows = 0;
        if (chunk < 0) {
            const bool active = len_ok && !(stop_len && L >= stop_len[b]);
            if (active) {
                tok = r == 0 ? tokens[(int64_t)b * stride + L - 1] : drafts[b * (R - 1) + r - 1];
                pos = L - 1 + r;
                pos0 = L - 1;
                rows = R;
            }
        } else {
            pos0 = chunk * R;
            rows = len_ok ? L - 1 - pos0 : 0;
            rows = rows < 0 ? 0 : (rows > R ? R : rows);
            if (r < rows) {
                tok = tokens[(int64_t)b * stride + pos0 + r];
                pos = pos0 + r;
            }
        }
        if (tok < 0 || tok >= vocab) { set_status(status, TASC_EINVAL); tok = 0; }
        rp.row_tok[m] = tok;
        rp.row_pos[m] = pos;
        if (r == 0) { rp.seq_pos0[b] = pos0; rp.seq_rows[b] = rows; }
        s_tok = tok;
    }
    __syncthreads();
    const __nv_bfloat16* e = embed + (size_t)s_tok * d;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = __bfloat162float(e[j]);
        x[(size_t)m * d + j] = v;
        ss += v * v;
        ActStore<__nv_bfloat16>::put(a_out, m, j, d, TB, v * gain[j]);
    }
    ss = block_sum(ss, red);
    for (int j = threadIdx.x; j < ssq_slots; j += blockDim.x) ssq[(size_t)m * ssq_slots + j] = j == 0 ? ss : 0.f;
    if (threadIdx.x == 0 && argmax) argmax[m] = 0ull;
}

// x[m] += sum_s P[s][m]; h[m] = RMSNorm(x[m]) * gain
template <typename T>
__global__ void __launch_bounds__(128)
residual_norm_kernel(const float* __restrict__ P, int splits, float* __restrict__ x, const float* __restrict__ gain,
                     float eps, T* __restrict__ h, int M, int d, int TB) {
    __shared__ float red[4];
    const int m = blockIdx.x;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        float v = x[(size_t)m * d + j];
        for (int s = 0; s < splits; ++s) v += P[((size_t)s * M + m) * d + j];
        x[(size_t)m * d + j] = v;
        ss += v * v;
    }
    if (!gain) return;
    const float inv = 1.0f / sqrtf(block_sum(ss, red) / (float)d + eps);
    for (int j = threadIdx.x; j < d; j += blockDim.x)
        ActStore<T>::put(h, m, j, d, TB, x[(size_t)m * d + j] * inv * gain[j]);
}

template <typename T>
__global__ void __launch_bounds__(128)
qkv_rope_append_kernel(const float* __restrict__ P, int splits, RowPlan rp, const float2* __restrict__ rope,
                       float* __restrict__ qbuf, T* __restrict__ k_pages, T* __restrict__ v_pages,
                       const int32_t* __restrict__ block_table, int max_pages, int page_size, long long n_pages,
                       int M, int R, int n_q, int n_kv, int hd, int max_positions, int* status) {
    const int m = blockIdx.x;
    const int pos = rp.row_pos[m];
    const int half = hd >> 1;
    const int qd = n_q * hd, kvd = n_kv * hd, N = qd + 2 * kvd;
    const int b = m / R;
    if (pos < 0) {
        for (int j = threadIdx.x; j < qd; j += blockDim.x) qbuf[(size_t)m * qd + j] = 0.f;
        return;
    }
    bool kv_ok = true;
    if (pos >= max_positions) { set_status(status, TASC_EINVAL); return; }
    const int pslot = pos / page_size;
    int page = 0;
    if (pslot >= max_pages) { set_status(status, TASC_ENOKV); kv_ok = false; }
    else {
        page = block_table[(size_t)b * max_pages + pslot];
        if (page < 0 || page >= n_pages) { set_status(status, TASC_ENOKV); kv_ok = false; }
    }
    const int slot = pos % page_size;
    const float2* cs = rope + (size_t)pos * half;
    auto acc = [&](int col) {
        float v = 0.f;
        for (int s = 0; s < splits; ++s) v += P[((size_t)s * M + m) * N + col];
        return v;
    };
    // q and k heads: rotate pairs (i, i + half)
    const int n_rot = (n_q + n_kv) * half;
    for (int t = threadIdx.x; t < n_rot; t += blockDim.x) {
        const int head = t / half, i = t % half;
        const float a = acc(head * hd + i), bb = acc(head * hd + i + half);
        const float2 c = cs[i];
        const float ra = a * c.x - bb * c.y, rb = bb * c.x + a * c.y;
        if (head < n_q) {
            qbuf[(size_t)m * qd + head * hd + i] = ra;
            qbuf[(size_t)m * qd + head * hd + i + half] = rb;
        } else if (kv_ok) {
            const int kh = head - n_q;
            T* dst = k_pages + (((size_t)page * n_kv + kh) * page_size + slot) * hd;
            dst[i] = Num<T>::from_f(ra);
            dst[i + half] = Num<T>::from_f(rb);
        }
    }
    if (kv_ok) {
        for (int t = threadIdx.x; t < kvd; t += blockDim.x) {
            const int kh = t / hd, i = t % hd;
            v_pages[(((size_t)page * n_kv + kh) * page_size + slot) * hd + i] = Num<T>::from_f(acc(qd + kvd + t));
        }
    }
}

template <typename T>
__global__ void silu_mul_kernel(const float* __restrict__ P, int splits, T* __restrict__ act, int M, int dff, int TB) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)M * dff) return;
    const int m = (int)(i / dff), j = (int)(i % dff);
    float g = 0.f, u = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float* row = P + ((size_t)s * M + m) * (2 * (size_t)dff);
        g += row[j];
        u += row[dff + j];
    }
    ActStore<T>::put(act, m, j, dff, TB, g / (1.0f + expf(-g)) * u);
}

__global__ void sum_partials_kernel(const float* __restrict__ P, int splits, float* __restrict__ y, size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float v = 0.f;
    for (int s = 0; s < splits; ++s) v += P[(size_t)s * n + i];
    y[i] = v;
}

__global__ void split_rows_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ buf, int M, int K, int TB) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)M * K) return;
    ActStore<__nv_bfloat16>::put(buf, (int)(i / K), (int)(i % K), K, TB, x[i]);
}

__global__ void fill_u64_kernel(unsigned long long* p, unsigned long long v, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

__global__ void accept_kernel(const unsigned long long* __restrict__ argmax, RowPlan rp, const int32_t* __restrict__ drafts,
                              const int32_t* __restrict__ forced, int32_t* tokens, int64_t stride, int32_t* len, int B, int R,
                              int32_t* n_accepted, int32_t* next_token, int32_t* target_tokens, long long* hist) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int k = R - 1;
    if (target_tokens)
        for (int i = 0; i < R; ++i) target_tokens[b * R + i] = (int32_t)packed_id(argmax[b * R + i]);
    if (rp.seq_rows[b] == 0) {
        n_accepted[b] = 0;
        next_token[b] = -1;
        return;
    }
    auto target = [&](int i) { return forced ? forced[b * R + i] : (int32_t)packed_id(argmax[b * R + i]); };
    int a = 0;
    while (a < k && drafts[b * k + a] == target(a)) ++a;
    const int nxt = target(a);
    const int L = len[b];
    int32_t* row = tokens + (int64_t)b * stride;
    int w = 0;
    for (; w < a && L + w < stride; ++w) row[L + w] = drafts[b * k + w];
    if (L + a < stride) { row[L + a] = nxt; w = a + 1; }
    len[b] = L + w;            // w = a + 1 unless the token buffer is full
    n_accepted[b] = a;
    next_token[b] = nxt;
    if (hist) atomicAdd(reinterpret_cast<unsigned long long*>(hist + a), 1ull);
}

// Self-test of the bounded wait that every barrier wait of the tensor-core kernels goes through: waits on an
// mbarrier that nothing will ever arrive at, for `budget` clock cycles, and records the outcome.
__global__ void wait_selftest_kernel(long long budget, int* status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
        if (!mbar_wait(smem_u32(&bar), 0, budget)) set_status(status, TASC_ETIMEOUT);
        mbar_inval(smem_u32(&bar));
    }
}

__global__ void rope_table_kernel(float2* table, int max_positions, int hd, float base) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int half = hd >> 1;
    if (i >= max_positions * half) return;
    const int pos = i / half, j = i % half;
    const double inv = pow((double)base, -2.0 * (double)j / (double)hd);
    const double ang = (double)pos * inv;
    table[i] = make_float2((float)cos(ang), (float)sin(ang));
}

__global__ void forced_targets_kernel(int mode, const int32_t* drafts, const int32_t* continuation, int64_t cont_stride,
                                      const int32_t* len, const int32_t* prompt_len, int forced_accept, int vocab, int B,
                                      int k, int32_t* targets) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= B * (k + 1)) return;
    const int b = t / (k + 1), i = t % (k + 1);
    int v;
    if (mode == TASC_MODE_CONTINUATION) {
        int64_t g = (int64_t)len[b] - prompt_len[b] + i;
        if (g < 0) g = 0;
        if (g >= cont_stride) g = cont_stride - 1;
        v = continuation[(int64_t)b * cont_stride + g];
    } else {
        v = i < forced_accept ? drafts[b * k + i] : (drafts[b * k + (i < k ? i : k - 1)] + 1) % vocab;
    }
    targets[t] = v;
}

// Single-token contexts t0, t0 + 1, ... as B sequences of length one (ids past the vocabulary repeat the last token).
__global__ void bigram_rows_kernel(int32_t* tokens, int32_t* len, int t0, int vocab, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    tokens[b] = min(t0 + b, vocab - 1);
    len[b] = 1;
}
__global__ void bigram_store_kernel(const unsigned long long* __restrict__ argmax, int32_t* table, int t0, int vocab, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B || t0 + b >= vocab) return;
    table[t0 + b] = (int32_t)packed_id(argmax[b]);
}

__global__ void gather_output_kernel(const int32_t* tokens, int64_t stride, const int32_t* prompt_len, int B, int max_new,
                                     int32_t* out) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= B * max_new) return;
    const int b = t / max_new, j = t % max_new;
    out[t] = tokens[(int64_t)b * stride + prompt_len[b] + j];
}

__global__ void min_generated_kernel(const int32_t* len, const int32_t* prompt_len, int B, int* out_min) {
    __shared__ int s;
    if (threadIdx.x == 0) s = 0x7FFFFFFF;
    __syncthreads();
    int v = 0x7FFFFFFF;
    for (int b = threadIdx.x; b < B; b += blockDim.x) v = min(v, len[b] - prompt_len[b]);
    atomicMin(&s, v);
    __syncthreads();
    if (threadIdx.x == 0) *out_min = s;
}

}  // namespace

void launch_rows_verify(const RowPlan& rp, const int32_t* tokens, int64_t stride, const int32_t* len,
                        const int32_t* stop_len, const int32_t* drafts, int B, int R, int vocab, int* status,
                        cudaStream_t stream) {
    ProfScope ps(K_ROWS, stream);
    rows_verify_kernel<<<(B * R + 127) / 128, 128, 0, stream>>>(rp, tokens, stride, len, stop_len, drafts, B, R, vocab, status);
}
void launch_rows_prefill(const RowPlan& rp, const int32_t* tokens, int64_t stride, const int32_t* len, int B, int R,
                         int chunk, int vocab, int* status, cudaStream_t stream) {
    ProfScope ps(K_ROWS, stream);
    rows_prefill_kernel<<<(B * R + 127) / 128, 128, 0, stream>>>(rp, tokens, stride, len, B, R, chunk, vocab, status);
}
template <typename T>
void launch_embed_norm(const T* embed, const int* row_tok, const float* gain, float eps, float* x, T* h, int M, int d,
                       int TB, cudaStream_t stream) {
    ProfScope ps(K_EMBED, stream);
    embed_norm_kernel<T><<<M, 128, 0, stream>>>(embed, row_tok, gain, eps, x, h, d, TB);
}
void launch_rows_embed(const RowPlan& rp, const int32_t* tokens, int64_t stride, const int32_t* len, const int32_t* stop_len,
                       const int32_t* drafts, int B, int R, int chunk, int vocab, int* status, const __nv_bfloat16* embed,
                       const float* gain, float* x, __nv_bfloat16* a_out, float* ssq, int ssq_slots, unsigned long long* argmax,
                       int d, int TB, cudaStream_t stream) {
    ProfScope ps(K_EMBED, stream);
    rows_embed_kernel<<<B * R, 128, 0, stream>>>(rp, tokens, stride, len, stop_len, drafts, R, chunk, vocab, status, embed, gain,
                                                 x, a_out, ssq, ssq_slots, argmax, d, TB);
}
template <typename T>
void launch_residual_norm(const float* partials, int splits, float* x, const float* gain, float eps, T* h, int M, int d,
                          int TB, cudaStream_t stream) {
    ProfScope ps(K_RESNORM, stream);
    residual_norm_kernel<T><<<M, 128, 0, stream>>>(partials, splits, x, gain, eps, h, M, d, TB);
}
template <typename T>
void launch_qkv_rope_append(const float* partials, int splits, const RowPlan& rp, const float2* rope, float* qbuf,
                            T* k_pages, T* v_pages, const int32_t* block_table, int max_pages, int page_size,
                            long long n_pages, int M, int R, int n_q, int n_kv, int hd, int max_positions, int* status,
                            cudaStream_t stream) {
    ProfScope ps(K_QKV_ROPE, stream);
    qkv_rope_append_kernel<T><<<M, 128, 0, stream>>>(partials, splits, rp, rope, qbuf, k_pages, v_pages, block_table,
                                                     max_pages, page_size, n_pages, M, R, n_q, n_kv, hd, max_positions, status);
}
template <typename T>
void launch_silu_mul(const float* partials, int splits, T* act, int M, int dff, int TB, cudaStream_t stream) {
    ProfScope ps(K_SILU, stream);
    const size_t n = (size_t)M * dff;
    silu_mul_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(partials, splits, act, M, dff, TB);
}
void launch_sum_partials(const float* partials, int splits, float* y, size_t n, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    sum_partials_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(partials, splits, y, n);
}
void launch_split_rows(const float* x, __nv_bfloat16* buf, int M, int K, int TB, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    const size_t n = (size_t)M * K;
    split_rows_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(x, buf, M, K, TB);
}
void launch_fill_u64(unsigned long long* p, unsigned long long v, int n, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    fill_u64_kernel<<<(n + 255) / 256, 256, 0, stream>>>(p, v, n);
}
void launch_accept(const unsigned long long* argmax, const RowPlan& rp, const int32_t* drafts,
                   const int32_t* forced_targets, int32_t* tokens, int64_t stride, int32_t* len, int B, int R,
                   int32_t* n_accepted, int32_t* next_token, int32_t* target_tokens, long long* hist,
                   cudaStream_t stream) {
    ProfScope ps(K_ACCEPT, stream);
    accept_kernel<<<(B + 63) / 64, 64, 0, stream>>>(argmax, rp, drafts, forced_targets, tokens, stride, len, B, R,
                                                    n_accepted, next_token, target_tokens, hist);
}
void launch_wait_selftest(long long budget_cycles, int* status, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    wait_selftest_kernel<<<1, 32, 0, stream>>>(budget_cycles, status);
}
void launch_rope_table(float2* table, int max_positions, int hd, float base, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    const int n = max_positions * (hd / 2);
    rope_table_kernel<<<(n + 255) / 256, 256, 0, stream>>>(table, max_positions, hd, base);
}
void launch_forced_targets(int mode, const int32_t* drafts, const int32_t* continuation, int64_t cont_stride,
                           const int32_t* len, const int32_t* prompt_len, int forced_accept, int vocab, int B, int k,
                           int32_t* targets, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    const int n = B * (k + 1);
    forced_targets_kernel<<<(n + 127) / 128, 128, 0, stream>>>(mode, drafts, continuation, cont_stride, len, prompt_len,
                                                               forced_accept, vocab, B, k, targets);
}
void launch_gather_output(const int32_t* tokens, int64_t stride, const int32_t* prompt_len, int B, int max_new,
                          int32_t* out, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    const int n = B * max_new;
    gather_output_kernel<<<(n + 255) / 256, 256, 0, stream>>>(tokens, stride, prompt_len, B, max_new, out);
}
void launch_bigram_rows(int32_t* tokens, int32_t* len, int t0, int vocab, int B, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    bigram_rows_kernel<<<(B + 127) / 128, 128, 0, stream>>>(tokens, len, t0, vocab, B);
}
void launch_bigram_store(const unsigned long long* argmax, int32_t* table, int t0, int vocab, int B, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    bigram_store_kernel<<<(B + 127) / 128, 128, 0, stream>>>(argmax, table, t0, vocab, B);
}
void launch_min_generated(const int32_t* len, const int32_t* prompt_len, int B, int* out_min, cudaStream_t stream) {
    ProfScope ps(K_OTHER, stream);
    min_generated_kernel<<<1, 128, 0, stream>>>(len, prompt_len, B, out_min);
}

#define TASC_INSTANTIATE(T)                                                                                              \
    template void launch_embed_norm<T>(const T*, const int*, const float*, float, float*, T*, int, int, int,             \
                                       cudaStream_t);                                                                    \
    template void launch_residual_norm<T>(const float*, int, float*, const float*, float, T*, int, int, int,             \
                                          cudaStream_t);                                                                 \
    template void launch_qkv_rope_append<T>(const float*, int, const RowPlan&, const float2*, float*, T*, T*,            \
                                            const int32_t*, int, int, long long, int, int, int, int, int, int, int*,     \
                                            cudaStream_t);                                                               \
    template void launch_silu_mul<T>(const float*, int, T*, int, int, int, cudaStream_t);
TASC_INSTANTIATE(float)

}  // namespace tasc
