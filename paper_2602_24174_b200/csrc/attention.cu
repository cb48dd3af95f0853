// Verify attention: the R = k+1 new query rows of every sequence against its paged KV cache.
// Grouped-query: the g = n_q / n_kv query heads that share a KV head are processed together, so each
// K/V element read from HBM serves g * R query rows.  The key range of a sequence is split over
// several CTAs (the batch alone cannot fill 148 SMs); each CTA keeps an online softmax per row and
// a second kernel merges the splits.  Row r of a sequence sees keys 0 .. pos0 + r.
//
// This kernel stages K/V tiles of 32 keys in shared memory (16-byte vector loads from the pages),
// computes scores with one warp per query row (lanes = keys) and accumulates P*V with lanes = head
// dimensions.  Math is float32.
#include "kernels.h"

namespace tasc {

namespace {

constexpr int TK = 32;            // keys per tile
constexpr int ATT_THREADS = 128;

template <typename T> struct Vec16;   // 16-byte vector access
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void load16_to_float(const T* src, float* dst) {
    const uint4 v = *reinterpret_cast<const uint4*>(src);
    if constexpr (sizeof(T) == 4) {
        dst[0] = __uint_as_float(v.x); dst[1] = __uint_as_float(v.y);
        dst[2] = __uint_as_float(v.z); dst[3] = __uint_as_float(v.w);
    } else {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            dst[2 * i] = __uint_as_float(w[i] << 16);
            dst[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

struct AttArgs {
    const void* q; const void* kp; const void* vp;
    const int32_t* block_table;
    int max_pages, page_size;
    long long n_pages;
    RowPlan rp;
    float* o_part;      // [B][n_q][R][splits][hd]
    float2* ml_part;    // [B][n_q][R][splits]
    int B, R, n_q, n_kv, hd, splits;
    float scale;
};

template <typename T>
__global__ void __launch_bounds__(ATT_THREADS)
attention_split_kernel(const AttArgs a) {
    extern __shared__ float sm[];
    const int sp = blockIdx.x, kh = blockIdx.y, b = blockIdx.z;
    const int rows = a.rp.seq_rows[b];
    const int pos0 = a.rp.seq_pos0[b];
    const int g = a.n_q / a.n_kv, hd = a.hd;
    const int G = g * a.R;                         // row slot index r = hl * R + rr
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ldk = hd + 1;
    float* Qs = sm;                                // [G][hd]
    float* Os = Qs + (size_t)G * hd;               // [G][hd]
    float* Ks = Os + (size_t)G * hd;               // [TK][hd + 1]
    float* Vs = Ks + (size_t)TK * ldk;             // [TK][hd]
    float* ms = Vs + (size_t)TK * hd;              // [G]
    float* ls = ms + G;                            // [G]

    const int total = pos0 + rows;                 // keys visible to the last row
    int chunk = (total + a.splits - 1) / a.splits;
    chunk = (chunk + TK - 1) / TK * TK;
    const int k_begin = sp * chunk;
    const int k_end = min(total, k_begin + chunk);

    const float* q = static_cast<const float*>(a.q);
    const int qd = a.n_q * hd;
    for (int i = threadIdx.x; i < G * hd; i += ATT_THREADS) {
        const int r = i / hd, d = i % hd;
        const int hl = r / a.R, rr = r % a.R;
        float v = 0.f;
        if (rr < rows) v = q[(size_t)(b * a.R + rr) * qd + (kh * g + hl) * hd + d] * a.scale;
        Qs[i] = v;
        Os[i] = 0.f;
    }
    for (int i = threadIdx.x; i < G; i += ATT_THREADS) { ms[i] = -INFINITY; ls[i] = 0.f; }
    __syncthreads();

    const T* kp = static_cast<const T*>(a.kp);
    const T* vp = static_cast<const T*>(a.vp);
    constexpr int VN = Vec16<T>::N;
    const int vec_per_row = hd / VN;

    for (int k0 = k_begin; k0 < k_end; k0 += TK) {
        // stage K and V rows k0 .. k0+TK-1 (zero beyond k_end)
        for (int i = threadIdx.x; i < TK * vec_per_row; i += ATT_THREADS) {
            const int j = i / vec_per_row, c = (i % vec_per_row) * VN;
            const int key = k0 + j;
            float kv[VN], vv[VN];
            int page = -1;
            if (key < k_end && key / a.page_size < a.max_pages)
                page = a.block_table[(size_t)b * a.max_pages + key / a.page_size];
            if (page >= 0 && page < a.n_pages) {      // ids outside the pool read as zeros, never as memory
                const size_t off = (((size_t)page * a.n_kv + kh) * a.page_size + key % a.page_size) * hd + c;
                load16_to_float<T>(kp + off, kv);
                load16_to_float<T>(vp + off, vv);
            } else {
#pragma unroll
                for (int e = 0; e < VN; ++e) { kv[e] = 0.f; vv[e] = 0.f; }
            }
#pragma unroll
            for (int e = 0; e < VN; ++e) { Ks[j * ldk + c + e] = kv[e]; Vs[j * hd + c + e] = vv[e]; }
        }
        __syncthreads();
        for (int r = warp; r < G; r += ATT_THREADS / 32) {
            const int rr = r % a.R;
            if (rr >= rows) continue;
            const int key = k0 + lane;
            const float* qr = Qs + (size_t)r * hd;
            const float* kr = Ks + lane * ldk;
            float s = 0.f;
            for (int d = 0; d < hd; ++d) s = fmaf(qr[d], kr[d], s);
            const bool vis = key < k_end && key <= pos0 + rr;
            s = vis ? s : -INFINITY;
            const float m_old = ms[r];
            const float m_new = fmaxf(m_old, warp_max(s));
            if (m_new == -INFINITY) continue;          // nothing visible yet for this row
            const float p = vis ? expf(s - m_new) : 0.f;
            const float alpha = expf(m_old - m_new);  // 0 when m_old = -inf
            const float psum = warp_sum(p);
            float* orow = Os + (size_t)r * hd;
            for (int d = lane; d < hd; d += 32) {
                float acc = orow[d] * alpha;
#pragma unroll 8
                for (int j = 0; j < TK; ++j) acc = fmaf(__shfl_sync(0xFFFFFFFFu, p, j), Vs[j * hd + d], acc);
                orow[d] = acc;
            }
            if (lane == 0) { ms[r] = m_new; ls[r] = ls[r] * alpha + psum; }
        }
        __syncthreads();
    }
    // write this split's partial result
    for (int i = threadIdx.x; i < G * hd; i += ATT_THREADS) {
        const int r = i / hd, d = i % hd;
        const int hl = r / a.R, rr = r % a.R;
        const size_t slot = (((size_t)b * a.n_q + kh * g + hl) * a.R + rr) * a.splits + sp;
        a.o_part[slot * hd + d] = Os[i];
        if (d == 0) a.ml_part[slot] = make_float2(ms[r], ls[r]);
    }
}

template <typename T>
__global__ void __launch_bounds__(128)
attention_combine_kernel(const float* __restrict__ o_part, const float2* __restrict__ ml_part, RowPlan rp, T* __restrict__ out,
                         int TB, int R, int n_q, int hd, int splits) {
    const int rr = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const size_t slot0 = (((size_t)b * n_q + h) * R + rr) * splits;
    const int m = b * R + rr, ld = n_q * hd;
    if (rr >= rp.seq_rows[b]) {
        for (int d = threadIdx.x; d < hd; d += blockDim.x) ActStore<T>::put(out, m, h * hd + d, ld, TB, 0.f);
        return;
    }
    float mx = -INFINITY;
    for (int s = 0; s < splits; ++s) mx = fmaxf(mx, ml_part[slot0 + s].x);
    float den = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float2 ml = ml_part[slot0 + s];
        if (ml.x != -INFINITY) den += expf(ml.x - mx) * ml.y;
    }
    for (int d = threadIdx.x; d < hd; d += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < splits; ++s) {
            const float m = ml_part[slot0 + s].x;
            if (m != -INFINITY) acc += expf(m - mx) * o_part[(slot0 + s) * hd + d];
        }
        ActStore<T>::put(out, m, h * hd + d, ld, TB, acc / den);
    }
}

size_t att_smem_bytes(int G, int hd) {
    return ((size_t)2 * G * hd + (size_t)TK * (hd + 1) + (size_t)TK * hd + 2 * (size_t)G) * sizeof(float);
}

}  // namespace

// Key-range splits per (sequence, KV head): enough CTAs to cover the SMs about twice, at least two
// 64-key tiles per split, at most 16 (the merge reads every split).
int attention_splits(int B, int n_kv, int max_ctx) {
    int s = (296 + B * n_kv - 1) / (B * n_kv);
    const int by_len = (max_ctx + 127) / 128;
    if (s > by_len) s = by_len;
    if (s > 16) s = 16;
    return s < 1 ? 1 : s;
}

size_t attention_scratch_bytes(int B, int R, int n_q, int hd, int n_splits) {
    const size_t slots = (size_t)B * n_q * R * n_splits;
    return slots * hd * sizeof(float) + slots * sizeof(float2);
}

template <typename T>
void launch_attention(const float* qbuf, const T* k_pages, const T* v_pages, const int32_t* block_table, int max_pages,
                      int page_size, long long n_pages, const RowPlan& rp, T* out, int TB, float* scratch, int B, int R,
                      int n_q, int n_kv, int hd, int n_splits, cudaStream_t stream) {
    AttArgs a;
    a.q = qbuf; a.kp = k_pages; a.vp = v_pages; a.block_table = block_table;
    a.max_pages = max_pages; a.page_size = page_size; a.n_pages = n_pages; a.rp = rp;
    const size_t slots = (size_t)B * n_q * R * n_splits;
    a.o_part = scratch;
    a.ml_part = reinterpret_cast<float2*>(scratch + slots * hd);
    a.B = B; a.R = R; a.n_q = n_q; a.n_kv = n_kv; a.hd = hd; a.splits = n_splits;
    a.scale = 1.0f / sqrtf((float)hd);
    const int G = (n_q / n_kv) * R;
    const size_t smem = att_smem_bytes(G, hd);
    static bool attr_f32 = false, attr_bf16 = false;
    bool& done = sizeof(T) == 4 ? attr_f32 : attr_bf16;
    if (!done) {
        cudaFuncSetAttribute(attention_split_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        done = true;
    }
    {
        ProfScope ps(K_ATT_SPLIT, stream);
        attention_split_kernel<T><<<dim3(n_splits, n_kv, B), ATT_THREADS, smem, stream>>>(a);
    }
    ProfScope ps(K_ATT_COMBINE, stream);
    attention_combine_kernel<T><<<dim3(R, n_q, B), hd < 128 ? 64 : 128, 0, stream>>>(a.o_part, a.ml_part, rp, out, TB, R, n_q, hd, n_splits);
}

template void launch_attention<float>(const float*, const float*, const float*, const int32_t*, int, int, long long,
                                      const RowPlan&, float*, int, float*, int, int, int, int, int, int, cudaStream_t);

}  // namespace tasc
