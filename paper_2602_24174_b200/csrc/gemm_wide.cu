// Projection GEMMs of the forward for passes with many token rows (M > 128: verify steps of large
// batches, prefill passes): the same products and fused consumers as gemm_fused.cu, in the orientation
// that suits a tensor-bound product.
//
// Shape of the work.  Y[128 tokens][BNW features] = X[128 tokens][K] * W[BNW rows][K]^T: the token rows
// supply UMMA M (TMEM lanes), the weight rows UMMA N (TMEM columns, BNW = 128 or 256).  Activations are
// float32 values carried as (hi, lo) bf16 row pairs in the tile layout [TBL hi rows][TBL lo rows]; one TMA
// box brings both halves of a k-block, and the hi and the lo rows are two MMAs into the SAME accumulator,
// so the sum hi + lo costs no extra pass.  (With TBL < 128 the MMA's last lanes read rows that belong to
// something else; a lane's result depends on its own row only, and those lanes are never stored.)
//
// Persistent CTAs.  One CTA per SM walks the (feature tile, token tile) pairs blockIdx.x, + gridDim.x, ...
// with two accumulators in TMEM: while the four epilogue warps drain tile j, the MMA warp already
// works on tile j + 1 in the other accumulator, and the TMA ring never stops between tiles.  A thread of
// the epilogue owns one token row (its TMEM lane) and 32 consecutive features per tcgen05.ld, so the
// row-wise consumers (RMS factor, RoPE pairs, sum of squares, row arg-max) need no exchange between threads.
//
// Split-K.  A product with few output tiles and a long reduction (the down-projection, the narrow QKV and
// O matrices) runs as clusters of S CTAs instead: one tile per cluster, CTA r takes the r-th share of the
// k-blocks, parks its accumulator in its own shared memory (the ring is idle by then), and after a cluster
// barrier finishes every S-th 32-feature unit of the tile, adding the S copies in rank order
// (ld.shared::cluster).  No partial sum reaches global memory and the result does not depend on timing.
//
// Warp roles (320 threads): warps 0-7 epilogue (TMEM lane quarter w % 4; the two warps of a quarter split the
// tile's 32-column units, since one warp per scheduler leaves the epilogue bound by instruction latency),
// warp 8 TMA producer, warp 9 TMEM allocation + MMA issue.  Every mbarrier wait is bounded and gives up early once another role of the
// CTA has failed; a wait that runs out records TASC_ETIMEOUT, and the CTA frees its TMEM and returns.
#include "kernels.h"

#include <algorithm>
#include <map>
#include <mutex>

namespace tasc {

namespace {

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 8;                 // two per TMEM lane quarter: they share the rows and split the 32-column units
constexpr int THREADS = (EPI_WARPS + 2) * 32;
constexpr int MAX_STAGES = 8;
constexpr int MAX_DYN_SMEM = 226 * 1024;

__device__ __forceinline__ bool wait_or_fail(uint32_t bar, uint32_t parity, volatile int* failed) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*failed) return false;
        if (clock64() - t0 > 1000000000ll) return false;
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(b)) << 16);
}
// 32 consecutive values of one row -> bf16, 64 bytes.
__device__ __forceinline__ void store_bf16x32(__nv_bfloat16* p, const float (&v)[32]) {
#pragma unroll
    for (int e = 0; e < 32; e += 8)
        *reinterpret_cast<uint4*>(p + e) = make_uint4(pack_bf16x2(v[e], v[e + 1]), pack_bf16x2(v[e + 2], v[e + 3]),
                                                      pack_bf16x2(v[e + 4], v[e + 5]), pack_bf16x2(v[e + 6], v[e + 7]));
}
// 32 consecutive values of one row -> (hi, lo) bf16, 64 bytes each.
__device__ __forceinline__ void store_hilo32(__nv_bfloat16* hi_ptr, __nv_bfloat16* lo_ptr, const float (&v)[32]) {
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
        uint32_t h[4], l[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            __nv_bfloat16 h0, l0, h1, l1;
            split_bf16(v[e + 2 * q], h0, l0);
            split_bf16(v[e + 2 * q + 1], h1, l1);
            h[q] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
            l[q] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
        }
        *reinterpret_cast<uint4*>(hi_ptr + e) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(lo_ptr + e) = make_uint4(l[0], l[1], l[2], l[3]);
    }
}
__device__ __forceinline__ void store_f32x32(float* p, const float (&v)[32]) {
#pragma unroll
    for (int e = 0; e < 32; e += 4) *reinterpret_cast<float4*>(p + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
}
__device__ __forceinline__ void load_f32x32(const float* p, float (&v)[32]) {
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const float4 t = *reinterpret_cast<const float4*>(p + e);
        v[e] = t.x; v[e + 1] = t.y; v[e + 2] = t.z; v[e + 3] = t.w;
    }
}
// 32 accumulator columns of this thread's TMEM lane, as floats.
__device__ __forceinline__ void acc32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    tmem_ld32(taddr, r);
    tmem_ld_wait();
#pragma unroll
    for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]);
}

template <int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const FusedArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);

    __shared__ uint64_t s_bars[2 * MAX_STAGES + 4];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;              // a bounded wait ran out somewhere in this CTA
    volatile int* failed = &s_fail;

    const int BNW = a.BNW, TBL = a.TBL, stages = a.stages, num_kb = a.num_kb;
    const uint32_t a_bytes = (uint32_t)(2 * TBL) * 128u;        // one k-block of the token tile: TBL hi rows, TBL lo rows
    const uint32_t w_bytes = (uint32_t)BNW * 128u;
    const uint32_t stage_bytes = a_bytes + w_bytes;
    const uint32_t bar_full = smem_u32(s_bars);
    const uint32_t bar_empty = bar_full + 8u * MAX_STAGES;
    const uint32_t bar_acc_full = bar_full + 16u * MAX_STAGES;  // [2]
    const uint32_t bar_acc_empty = bar_acc_full + 16u;          // [2]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = a.n_ft * a.n_tt;
    // S = 1: persistent, tiles blockIdx.x, + gridDim.x, ...   S > 1: the grid is S * n_tiles CTAs, one tile per cluster
    const int S = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int tile0 = S > 1 ? (int)blockIdx.x / S : (int)blockIdx.x;
    const int tstep = S > 1 ? n_tiles : (int)gridDim.x;
    const int my_tiles = tile0 < n_tiles ? (n_tiles - tile0 + tstep - 1) / tstep : 0;
    const int kb0 = (int)(((long long)num_kb * rank) / S);
    const int nkb = (int)(((long long)num_kb * (rank + 1)) / S) - kb0;      // k-blocks of this CTA (all of them when S = 1)
    constexpr int XPAD = 4;                                                 // floats: rows of the parked tile fall on distinct banks
    float* xch = reinterpret_cast<float*>(smem);                            // [128][BNW + XPAD], split-K only
    constexpr int FLD = 4 * 32 + XPAD;                                      // a CTA finishes at most four 32-column chunks of a split tile
    float* fin = xch + 128 * (BNW + XPAD);                                  // [128][FLD] the S copies of this CTA's chunks, added up
    uint32_t own_mask = 0u;                                                 // split-K: the tile's 32-column chunks that this CTA finishes
    const int FT = EPI == EPI_SWIGLU ? BNW / 2 : BNW;           // output features per tile
    auto fail = [&]() { set_status(a.status, TASC_ETIMEOUT); *failed = 1; };
#ifdef TASC_TIMELINE
    const unsigned long long g_t0 = global_ns();
    unsigned long long g_ta = 0, g_tb = 0, g_tc = 0, g_td = 0, g_te = 0, g_tf = 0;
#endif

    if (threadIdx.x == 0) {
        s_fail = 0;
        for (int s = 0; s < stages; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8u * b, 1);
            mbar_init(bar_acc_empty + 8u * b, EPI_WARPS * 32);
        }
        fence_barrier_init();
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
    }
    if (warp == EPI_WARPS + 1) {
        tmem_alloc(smem_u32(&s_tmem), (uint32_t)(2 * BNW));
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem;

    if (warp == EPI_WARPS) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_w = a.n_tt > 1 ? policy_evict_last() : policy_evict_first();   // a weight tile is read once per token tile
            const uint64_t pol_x = policy_evict_last();                                       // token rows are read by every feature tile
            const int total = my_tiles * nkb;
            auto load_w = [&](int i) {
                const int tile = tile0 + (i / nkb) * tstep;
                const int f0 = (tile / a.n_tt) * FT, kc = (kb0 + i % nkb) * BK;
                const int s = i % stages;
                const uint32_t dst = smem_u32(smem + (size_t)s * stage_bytes) + a_bytes, bar = bar_full + 8u * s;
                if (EPI == EPI_SWIGLU) {                   // FT gate rows, then the FT matching up rows (boxes of 64 rows)
                    for (int r = 0; r < FT; r += 64) {
                        tma_load_2d_hint(dst + (uint32_t)r * 128u, &tmW, kc, f0 + r, bar, pol_w);
                        tma_load_2d_hint(dst + (uint32_t)(FT + r) * 128u, &tmW, kc, a.N + f0 + r, bar, pol_w);
                    }
                } else {                                   // boxes of 128 rows
                    for (int r = 0; r < BNW; r += 128) tma_load_2d_hint(dst + (uint32_t)r * 128u, &tmW, kc, f0 + r, bar, pol_w);
                }
            };
            auto load_x = [&](int i) {
                const int tile = tile0 + (i / nkb) * tstep;
                const int s = i % stages;
                tma_load_2d_hint(smem_u32(smem + (size_t)s * stage_bytes), &tmX, (kb0 + i % nkb) * BK, (tile % a.n_tt) * 2 * TBL,
                                 bar_full + 8u * s, pol_x);
            };
            // The weights of the first stages depend on no earlier kernel: they are requested before the
            // preceding grid has finished, the token rows after it.
            const int pre = total < stages ? total : stages;
            for (int i = 0; i < pre; ++i) {
                mbar_expect_tx(bar_full + 8u * (i % stages), stage_bytes);
                load_w(i);
            }
            griddep_wait();
            for (int i = 0; i < pre; ++i) load_x(i);
            for (int i = pre; i < total; ++i) {
                const int s = i % stages;
                if (!wait_or_fail(bar_empty + 8u * s, (((uint32_t)(i / stages)) & 1u) ^ 1u, failed)) { fail(); break; }
                mbar_expect_tx(bar_full + 8u * s, stage_bytes);
                load_w(i);
                load_x(i);
            }
            griddep_launch_dependents();
        }
        __syncwarp();
    } else if (warp == EPI_WARPS + 1) {
        // ------------------------------------------------------------ MMA issue
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_f32(128, BNW);
            int it = 0;
            bool ok = true;
            for (int j = 0; j < my_tiles && ok; ++j) {
                const int b = j & 1;
                if (!wait_or_fail(bar_acc_empty + 8u * b, (((uint32_t)(j >> 1)) & 1u) ^ 1u, failed)) { fail(); break; }
                tc_fence_after();
                const uint32_t d = tmem_base + (uint32_t)(b * BNW);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % stages;
                    if (!wait_or_fail(bar_full + 8u * s, ((uint32_t)(it / stages)) & 1u, failed)) { fail(); ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint32_t sb = sa + a_bytes;
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        umma_bf16(d, umma_desc_k_sw128(sa + kk * UMMA_K * 2), umma_desc_k_sw128(sb + kk * UMMA_K * 2), idesc,
                                  (kb > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        umma_bf16(d, umma_desc_k_sw128(sa + (uint32_t)TBL * 128u + kk * UMMA_K * 2),
                                  umma_desc_k_sw128(sb + kk * UMMA_K * 2), idesc, 1u);
                    umma_commit(bar_empty + 8u * s);
                }
                if (ok) umma_commit(bar_acc_full + 8u * b);
            }
        }
        __syncwarp();
    }

    // ---------------------------------------------------------------- epilogue: one token row per thread (warps 0-7)
    const int quarter = warp & 3, wq = (warp >> 2) & 1;              // TMEM lane quarter; which of the quarter's two warps
    const int rowl = quarter * 32 + lane;                             // row within the token tile = TMEM lane
    const int XLD = BNW + XPAD;
    uint32_t peer[8];
    {
#pragma unroll
        for (int s = 0; s < 8; ++s) peer[s] = cluster_map(smem_u32(xch), (uint32_t)(s < S ? s : 0));
    }
    // Finishes tile `tile`.  `acc` = TMEM address of this thread's lane in the tile's accumulator.  With split-K the
    // 32-column units come from the S parked copies instead, added in rank order, and this CTA takes every S-th unit.
    auto finish_tile = [&](int tile, uint32_t acc) {
        const int ft = tile / a.n_tt, tt = tile % a.n_tt;
        const int f0 = ft * FT;
        const int m = tt * TBL + rowl;
        const bool rowok = rowl < TBL && m < a.M;
        const size_t orow = (size_t)tt * (2 * TBL) + rowl;            // row of the (hi, lo) output layout; lo at + TBL
        auto get32 = [&](int col, float (&v)[32]) {
            if (S == 1) {
                acc32(acc + (uint32_t)col, v);
            } else {
                // the reduced columns of this CTA's units, packed in the order of their 32-column chunks
                const int jc = __popc(own_mask & ((1u << (col >> 5)) - 1u));
                const float* src = fin + (size_t)rowl * FLD + jc * 32;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float4 q = *reinterpret_cast<const float4*>(src + 4 * e);
                    v[4 * e] = q.x; v[4 * e + 1] = q.y; v[4 * e + 2] = q.z; v[4 * e + 3] = q.w;
                }
            }
        };
        int unit = 0;                                                 // running index of the tile's work units
        int owned = 0;                                                // ... of those of this CTA (every S-th)
        auto mine = [&]() {                                           // the quarter's two warps alternate over the CTA's units
            const bool own = (unit++ % S) == rank;
            return own && (owned++ & 1) == wq;
        };
        float sc = 1.0f;
        if (a.ssq_in && rowok) {
            float ss = 0.f;
            if (a.ssq_slots % 4 == 0) {
                const float4* sp = reinterpret_cast<const float4*>(a.ssq_in + (size_t)m * a.ssq_slots);
                for (int q = 0; q < a.ssq_slots / 4; ++q) { const float4 t = sp[q]; ss += (t.x + t.y) + (t.z + t.w); }
            } else {
                for (int q = 0; q < a.ssq_slots; ++q) ss += a.ssq_in[(size_t)m * a.ssq_slots + q];
            }
            sc = 1.0f / sqrtf(ss * a.inv_d + a.eps);
        }

        if (EPI == EPI_SWIGLU) {
            for (int c = 0; c < FT && f0 + c < a.N; c += 32) {
                if (!mine()) continue;
                float g[32], u[32];
                get32(c, g);
                get32(FT + c, u);
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float g0 = g[e] * sc, u0 = u[e] * sc;
                    g[e] = __fdividef(g0, 1.0f + __expf(-g0)) * u0;
                }
                if (rowok) store_hilo32(a.a_out + orow * a.N + f0 + c, a.a_out + (orow + TBL) * a.N + f0 + c, g);
            }
        } else if (EPI == EPI_RESID) {
            // ssq_out has one slot per 32 features here (a.ssq_out_slots of them, a multiple of four per 128 features)
            for (int c = 0; c < BNW && f0 + c < a.N; c += 32) {
                if (!mine()) continue;
                const int f = f0 + c;
                float v[32], x[32];
                get32(c, v);
                if (rowok) {
                    float* xrow = a.x + (size_t)m * a.N + f;
                    load_f32x32(xrow, x);
                    float ss = 0.f;
#pragma unroll
                    for (int e = 0; e < 32; ++e) { x[e] += v[e]; ss += x[e] * x[e]; }
                    store_f32x32(xrow, x);
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        const float4 g4 = __ldg(reinterpret_cast<const float4*>(a.gain + f + e));
                        x[e] *= g4.x; x[e + 1] *= g4.y; x[e + 2] *= g4.z; x[e + 3] *= g4.w;
                    }
                    store_hilo32(a.a_out + orow * a.N + f, a.a_out + (orow + TBL) * a.N + f, x);
                    a.ssq_out[(size_t)m * a.ssq_out_slots + f / 32] = ss;
                    if (f + 32 >= a.N)                                // the slots past the last 32 features
                        for (int q = f / 32 + 1; q < a.ssq_out_slots; ++q) a.ssq_out[(size_t)m * a.ssq_out_slots + q] = 0.f;
                }
            }
        } else if (EPI == EPI_QKV) {
            const int hd = a.hd, half = hd >> 1;
            const int qd = a.n_q * hd, kvd = a.n_kv * hd;
            int pos = -1, page = -1;
            if (rowok) {
                pos = a.row_pos[m];
                if (pos >= a.max_positions) { set_status(a.status, TASC_EINVAL); pos = -1; }
                if (pos >= 0 && f0 + BNW > qd) {                      // the tile holds K or V heads
                    const int pslot = pos / a.page_size;
                    if (pslot < a.max_pages) page = a.block_table[(size_t)(m / a.R) * a.max_pages + pslot];
                    if (page < 0 || page >= a.n_pages) { set_status(a.status, TASC_ENOKV); page = -1; }
                }
            }
            for (int hc = 0; hc < BNW && f0 + hc < a.N; hc += hd) {
                const int fh = f0 + hc;                               // first feature of this head
                if (fh < qd + kvd) {
                    // a query or key head: rotate the pairs (i, i + half); a unit is 32 pairs
                    const bool is_q = fh < qd;
                    __nv_bfloat16* kdst = nullptr;
                    if (!is_q && pos >= 0 && page >= 0)
                        kdst = a.k_pages + (((size_t)page * a.n_kv + (fh - qd) / hd) * a.page_size + pos % a.page_size) * hd;
                    for (int jj = 0; jj < half; jj += 32) {
                        if (!mine()) continue;
                        float lo[32], hi[32];
                        get32(hc + jj, lo);
                        get32(hc + half + jj, hi);
                        // (cos, sin) of the pair indices jj .. jj + 31 of this row's position: 64 floats, two units
                        if (pos >= 0) {
                            const float4* cs = reinterpret_cast<const float4*>(a.rope + (size_t)pos * half + jj);
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                const float4 t = cs[e >> 1];          // (cos, sin) of pair indices jj + e, jj + e + 1
                                const float a0 = lo[e] * sc, b0 = hi[e] * sc, a1 = lo[e + 1] * sc, b1 = hi[e + 1] * sc;
                                lo[e] = a0 * t.x - b0 * t.y;     hi[e] = b0 * t.x + a0 * t.y;
                                lo[e + 1] = a1 * t.z - b1 * t.w; hi[e + 1] = b1 * t.z + a1 * t.w;
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; ++e) { lo[e] = 0.f; hi[e] = 0.f; }
                        }
                        if (is_q) {
                            if (rowok) {
                                store_f32x32(a.qbuf + (size_t)m * qd + fh + jj, lo);
                                store_f32x32(a.qbuf + (size_t)m * qd + fh + half + jj, hi);
                            }
                        } else if (kdst) {
                            store_bf16x32(kdst + jj, lo);
                            store_bf16x32(kdst + half + jj, hi);
                        }
                    }
                } else {
                    // a value head
                    __nv_bfloat16* vdst = nullptr;
                    if (pos >= 0 && page >= 0)
                        vdst = a.v_pages + (((size_t)page * a.n_kv + (fh - qd - kvd) / hd) * a.page_size + pos % a.page_size) * hd;
                    for (int c = 0; c < hd; c += 32) {
                        if (!mine()) continue;
                        float v[32];
                        get32(hc + c, v);
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] *= sc;
                        if (vdst) store_bf16x32(vdst + c, v);
                    }
                }
            }
        } else if (EPI == EPI_LM) {
            // the row's largest logit in this tile (smallest id on ties), merged across tiles by an atomic max on
            // the packed (value, id) word
            uint32_t bk = 0u, bi = 0xFFFFFFFFu;
            for (int c = 0; c < BNW && f0 + c < a.N; c += 32) {
                if (!mine()) continue;
                float v[32];
                get32(c, v);
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const uint32_t k = float_key(v[e]);
                    if (bi == 0xFFFFFFFFu || k > bk) { bk = k; bi = (uint32_t)(f0 + c + e); }
                }
                if (a.logits && rowok) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] *= sc;
                    store_f32x32(a.logits + (size_t)m * a.N + f0 + c, v);
                }
            }
            if (rowok && bi != 0xFFFFFFFFu)
                atomicMax(&a.argmax[m], ((unsigned long long)bk << 32) | (unsigned long long)(0xFFFFFFFFu - bi));
        }
    };

    if (warp < EPI_WARPS) {
        griddep_wait();
#ifdef TASC_TIMELINE
        g_ta = global_ns();
#endif
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        if (S == 1) {
            for (int j = 0; j < my_tiles; ++j) {
                const int b = j & 1;
                bool ok = wait_or_fail(bar_acc_full + 8u * b, ((uint32_t)(j >> 1)) & 1u, failed);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) { if (lane == 0) fail(); break; }
#ifdef TASC_TIMELINE
                if (j == 0) g_tb = global_ns();
                if (j == my_tiles - 1) g_tc = global_ns();
#endif
                tc_fence_after();
                finish_tile(tile0 + j * tstep, lane_base + (uint32_t)(b * BNW));
                tc_fence_before();
                mbar_arrive(bar_acc_empty + 8u * b);
            }
        } else if (my_tiles > 0) {
            // split-K, part 1: this CTA's partial tile -> its shared memory (zeros after a failed wait, so that the
            // peers read something defined)
            bool ok = nkb > 0 && wait_or_fail(bar_acc_full, 0u, failed);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok && nkb > 0 && lane == 0) fail();
#ifdef TASC_TIMELINE
            g_tb = global_ns();
#endif
            tc_fence_after();
            for (int c = 32 * wq; c < BNW; c += 64) {
                float v[32];
                if (ok) {
                    acc32(lane_base + (uint32_t)c, v);
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0.f;
                }
                store_f32x32(xch + (size_t)rowl * XLD + c, v);
            }
            tc_fence_before();
        }
    }
    if (S > 1) {
        // every CTA's partial tile is in its shared memory (release / acquire at cluster scope)
#ifdef TASC_TIMELINE
        g_tc = global_ns();
#endif
        cluster_arrive();
        cluster_wait();
#ifdef TASC_TIMELINE
        g_td = global_ns();
#endif
        if (warp < EPI_WARPS && my_tiles > 0) {
            // split-K, part 2: the chunks of this CTA's units (every S-th unit of the tile, in the order finish_tile meets
            // them), summed over the S parked copies in rank order into `fin`.  A work item is one chunk of one lane
            // quarter (32 rows x 32 columns); eight consecutive lanes cover the 128 bytes of a row, so a warp-wide
            // remote read touches 4 rows, and the reads of all copies are in flight together.
            {
                const int f0 = (tile0 / a.n_tt) * FT;
                int unit = 0;
                auto take = [&](int c0, int c1) {
                    if ((unit++ % S) == rank) { own_mask |= 1u << (c0 >> 5); if (c1 >= 0) own_mask |= 1u << (c1 >> 5); }
                };
                if (EPI == EPI_QKV) {
                    const int hd = a.hd, half = hd >> 1, qkd = (a.n_q + a.n_kv) * hd;
                    for (int hc = 0; hc < BNW && f0 + hc < a.N; hc += hd) {
                        if (f0 + hc < qkd) { for (int jj = 0; jj < half; jj += 32) take(hc + jj, hc + half + jj); }
                        else { for (int c = 0; c < hd; c += 32) take(hc + c, -1); }
                    }
                } else {
                    for (int c = 0; c < BNW && f0 + c < a.N; c += 32) take(c, -1);
                }
            }
            const int n_own = __popc(own_mask);
            for (int idx = warp; idx < n_own * 4; idx += EPI_WARPS) {
                const int jc = idx >> 2, q = idx & 3;
                const int chunk = __fns(own_mask, 0, jc + 1);         // the jc-th chunk of the mask
                const uint32_t off = (uint32_t)((q * 32 + (lane >> 3)) * XLD + chunk * 32 + 4 * (lane & 7)) * 4u;
                float* dst = fin + (size_t)(q * 32 + (lane >> 3)) * FLD + jc * 32 + 4 * (lane & 7);
#pragma unroll
                for (int ib = 0; ib < 8; ib += 2) {                   // rows lane / 8 + 4 i, two i at a time: 2 S reads in flight
                    float4 u[8][2];
#pragma unroll
                    for (int s2 = 0; s2 < 8; ++s2)
                        if (s2 < S) {
                            u[s2][0] = ld_cluster_f4(peer[s2] + off + (uint32_t)(4 * ib * XLD) * 4u);
                            u[s2][1] = ld_cluster_f4(peer[s2] + off + (uint32_t)(4 * (ib + 1) * XLD) * 4u);
                        }
                    float4 t0 = u[0][0], t1 = u[0][1];
#pragma unroll
                    for (int s2 = 1; s2 < 8; ++s2)
                        if (s2 < S) {
                            t0.x += u[s2][0].x; t0.y += u[s2][0].y; t0.z += u[s2][0].z; t0.w += u[s2][0].w;
                            t1.x += u[s2][1].x; t1.y += u[s2][1].y; t1.z += u[s2][1].z; t1.w += u[s2][1].w;
                        }
                    *reinterpret_cast<float4*>(dst + (size_t)(4 * ib) * FLD) = t0;
                    *reinterpret_cast<float4*>(dst + (size_t)(4 * (ib + 1)) * FLD) = t1;
                }
            }
            asm volatile("bar.sync 1, %0;" ::"n"(EPI_WARPS * 32) : "memory");   // the eight epilogue warps
            finish_tile(tile0, 0u);
        }
#ifdef TASC_TIMELINE
        g_te = global_ns();
#endif
        // peers may still be reading this CTA's partial tile
        cluster_arrive();
        cluster_wait();
    }
#ifdef TASC_TIMELINE
    g_tf = global_ns();
#endif
    __syncthreads();
    if (s_fail && warp == EPI_WARPS && lane == 0) {
        // after a timeout: give this CTA's own tile loads that may still be in flight a bounded time to land
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
    }
    __syncthreads();
    if (warp == EPI_WARPS + 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)(2 * BNW));
    }
#ifdef TASC_TIMELINE
    if (threadIdx.x == 0) ctalog_put(g_t0, g_ta, g_tb, 20 + EPI, g_tc, g_td, g_te, g_tf);
#endif
}

template <int EPI>
tasc_status prepare_wide() {
    static std::mutex mu;
    static bool attr_done[64] = {false};
    int dev = 0;
    TASC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return TASC_EINVAL;
    std::lock_guard<std::mutex> lk(mu);
    if (!attr_done[dev]) {
        TASC_CUDA_TRY(cudaFuncSetAttribute(gemm_wide_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN_SMEM));
        attr_done[dev] = true;
    }
    return TASC_OK;
}

template <int EPI>
tasc_status launch_wide(const CUtensorMap* tmW, const CUtensorMap* tmX, const FusedArgs& a, const FusedPlan& p, int kind,
                        cudaStream_t stream) {
    tasc_status pst = prepare_wide<EPI>();
    if (pst != TASC_OK) return pst;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid, 1, 1);
    cfg.blockDim = dim3(THREADS, 1, 1);
    cfg.dynamicSmemBytes = (size_t)p.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute at[2];
    int n = 0;
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (p.S > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = (unsigned)p.S;
        at[n].val.clusterDim.y = 1;
        at[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    ProfScope ps(kind, stream);
    TASC_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_wide_kernel<EPI>, *tmW, *tmX, a));
    return TASC_OK;
}

// Clusters of S CTAs with `smem` bytes each that the device can hold at once (0 if the query fails).
template <int EPI>
int wide_clusters(int S, int smem) {
    if (prepare_wide<EPI>() != TASC_OK) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)S, 1, 1);
    cfg.blockDim = dim3(THREADS, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)S;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_wide_kernel<EPI>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

int wide_clusters_any(int epi, int S, int smem) {
    static std::mutex mu;
    static std::map<long long, int> cache;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    const long long key = (((long long)dev * 8 + epi) * 32 + S) * (1ll << 20) + smem;
    std::lock_guard<std::mutex> lk(mu);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    int n = 0;
    switch (epi) {
        case EPI_QKV:    n = wide_clusters<EPI_QKV>(S, smem); break;
        case EPI_RESID:  n = wide_clusters<EPI_RESID>(S, smem); break;
        default: break;
    }
    cache[key] = n;
    return n;
}

int sm_count() {
    static std::mutex mu;
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 148; }
    std::lock_guard<std::mutex> lk(mu);
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { (void)cudaGetLastError(); n = 148; }
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace

bool plan_wide(int M, int N, int K, int epi, int hd, FusedPlan& p, int token_tile) {
    if ((M <= 128 && token_tile <= 0) || N % 32 || K % 8) return false;
    if (epi != EPI_QKV && epi != EPI_RESID && epi != EPI_SWIGLU && epi != EPI_LM) return false;
    if (epi == EPI_QKV && hd != 64 && hd != 128) return false;
    p.TBL = token_tile > 0 ? token_tile : gemm_token_tile(M, true, 3, true);
    p.TB = p.TBL;
    p.BN = 2 * p.TBL;
    p.m_tiles = (M + p.TBL - 1) / p.TBL;
    p.num_kb = (K + BK - 1) / BK;
    p.wide = 1;
    const int sms = sm_count();
    // Tile width and k-splits, by a cost in SM cycles.  A k-block of a tile of `bnw` features is 8 MMAs of bnw / 2 cycles
    // and brings (2 TBL + bnw) rows of 128 bytes into shared memory, which an SM takes in at about 40 bytes per cycle
    // (measured: 0.97 us per k-block at 256 features, 0.70 us at 128).  A persistent grid (S = 1) pays one epilogue that
    // nothing hides; a split-K grid pays the parking of the tile, two cluster barriers and the pull of S copies.
    const bool may_split = epi == EPI_QKV || epi == EPI_RESID;
    double best_cost = -1.;
    for (int bnw = 256; bnw >= 128; bnw >>= 1) {
        const int ft = epi == EPI_SWIGLU ? bnw / 2 : bnw;
        const int tiles = ((N + ft - 1) / ft) * p.m_tiles;
        const int stage_bytes = (2 * p.TBL + bnw) * 128;
        const int st = std::max(2, std::min((200 * 1024) / stage_bytes, MAX_STAGES));
        const int data = std::max(st * stage_bytes, 128 * (bnw + 4) * 4 + 128 * (4 * 32 + 4) * 4);
        const int smem = std::min(std::max(1024 + data, 120 * 1024), MAX_DYN_SMEM);
        const double per_kb = std::max(4.0 * bnw, (2.0 * p.TBL + bnw) * 128.0 / 40.0);
        for (int S = 1; S <= (may_split ? 8 : 1); ++S) {
            if (S > p.num_kb || (S > 1 && tiles * S > sms)) break;
            if (S > 1) {
                const int fit = wide_clusters_any(epi, S, smem);
                if (fit <= 0 || tiles > fit) continue;
            }
            const int waves = S > 1 ? 1 : (tiles + sms - 1) / sms;
            const double cost = (double)waves * ((p.num_kb + S - 1) / S) * per_kb + (S > 1 ? 6000.0 + 10.0 * bnw : 12.0 * bnw);
            if (best_cost < 0. || cost < best_cost) {
                best_cost = cost;
                p.BNW = bnw; p.S = S; p.out_tiles = (N + ft - 1) / ft; p.stages = st; p.data_bytes = data; p.smem_bytes = smem;
                p.grid = S > 1 ? tiles * S : std::min(tiles, sms);
            }
        }
    }
    return best_cost >= 0.;
}

tasc_status launch_gemm_wide(int epi, const CUtensorMap* tmW, const CUtensorMap* tmX, FusedArgs a, const FusedPlan& p,
                             cudaStream_t stream) {
    a.num_kb = p.num_kb; a.BN = p.BN; a.TB = p.TB; a.TBL = p.TBL; a.stages = p.stages; a.pair = 1; a.data_bytes = p.data_bytes;
    a.BNW = p.BNW; a.n_ft = p.out_tiles; a.n_tt = p.m_tiles;
    switch (epi) {
        case EPI_QKV:    return launch_wide<EPI_QKV>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_RESID:  return launch_wide<EPI_RESID>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_SWIGLU: return launch_wide<EPI_SWIGLU>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_LM:     return launch_wide<EPI_LM>(tmW, tmX, a, p, K_GEMM_LM, stream);
        default: return TASC_EINVAL;
    }
}

}  // namespace tasc
