// Projection GEMMs of the verify forward with their consumers fused in: tcgen05 MMA with float32
// accumulators in TMEM, weights streamed by TMA, split-K reduced through distributed shared memory
// inside a thread-block cluster, and the stage that follows the product (RoPE + KV append, residual +
// next norm's input, SiLU * up, LM-head argmax) done on the reduced tile before anything goes to HBM.
//
// Shape of the work.  Y^T[128 features][tokens] = W[128 rows][K] * X^T, operands swapped because the
// step has few token rows (M = B * (k+1)) and large weight matrices: the weight tile supplies UMMA M,
// the token rows UMMA N.  Activations are float32 values carried as (hi, lo) bf16 row pairs in the
// tile-local layout [TB hi rows][TB lo rows], both halves go through one MMA (N = 2 TB) and the
// accumulator columns j and j + TB are added afterwards.
//
// Split-K.  The narrow matrices of small models give few 128-row tiles, so a cluster of S CTAs shares
// one output tile and splits the k-range.  Each CTA copies its accumulator to its own shared memory;
// after a cluster barrier CTA r reads, for its 1/S share of the token columns, the S copies
// (ld.shared::cluster, all issued before the first is used), adds them in rank order and runs the
// epilogue for those columns.  No partial sum reaches global memory, there are no atomics, and the
// result does not depend on timing.
//
// RMSNorm without a row-wide pass.  The producer of a normalised input writes x * gain (as hi/lo)
// and, per 128-feature tile, the row's partial sum of squares; the consumer GEMM multiplies its
// output row by 1 / sqrt(mean(x^2) + eps), which commutes with the product.
//
// Launch overlap.  Kernels are launched with programmatic stream serialisation: a CTA sets up its
// barriers and TMEM and streams the first weight tiles of its k-range into the ring (weights do not
// depend on earlier kernels), then waits for the preceding grid (griddepcontrol.wait) before it
// touches activations, and releases the next grid once its last weight load has been issued.
//
// Warp roles (192 threads): warps 0-3 epilogue (TMEM lane quarter w), warp 4 TMA producer, warp 5
// TMEM allocation + MMA issue; all of them reduce and finish token columns afterwards.  Where a CTA
// finishes a dozen columns or more, that part is bound by instruction latency (one warp per scheduler),
// and the launch carries six more warps (384 threads) that do nothing else.  Every mbarrier wait is bounded; a wait that runs out records
// TASC_ETIMEOUT, the CTA still takes part in the cluster barriers, frees its TMEM and returns.
#include "kernels.h"

#include <algorithm>
#include <map>
#include <mutex>

namespace tasc {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int THREADS = 192;                  // six warps; launches with many token columns per CTA add six more that only finish columns
constexpr int MAX_THREADS = 384;
constexpr int FINISHERS_MIN_COLS = 12;
constexpr double LM_WIDE_MIN_MB = 100.0;
constexpr int MAX_DYN_SMEM = 226 * 1024;      // 227 KB per CTA minus the kernel's static shared memory

#ifdef TASC_TIMELINE
// Development aid, compiled only with -DTASC_TIMELINE: cycle stamps of the phases of every CTA.
__device__ long long g_timeline[4096][16];
#define TL(slot) do { if (cta_lin < 4096) g_timeline[cta_lin][slot] = clock64() - tl0; } while (0)
#else
#define TL(slot) do { } while (0)
#endif

__device__ __forceinline__ float4 shfl_xor4(float4 v, int d) {
    float4 r;
    r.x = __shfl_xor_sync(0xFFFFFFFFu, v.x, d);
    r.y = __shfl_xor_sync(0xFFFFFFFFu, v.y, d);
    r.z = __shfl_xor_sync(0xFFFFFFFFu, v.z, d);
    r.w = __shfl_xor_sync(0xFFFFFFFFu, v.w, d);
    return r;
}

// Four consecutive values -> (hi, lo) bf16 quadruples, 8 bytes each.
__device__ __forceinline__ void store_hilo4(__nv_bfloat16* hi_ptr, __nv_bfloat16* lo_ptr, const float v[4]) {
    __nv_bfloat16 h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) split_bf16(v[e], h[e], l[e]);
    uint2 ph, pl;
    ph.x = (uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16);
    ph.y = (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16);
    pl.x = (uint32_t)__bfloat16_as_ushort(l[0]) | ((uint32_t)__bfloat16_as_ushort(l[1]) << 16);
    pl.y = (uint32_t)__bfloat16_as_ushort(l[2]) | ((uint32_t)__bfloat16_as_ushort(l[3]) << 16);
    *reinterpret_cast<uint2*>(hi_ptr) = ph;
    *reinterpret_cast<uint2*>(lo_ptr) = pl;
}
__device__ __forceinline__ void store_bf16x4(__nv_bfloat16* p, const float v[4]) {
    uint2 u;
    u.x = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[0])) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[1])) << 16);
    u.y = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[2])) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[3])) << 16);
    *reinterpret_cast<uint2*>(p) = u;
}

// EW: warps of the CTA (6, or 12 with the additional column finishers); all of them reduce and finish columns.
template <int EPI, int EW>
__global__ void __launch_bounds__(EW * 32, 1)
gemm_fused_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const FusedArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);

    const int BN = a.BN, stages = a.stages, TB = a.TB, TBL = a.TBL;   // TB tokens per CTA = one or more layout tiles of TBL
    const uint32_t b_stage_bytes = (uint32_t)BN * BK * 2;
    const uint32_t stage_bytes = A_STAGE_BYTES + b_stage_bytes;
    // [TB][128] this CTA's partial tile; behind the ring, except for the LM head, which has no cluster exchange
    // and parks it in the ring once its MMAs are done
    float* xch = reinterpret_cast<float*>(EPI == EPI_LM ? smem : smem + (size_t)stages * stage_bytes);
    float* fin = reinterpret_cast<float*>(smem);                                          // [per][128] reduced columns (the ring is idle by then)
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + a.data_bytes);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8u * stages;
    const uint32_t bar_acc = bar_full + 16u * stages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * stages + 1);
    float* s_inv = reinterpret_cast<float*>(bars + 2 * stages + 2);                       // [128]

    const int S = (int)cluster_nctarank();
    const int rank = (int)cluster_ctarank();
    const int out_tile = blockIdx.y, m_tile = blockIdx.z;
    const int kb_begin = (int)(((long long)a.num_kb * rank) / S);
    const int kb_end = (int)(((long long)a.num_kb * (rank + 1)) / S);
    const int n_kb = kb_end - kb_begin;
    const int f0 = out_tile * (EPI == EPI_SWIGLU ? 64 : BM);   // first output feature of the tile
    const int m0 = m_tile * BN;                                // first row of the tile in the activation buffer
    const int t0 = m_tile * TB;                                // first token of the tile
    int valid = a.M - t0;                                      // token columns in use
    valid = valid > TB ? TB : valid;
    const int per = (valid + S - 1) / S;                       // token columns reduced and finished by each CTA of the cluster

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef TASC_TIMELINE
    const long long tl0 = clock64();
    const unsigned long long g_t0 = global_ns();
    __shared__ unsigned long long g_ta, g_tb, g_tc, g_td, g_te, g_tf;
    const int cta_lin = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
#endif
    uint32_t ncols = 32;
    while ((int)ncols < BN) ncols <<= 1;
    __shared__ int s_fail;              // a bounded wait ran out somewhere in this CTA
    auto fail = [&]() { set_status(a.status, TASC_ETIMEOUT); s_fail = 1; };

    const uint64_t pol_w = policy_evict_first();   // weights are read once per step
    const uint64_t pol_x = policy_evict_last();    // token rows are re-read by every CTA
    auto load_w = [&](int i, uint32_t dstA, uint32_t bar) {
        const int kc = (kb_begin + i) * BK;
        if (EPI == EPI_SWIGLU) {                   // 64 gate rows, then the 64 matching up rows
            tma_load_2d_hint(dstA, &tmW, kc, f0, bar, pol_w);
            tma_load_2d_hint(dstA + A_STAGE_BYTES / 2, &tmW, kc, a.N + f0, bar, pol_w);
        } else {
            tma_load_2d_hint(dstA, &tmW, kc, f0, bar, pol_w);
        }
    };
    const int pre = n_kb < stages ? n_kb : stages;

    // Token columns this CTA reduces and finishes: [rank * per, rank * per + count).
    int count = valid - rank * per;
    count = count < 0 ? 0 : (count > per ? per : count);
    // Global operands of the epilogue of one column (position, rotary factors, KV page, residual row).  The
    // first NPF columns of every warp are fetched while the MMAs run, so their latency is off the tail.
    struct Pre { float4 x, cs01, cs23; int pos, page; };
    constexpr int NPF = 3;
    // every warp reduces and finishes columns: column tl belongs to warp tl % EW
    auto prefetch = [&](int tl) -> Pre {
        Pre q;
        q.x = q.cs01 = q.cs23 = make_float4(0.f, 0.f, 0.f, 0.f);
        q.pos = -1; q.page = -1;
        const int m = t0 + rank * per + tl;
        const int f = f0 + 4 * lane;
        if (EPI == EPI_QKV) {
            const int hd = a.hd, half = hd >> 1;
            const int qd = a.n_q * hd, kvd = a.n_kv * hd;
            int pos = a.row_pos[m];
            if (pos >= a.max_positions) { set_status(a.status, TASC_EINVAL); pos = -1; }
            q.pos = pos;
            if (pos >= 0 && f < qd + kvd) {
                const float4* cs = reinterpret_cast<const float4*>(a.rope + (size_t)pos * half + ((f % hd) % half));
                q.cs01 = cs[0];                                  // (cos, sin) of four consecutive pair indices
                q.cs23 = cs[1];
            }
            if (pos >= 0 && f >= qd && f < qd + 2 * kvd) {
                const int pslot = pos / a.page_size;
                if (pslot < a.max_pages) q.page = a.block_table[(size_t)(m / a.R) * a.max_pages + pslot];
                if (q.page < 0 || q.page >= a.n_pages) { set_status(a.status, TASC_ENOKV); q.page = -1; }
            }
        } else if (EPI == EPI_RESID) {
            if (f < a.N) q.x = *reinterpret_cast<const float4*>(a.x + (size_t)m * a.N + f);
        }
        return q;
    };
    float4 gain4 = make_float4(0.f, 0.f, 0.f, 0.f);
    auto finish = [&](int tl, const Pre& q) {
        const int t = rank * per + tl;
        const float4 acc = *reinterpret_cast<const float4*>((S > 1 ? fin + (size_t)tl * BM : xch + (size_t)t * BM) + 4 * lane);
        const int m = t0 + t;
        if (EPI == EPI_PLAIN) {
            const float sc = a.ssq_in ? s_inv[t] : 1.0f;
            const float v[4] = {acc.x * sc, acc.y * sc, acc.z * sc, acc.w * sc};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int f = f0 + 4 * lane + e;
                if (f < a.N) a.y[(size_t)m * a.N + f] = v[e];
            }
        } else if (EPI == EPI_QKV) {
            const float sc = s_inv[t];
            const float4 sacc = make_float4(acc.x * sc, acc.y * sc, acc.z * sc, acc.w * sc);
            const int hd = a.hd, half = hd >> 1;
            const float4 partner = shfl_xor4(sacc, half >> 2);
            const int f = f0 + 4 * lane;
            const int qd = a.n_q * hd, kvd = a.n_kv * hd;
            const int pos = q.pos;
            float v[4] = {sacc.x, sacc.y, sacc.z, sacc.w};
            if (f < qd + kvd && pos >= 0) {
                const float co[4] = {q.cs01.x, q.cs01.z, q.cs23.x, q.cs23.z};
                const float si[4] = {q.cs01.y, q.cs01.w, q.cs23.y, q.cs23.w};
                const float pv[4] = {partner.x, partner.y, partner.z, partner.w};
                const float sgn = (f % hd) < half ? -1.0f : 1.0f;   // first half: a c - b s; second half: b c + a s
#pragma unroll
                for (int e = 0; e < 4; ++e) v[e] = v[e] * co[e] + sgn * pv[e] * si[e];
            }
            if (f < qd) {
                if (pos < 0) { v[0] = v[1] = v[2] = v[3] = 0.f; }
                *reinterpret_cast<float4*>(a.qbuf + (size_t)m * qd + f) = make_float4(v[0], v[1], v[2], v[3]);
            } else if (f < qd + 2 * kvd && pos >= 0 && q.page >= 0) {
                const bool is_k = f < qd + kvd;
                const int gidx = f - qd - (is_k ? 0 : kvd);
                const int kh = gidx / hd, i = gidx % hd;
                __nv_bfloat16* base = is_k ? a.k_pages : a.v_pages;
                store_bf16x4(base + (((size_t)q.page * a.n_kv + kh) * a.page_size + pos % a.page_size) * hd + i, v);
            }
        } else if (EPI == EPI_RESID) {
            const int f = f0 + 4 * lane;
            float ss = 0.f;
            if (f < a.N) {
                const float4 xv = make_float4(q.x.x + acc.x, q.x.y + acc.y, q.x.z + acc.z, q.x.w + acc.w);
                *reinterpret_cast<float4*>(a.x + (size_t)m * a.N + f) = xv;
                ss = xv.x * xv.x + xv.y * xv.y + xv.z * xv.z + xv.w * xv.w;
                const float v[4] = {xv.x * gain4.x, xv.y * gain4.y, xv.z * gain4.z, xv.w * gain4.w};
                const size_t row = (size_t)(m / TBL) * (2 * TBL) + m % TBL;
                store_hilo4(a.a_out + row * a.N + f, a.a_out + (row + TBL) * a.N + f, v);
            }
            ss = warp_sum(ss);
            if (lane == 0) {
                float* slot = a.ssq_out + (size_t)m * a.ssq_out_slots + (size_t)out_tile * a.ssq_sub;
                slot[0] = ss;
                for (int j = 1; j < a.ssq_sub; ++j) slot[j] = 0.f;
            }
        } else if (EPI == EPI_SWIGLU) {
            const float sc = s_inv[t];
            // lanes 0-15 hold four gate features each, lanes 16-31 the matching up features: after the exchange both
            // lanes of a pair have all eight values, and each finishes two of the four outputs
            const float4 oth = shfl_xor4(acc, 16);
            const bool low = lane < 16;
            const float4 g4 = low ? acc : oth, u4 = low ? oth : acc;
            const int j = f0 + 4 * (lane & 15) + (low ? 0 : 2);
            if (j < a.N) {                                       // d_ff is a multiple of 8: j + 1 < N as well
                const float g0 = (low ? g4.x : g4.z) * sc, g1 = (low ? g4.y : g4.w) * sc;
                const float u0 = (low ? u4.x : u4.z) * sc, u1 = (low ? u4.y : u4.w) * sc;
                const float v0 = g0 / (1.0f + expf(-g0)) * u0, v1 = g1 / (1.0f + expf(-g1)) * u1;
                __nv_bfloat16 h0, l0, h1, l1;
                split_bf16(v0, h0, l0);
                split_bf16(v1, h1, l1);
                const size_t row = (size_t)(m / TBL) * (2 * TBL) + m % TBL;
                *reinterpret_cast<uint32_t*>(a.a_out + row * a.N + j) =
                    (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                *reinterpret_cast<uint32_t*>(a.a_out + (row + TBL) * a.N + j) =
                    (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
            }
        }
    };
    Pre pf[NPF];
    // Where the epilogue's operands were complete before the preceding grid began (a.early: the row plan, rotary
    // table and page ids of a QKV launch that does not follow the row-plan kernel; the residual rows and gain of a
    // RESID launch), they are requested ahead of griddepcontrol.wait, otherwise after it.
    auto late_prefetch = [&]() {
        if (EPI != EPI_LM) {
#pragma unroll
            for (int i = 0; i < NPF; ++i)
                if (warp + EW * i < count) pf[i] = prefetch(warp + EW * i);
            if (EPI == EPI_RESID && f0 + 4 * lane < a.N) gain4 = *reinterpret_cast<const float4*>(a.gain + f0 + 4 * lane);
        }
    };

    if (warp == 4) {
        if (lane == 0) {
            s_fail = 0;
            for (int s = 0; s < stages; ++s) {
                mbar_init(bar_full + 8u * s, 1);
                mbar_init(bar_empty + 8u * s, 1);
            }
            mbar_init(bar_acc, 1);
            fence_barrier_init();
            tma_prefetch_desc(&tmW);
            tma_prefetch_desc(&tmX);
        }
        __syncwarp();
        // The weights of the first stages depend on no earlier kernel: their loads start before the rest of
        // the CTA is set up and before the preceding grid has finished.  One lane per stage: a lane that has
        // issued its copy does not wait for the others'.
        if (lane < pre) {
            const uint32_t dstA = smem_u32(smem + (size_t)lane * stage_bytes);
            mbar_expect_tx_only(bar_full + 8u * lane, A_STAGE_BYTES);
            load_w(lane, dstA, bar_full + 8u * lane);
        }
        if (lane == 0) TL(1);
        __syncwarp();
    } else if (warp == 5) {
        tmem_alloc(smem_u32(tmem_slot), ncols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) TL(0);

    if (warp == 4) {
        // ------------------------------------------------------------ TMA producer
        if (a.early) late_prefetch();
        griddep_wait();                 // every lane: the token rows below, and the epilogue operands later
        if (lane < pre) {
            const uint32_t dstB = smem_u32(smem + (size_t)lane * stage_bytes) + A_STAGE_BYTES;
            mbar_expect_tx(bar_full + 8u * lane, b_stage_bytes);
            tma_load_2d_hint(dstB, &tmX, (kb_begin + lane) * BK, m0, bar_full + 8u * lane, pol_x);
        }
        __syncwarp();
        if (lane == 0) {
            TL(2);
            for (int i = pre; i < n_kb; ++i) {
                const int s = i % stages;
                const uint32_t round = (uint32_t)(i / stages);
                if (!mbar_wait(bar_empty + 8u * s, (round & 1u) ^ 1u)) { fail(); break; }
                const uint32_t dstA = smem_u32(smem + (size_t)s * stage_bytes);
                mbar_expect_tx(bar_full + 8u * s, stage_bytes);
                load_w(i, dstA, bar_full + 8u * s);
                tma_load_2d_hint(dstA + A_STAGE_BYTES, &tmX, (kb_begin + i) * BK, m0, bar_full + 8u * s, pol_x);
            }
            griddep_launch_dependents();
            TL(3);
        }
        __syncwarp();
        if (!a.early) late_prefetch();
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issue
        if (a.early) late_prefetch();
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_f32(BM, BN);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % stages;
                const uint32_t round = (uint32_t)(i / stages);
                if (!mbar_wait(bar_full + 8u * s, round & 1u)) { fail(); ok = false; break; }
                if (i == 0) TL(4);
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
                for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                    const uint64_t da = umma_desc_k_sw128(sa + kk * UMMA_K * 2);
                    const uint64_t db = umma_desc_k_sw128(sb + kk * UMMA_K * 2);
                    umma_bf16(tmem_base, da, db, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar_empty + 8u * s);
            }
            if (ok) umma_commit(bar_acc);
            TL(5);
        }
        __syncwarp();
        griddep_wait();
        if (!a.early) late_prefetch();
    } else if (warp >= 6) {
        // ------------------------------------------------------------ the additional column finishers: nothing to do before part 2
        if (a.early) late_prefetch();
        griddep_wait();
        if (!a.early) late_prefetch();
    } else {
        // ------------------------------------------------------------ epilogue, part 1: accumulator -> shared memory
        if (a.early) late_prefetch();
        griddep_wait();
#ifdef TASC_TIMELINE
        if (threadIdx.x == 0) g_ta = global_ns();
#endif
        if (!a.early) late_prefetch();
        if (EPI == EPI_QKV || EPI == EPI_SWIGLU || EPI == EPI_LM || (EPI == EPI_PLAIN && a.ssq_in)) {
            for (int t = threadIdx.x; t < TB; t += 128) {
                const int m = t0 + t;
                float ss = 0.f;
                if (m < a.M)
                    for (int j = 0; j < a.ssq_slots; ++j) ss += a.ssq_in[(size_t)m * a.ssq_slots + j];
                s_inv[t] = 1.0f / sqrtf(ss * a.inv_d + a.eps);
            }
        }
        bool have = n_kb > 0;
        if (have && !mbar_wait(bar_acc, 0)) { fail(); have = false; }
        if (threadIdx.x == 0) TL(6);
#ifdef TASC_TIMELINE
        if (threadIdx.x == 0) g_tb = global_ns();
#endif
        tc_fence_after();
        asm volatile("bar.sync 1, 128;" ::: "memory");          // s_inv visible to the four epilogue warps
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        const int fl = warp * 32 + lane;                        // this thread's feature (TMEM lane) within the tile
        // accumulator columns of layout tile lt: [lt * 2 TBL, +TBL) from the hi rows, the next TBL from the lo rows
        for (int lt = 0; lt * TBL < TB; ++lt) {
            const uint32_t col0 = (uint32_t)(lt * 2 * TBL);
            for (int c = 0; c < TBL; c += 32) {
                const bool wide = c + 32 <= TBL;                // TBL is a multiple of 16
                uint32_t r[32];
                if (have) {
                    if (wide) {
                        uint32_t r2[32];
                        tmem_ld32(lane_base + col0 + (uint32_t)c, r);
                        tmem_ld32(lane_base + col0 + (uint32_t)(TBL + c), r2);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                    } else {
                        uint32_t q[16], q2[16];
                        tmem_ld16(lane_base + col0 + (uint32_t)c, q);
                        tmem_ld16(lane_base + col0 + (uint32_t)(TBL + c), q2);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(q[j]) + __uint_as_float(q2[j]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (j < 16 || wide) xch[(lt * TBL + c + j) * BM + fl] = __uint_as_float(r[j]);
            }
        }
    }
    if (threadIdx.x == 0) TL(7);
#ifdef TASC_TIMELINE
    if (threadIdx.x == 0) g_tc = global_ns();
#endif
    tc_fence_before();
    // every CTA's partial tile is in its shared memory (release / acquire at cluster scope)
    cluster_arrive();
    cluster_wait();
    if (threadIdx.x == 0) TL(8);
#ifdef TASC_TIMELINE
    if (threadIdx.x == 0) g_td = global_ns();
#endif

    if (EPI != EPI_LM) {
        // ------------------------------------------------------------ epilogue, part 2: sum the S partial copies of this CTA's columns
        if (S > 1) {
            // pull: all S remote reads of a column are issued before the first is used, then added in rank order
            const uint32_t xch_addr = smem_u32(xch) + (uint32_t)(lane * 16);
            uint32_t peer[8];
#pragma unroll
            for (int s = 0; s < 8; ++s) peer[s] = cluster_map(xch_addr, (uint32_t)(s < S ? s : 0));
            for (int tl = warp; tl < count; tl += 2 * EW) {       // two columns per round: 2 S reads in flight
                const bool two = tl + EW < count;
                const uint32_t toff0 = (uint32_t)(rank * per + tl) * (BM * 4), toff1 = toff0 + (uint32_t)EW * (BM * 4);
                float4 p0[8], p1[8];
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    if (s < S) {
                        p0[s] = ld_cluster_f4(peer[s] + toff0);
                        if (two) p1[s] = ld_cluster_f4(peer[s] + toff1);
                    }
                float4 a0 = p0[0], a1 = p1[0];
#pragma unroll
                for (int s = 1; s < 8; ++s)
                    if (s < S) {
                        a0.x += p0[s].x; a0.y += p0[s].y; a0.z += p0[s].z; a0.w += p0[s].w;
                        a1.x += p1[s].x; a1.y += p1[s].y; a1.z += p1[s].z; a1.w += p1[s].w;
                    }
                *reinterpret_cast<float4*>(fin + (size_t)tl * BM + 4 * lane) = a0;      // read back by the same lane below
                if (two) *reinterpret_cast<float4*>(fin + (size_t)(tl + EW) * BM + 4 * lane) = a1;
            }
        }
    }
#ifdef TASC_TIMELINE
    if (threadIdx.x == 0) g_te = global_ns();
#endif
    // this CTA has finished reading its peers' shared memory; they may leave while it runs the epilogue
    cluster_arrive();
    if (EPI != EPI_LM) {
#pragma unroll
        for (int i = 0; i < NPF; ++i)
            if (warp + EW * i < count) finish(warp + EW * i, pf[i]);
        for (int tl = warp + EW * NPF; tl < count; tl += EW) finish(tl, prefetch(tl));
    } else {
        // LM head: per token row the largest logit of this 128-feature tile (smallest id on ties), merged
        // across tiles by an atomic max on the packed (value, id) word; the logits themselves are not stored
        // (two token rows per round: their reductions are independent and overlap)
        const int f = f0 + 4 * lane;
        for (int tb = warp; tb < valid; tb += 2 * EW) {
            float4 acc[2];
            uint32_t bk[2], bi[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int t = tb + u * EW;
                acc[u] = t < valid ? *reinterpret_cast<const float4*>(xch + (size_t)t * BM + 4 * lane) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const float v[4] = {acc[u].x, acc[u].y, acc[u].z, acc[u].w};
                // largest key of the warp's 128 features, then the smallest id that has it: two warp-wide reductions
                bk[u] = 0u; bi[u] = 0xFFFFFFFFu;
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (f + e < a.N) {
                        const uint32_t k = float_key(v[e]);
                        if (bi[u] == 0xFFFFFFFFu || k > bk[u]) { bk[u] = k; bi[u] = (uint32_t)(f + e); }
                    }
            }
            uint32_t mk[2], id[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) mk[u] = __reduce_max_sync(0xFFFFFFFFu, bk[u]);
#pragma unroll
            for (int u = 0; u < 2; ++u) id[u] = __reduce_min_sync(0xFFFFFFFFu, (bk[u] == mk[u]) ? bi[u] : 0xFFFFFFFFu);
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int t = tb + u * EW;
                if (t >= valid) continue;
                if (lane == 0 && id[u] != 0xFFFFFFFFu)
                    atomicMax(&a.argmax[t0 + t], ((unsigned long long)mk[u] << 32) | (unsigned long long)(0xFFFFFFFFu - id[u]));
                if (a.logits) {
                    const float sc = s_inv[t];
                    const float v[4] = {acc[u].x, acc[u].y, acc[u].z, acc[u].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (f + e < a.N) a.logits[(size_t)(t0 + t) * a.N + f + e] = v[e] * sc;
                }
            }
        }
    }
    if (threadIdx.x == 0) TL(9);
#ifdef TASC_TIMELINE
    if (threadIdx.x == 0) g_tf = global_ns();
#endif
    // peers may still be reading this CTA's partial tile
    cluster_wait();
    if (s_fail && warp == 4 && lane == 0) {
        // after a timeout: give this CTA's own tile loads that may still be in flight a bounded time to land
        for (int i = 0; i < n_kb; ++i) {
            const int s = i % stages;
            if (i + stages >= n_kb) (void)mbar_wait(bar_full + 8u * s, (uint32_t)(i / stages) & 1u, 2000000ll);
        }
    }
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, ncols);
    }
    if (threadIdx.x == 0) TL(10);
#ifdef TASC_TIMELINE
    if (threadIdx.x == 0) ctalog_put(g_t0, g_ta, g_tb, EPI, g_tc, g_td, g_te, g_tf);
#endif
}

template <int EPI>
tasc_status prepare_epi() {
    static bool attr_done[64] = {false};
    int dev = 0;
    TASC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return TASC_EINVAL;
    if (!attr_done[dev]) {
        TASC_CUDA_TRY(cudaFuncSetAttribute(gemm_fused_kernel<EPI, 6>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN_SMEM));
        TASC_CUDA_TRY(cudaFuncSetAttribute(gemm_fused_kernel<EPI, 12>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN_SMEM));
        attr_done[dev] = true;
    }
    return TASC_OK;
}

// Clusters of S CTAs with `smem` bytes each that the device can hold at once (0 if the query fails).
template <int EPI>
int max_active_clusters(int S, int smem) {
    if (prepare_epi<EPI>() != TASC_OK) return 0;
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
    if (cudaOccupancyMaxActiveClusters(&n, gemm_fused_kernel<EPI, 6>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

int max_active_clusters_any(int epi, int S, int smem) {
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
        case EPI_PLAIN:  n = max_active_clusters<EPI_PLAIN>(S, smem); break;
        case EPI_QKV:    n = max_active_clusters<EPI_QKV>(S, smem); break;
        case EPI_RESID:  n = max_active_clusters<EPI_RESID>(S, smem); break;
        case EPI_SWIGLU: n = max_active_clusters<EPI_SWIGLU>(S, smem); break;
        case EPI_LM:     n = max_active_clusters<EPI_LM>(S, smem); break;
        default: break;
    }
    cache[key] = n;
    return n;
}

template <int EPI>
tasc_status launch_epi(const CUtensorMap* tmW, const CUtensorMap* tmX, const FusedArgs& a, const FusedPlan& p, int kind,
                       cudaStream_t stream) {
    tasc_status pst = prepare_epi<EPI>();
    if (pst != TASC_OK) return pst;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.S, (unsigned)p.out_tiles, (unsigned)p.m_tiles);
    cfg.blockDim = dim3((unsigned)(p.threads == MAX_THREADS ? MAX_THREADS : THREADS), 1, 1);
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
    if (p.threads == MAX_THREADS) TASC_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_fused_kernel<EPI, 12>, *tmW, *tmX, a));
    else TASC_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_fused_kernel<EPI, 6>, *tmW, *tmX, a));
    return TASC_OK;
}

}  // namespace

FusedPlan plan_fused(int M, int N, int K, int epi, int few_tiles, int hd, double wide_min_mb) {
    FusedPlan p = {};
    const bool many_rows = wide_min_mb >= 0.0 && M > 128;
    const double mb = 2.0 * (double)(epi == EPI_SWIGLU ? 2 * N : N) * (double)K / 1e6;
    // (from 512 rows on, matrices of a little more than half that size gain as well)
    if (many_rows && (mb >= wide_min_mb || (M >= 512 && mb >= 0.55 * wide_min_mb)) && plan_wide(M, N, K, epi, hd, p)) return p;
    p = {};
    p.TBL = gemm_token_tile(M, true, few_tiles, many_rows);
    // The LM head of a pass of 97 .. 128 rows in one token tile: the largest matrix of the model is tensor-bound there
    // (2 V d_model x 128 lanes x 2 passes), and the few-row kernel's 128-row weight tiles stream it at half the rate the
    // many-row kernel reaches (measured on the 1.5B shape at 112 rows: 140 -> 85 us).
    if (epi == EPI_LM && !many_rows && M > 96 && M <= 128 && p.TBL >= M && mb >= LM_WIDE_MIN_MB) {
        FusedPlan w = {};
        if (plan_wide(M, N, K, epi, hd, w, p.TBL)) return w;
    }
    // The LM head streams the largest matrix once and has no split-K exchange: one CTA takes as many layout tiles
    // as an MMA holds (256 columns), so that a weight tile is fetched by one CTA, not by one per token tile.
    const int span = epi == EPI_LM ? std::max(1, std::min((M + p.TBL - 1) / p.TBL, 128 / p.TBL)) : 1;
    p.TB = span * p.TBL;
    p.BN = 2 * p.TB;
    p.m_tiles = (M + p.TB - 1) / p.TB;
    p.out_tiles = epi == EPI_SWIGLU ? (N + 63) / 64 : (N + BM - 1) / BM;
    p.num_kb = (K + BK - 1) / BK;
    const int tiles = p.out_tiles * p.m_tiles;
    int S = 1;
    if (epi != EPI_LM) {
        S = std::max(1, 148 / tiles);
        S = std::min(S, 8);
        S = std::min(S, p.num_kb);
        // Fewer splits than fit can be faster.  Per kernel, in microseconds as measured on the 576- and 1536-wide
        // products: a CTA's MMA chain takes about 0.46 per k-block; its epilogue about 0.5 per round of six token
        // columns (one per warp) of the columns it finishes; and a grid that takes more than about two thirds of
        // the SMs keeps the next kernel's CTAs from starting (and from fetching their weights) while this one
        // runs, about 0.035 per CTA beyond 96.  Ties go to the larger cluster.
        // (With a single token tile the chain's kernels are narrow and the largest cluster stays the best.)
        const int cols = std::min(p.TB, M);
        int best = S;
        float best_cost = 1e30f;
        for (int s = 1; s <= S && p.m_tiles >= 2; ++s) {
            const int ctas = tiles * s;
            const int rounds = ((cols + s - 1) / s + 5) / 6;
            const float cost = 0.46f * (float)((p.num_kb + s - 1) / s) + 0.5f * (float)rounds +
                               0.035f * (float)std::max(0, ctas - 96) - 0.01f * (float)s;
            if (cost < best_cost) { best_cost = cost; best = s; }
        }
        S = best;
    }
    const int stage_bytes = A_STAGE_BYTES + p.BN * BK * 2;
    int ncols = 32;
    while (ncols < p.BN) ncols <<= 1;
    // the CTA's partial tile for the split-K exchange, not aliased with the ring (the LM head reuses the ring)
    const int xch_bytes = epi == EPI_LM ? 0 : p.TB * BM * 4;
    for (;; --S) {
        p.S = S;
        const int kb_per = (p.num_kb + S - 1) / S;
        // A CTA's streaming rate is its bytes in flight over the memory latency.  A grid of one wave (at most
        // one CTA per SM anyway) gets a ring of up to 200 KB; a grid of several waves keeps about 100 KB per
        // CTA so that two CTAs share an SM and cover each other's start-up and epilogue.
        const bool one_wave = tiles * S <= 148;
        const int budget = ((ncols <= 128 || epi == EPI_LM) && !one_wave ? 108 * 1024 : 216 * 1024) - xch_bytes;
        int st = budget / stage_bytes;
        st = std::max(2, std::min(st, 8));
        st = std::min(st, std::max(2, kb_per));
        p.stages = st;
        p.data_bytes = std::max(st * stage_bytes, p.TB * BM * 4) + xch_bytes;
        int smem = 1024 + p.data_bytes + (2 * st + 2) * 8 + 128 * 4;
        // TMEM columns held by co-resident CTAs must never exceed 512, or CTAs of different clusters can
        // block each other's allocation while waiting at a cluster barrier: shared memory limits residency.
        // (The LM head has no cluster barrier to wait at; two of its CTAs with 256 columns each share an SM.)
        if (epi != EPI_LM) smem = std::max(smem, ncols * 454 + 1);
        p.smem_bytes = std::min(smem, MAX_DYN_SMEM);
        if (S == 1) break;
        // All clusters of the grid should be resident at once: a second, nearly empty wave doubles the
        // kernel's time.  (Clusters occupy whole groups of SMs inside a GPC, so fewer fit than SMs / S.)
        const int fit = max_active_clusters_any(epi, S, p.smem_bytes);
        if (fit <= 0 || tiles <= fit) break;
    }
    // token columns a CTA reduces and finishes after the cluster exchange
    const int cols_cta = (std::min(p.TB, M) + p.S - 1) / p.S;
    // (only for grids of one wave: with two CTAs per SM the schedulers have warps enough, and twelve warps of 100 to 126
    // registers would not leave room for the second CTA)
    p.threads = (epi != EPI_LM && epi != EPI_PLAIN && cols_cta >= FINISHERS_MIN_COLS && tiles * p.S <= 148) ? MAX_THREADS : THREADS;
    return p;
}

tasc_status launch_gemm_fused(int epi, const CUtensorMap* tmW, const CUtensorMap* tmX, FusedArgs a, const FusedPlan& p,
                              cudaStream_t stream) {
    if (a.M <= 0 || a.N <= 0 || a.K <= 0) return TASC_EINVAL;
    if (p.wide) return launch_gemm_wide(epi, tmW, tmX, a, p, stream);
    a.num_kb = p.num_kb; a.BN = p.BN; a.TB = p.TB; a.TBL = p.TBL; a.stages = p.stages; a.pair = 1; a.data_bytes = p.data_bytes;
    switch (epi) {
        case EPI_PLAIN:  return launch_epi<EPI_PLAIN>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_QKV:    return launch_epi<EPI_QKV>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_RESID:  return launch_epi<EPI_RESID>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_SWIGLU: return launch_epi<EPI_SWIGLU>(tmW, tmX, a, p, K_GEMM, stream);
        case EPI_LM:     return launch_epi<EPI_LM>(tmW, tmX, a, p, K_GEMM_LM, stream);
        default: return TASC_EINVAL;
    }
}

#ifdef TASC_TIMELINE
__device__ CtaRec g_ctalog[1 << 18];
__device__ unsigned int g_ctalog_n;
extern "C" int tasc_debug_ctalog(void* out, int max_recs, int reset) {
    unsigned int n = 0;
    if (cudaMemcpyFromSymbol(&n, g_ctalog_n, sizeof(n)) != cudaSuccess) return -1;
    if (n > (1u << 18)) n = 1u << 18;
    if ((int)n > max_recs) n = (unsigned int)max_recs;
    if (n && cudaMemcpyFromSymbol(out, g_ctalog, (size_t)n * sizeof(CtaRec)) != cudaSuccess) return -1;
    if (reset) { const unsigned int z = 0; cudaMemcpyToSymbol(g_ctalog_n, &z, sizeof(z)); }
    return (int)n;
}
extern "C" int tasc_debug_timeline(long long* out, int n_ctas) {
    return (int)cudaMemcpyFromSymbol(out, g_timeline, (size_t)n_ctas * 16 * sizeof(long long));
}
#endif

}  // namespace tasc
