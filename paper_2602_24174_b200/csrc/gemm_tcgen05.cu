// General-purpose bf16 GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA, with split-K
// partial sums in global memory: the exported building block (tasc_gemm_bf16, tasc_gemm_bf16_static).
// The verify forward itself runs the fused variant in gemm_fused.cu, which shares this kernel's operand
// layout and pipeline but reduces split-K inside a cluster and fuses the consumer stage.
//
// Operands are swapped: the weight tile supplies the 128 rows of the MMA (UMMA M = 128), the token rows
// are the MMA's N (16..256); D^T[128 weight rows][BN tokens] accumulates in TMEM in float32.  Each CTA
// streams a [128 x k-range] slab of W through a multi-stage TMA -> shared-memory ring; split-K spreads a
// matrix with few row tiles over all SMs and the slices are added in fixed order afterwards.
//
// Warp roles (192 threads): warps 0-3 epilogue (TMEM lanes 32w..32w+31), warp 4 TMA producer,
// warp 5 TMEM allocation + MMA issue.  Every wait is bounded; on timeout the CTA records
// TASC_ETIMEOUT, skips the remaining work, releases TMEM and returns.
#include "kernels.h"

#include <algorithm>
#include <mutex>

namespace tasc {

namespace {

constexpr int BM = 128;           // weight rows per tile (UMMA M)
constexpr int BK = 64;            // k elements per stage: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int GEMM_THREADS = 192;

struct GemmArgs {
    float* partials;
    int M, N, K;
    int num_kb, splits, m_tiles, BN, stages;
    int pair;                       // 1: columns j and j + BN/2 of the accumulator belong to the same token
    int* status;
};

__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const GemmArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);

    const int BN = a.BN, stages = a.stages;
    const uint32_t b_stage_bytes = (uint32_t)BN * BK * 2;
    const uint32_t stage_bytes = A_STAGE_BYTES + b_stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8u * stages;
    const uint32_t bar_acc = bar_full + 16u * stages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * stages + 1);

    int bid = blockIdx.x;
    const int m_tile = bid % a.m_tiles; bid /= a.m_tiles;
    const int split = bid % a.splits;
    const int out_tile = bid / a.splits;
    const int kb_begin = (int)(((long long)a.num_kb * split) / a.splits);
    const int kb_end = (int)(((long long)a.num_kb * (split + 1)) / a.splits);
    const int n_kb = kb_end - kb_begin;
    const int f0 = out_tile * BM;       // first weight row (output feature) of the tile
    const int m0 = m_tile * BN;         // first row of the tile in the activation buffer
    const int TBk = a.pair ? BN / 2 : BN;   // tokens per tile
    const int t0 = m_tile * TBk;        // first token of the tile

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t ncols = 32;
    while ((int)ncols < BN) ncols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, 1);
        }
        mbar_init(bar_acc, 1);
        fence_barrier_init();
    }
    if (warp == 4 && lane == 0) {
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
    }
    if (warp == 5) {
        tmem_alloc(smem_u32(tmem_slot), ncols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();   // weights are read once per step
            const uint64_t pol_x = policy_evict_last();    // the token rows are re-read by every CTA
            for (int i = 0; i < n_kb; ++i) {
                const int s = i % stages;
                const uint32_t round = (uint32_t)(i / stages);
                if (!mbar_wait(bar_empty + 8u * s, (round & 1u) ^ 1u)) { set_status(a.status, TASC_ETIMEOUT); break; }
                const uint32_t dstA = smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t dstB = dstA + A_STAGE_BYTES;
                mbar_expect_tx(bar_full + 8u * s, stage_bytes);
                const int kc = (kb_begin + i) * BK;
                tma_load_2d_hint(dstA, &tmW, kc, f0, bar_full + 8u * s, pol_w);
                tma_load_2d_hint(dstB, &tmX, kc, m0, bar_full + 8u * s, pol_x);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issue
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_f32(BM, BN);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % stages;
                const uint32_t round = (uint32_t)(i / stages);
                if (!mbar_wait(bar_full + 8u * s, round & 1u)) { set_status(a.status, TASC_ETIMEOUT); ok = false; break; }
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
                for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                    const uint64_t da = umma_desc_k_sw128(sa + kk * UMMA_K * 2);
                    const uint64_t db = umma_desc_k_sw128(sb + kk * UMMA_K * 2);
                    umma_bf16(tmem_base, da, db, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar_empty + 8u * s);     // frees the stage once these MMAs have read it
            }
            if (ok) umma_commit(bar_acc);            // accumulator complete
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 0..3)
        bool have = n_kb > 0;
        if (have) {
            if (!mbar_wait(bar_acc, 0)) { set_status(a.status, TASC_ETIMEOUT); have = false; }
        }
        tc_fence_after();
        const int f = f0 + warp * 32 + lane;
        const bool f_ok = f < a.N;
        for (int c = 0; c < TBk / 16; ++c) {
            uint32_t r[16];
            if (have) {
                const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
                tmem_ld16(lane_base + (uint32_t)(c * 16), r);
                if (a.pair) {
                    uint32_t r2[16];
                    tmem_ld16(lane_base + (uint32_t)(TBk + c * 16), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                } else {
                    tmem_ld_wait();
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) r[j] = 0u;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int m = t0 + c * 16 + j;
                if (f_ok && m < a.M) a.partials[((size_t)split * a.M + m) * a.N + f] = __uint_as_float(r[j]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem_base, ncols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    });
    return fn;
}

int stage_bytes_for(int BN) { return A_STAGE_BYTES + BN * BK * 2; }
int smem_for(int BN, int stages) { return 1024 + stages * stage_bytes_for(BN) + (2 * stages + 2) * 8; }

}  // namespace

tasc_status encode_tmap_bf16(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return TASC_ECUDA;
    if ((reinterpret_cast<uintptr_t>(ptr) & 15u) || (cols % 8u) || box_rows == 0 || box_rows > 256) return TASC_EINVAL;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TASC_OK : TASC_ECUDA;
}

tasc_status encode_tmap_kv(CUtensorMap* map, const void* ptr, uint64_t rows, int hd) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return TASC_ECUDA;
    if ((reinterpret_cast<uintptr_t>(ptr) & 15u) || (hd != 32 && hd != 64 && hd != 128) || rows == 0) return TASC_EINVAL;
    cuuint64_t dims[2] = {(cuuint64_t)hd, rows};
    cuuint64_t strides[1] = {(cuuint64_t)hd * 2};
    cuuint32_t box[2] = {(cuuint32_t)(hd < 64 ? hd : 64), 16};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, hd < 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TASC_OK : TASC_ECUDA;
}

int gemm_token_tile(int M, bool pair, int few_tiles, bool many_rows) {
    const int cap = pair ? 128 : 256;                 // tokens per tile (UMMA N <= 256)
    int m_tiles = (M + cap - 1) / cap;
    // An MMA over a 128-row weight tile takes the same time for any number of token columns, while the split-K
    // exchange, the accumulator read-out and the epilogue of a CTA grow with its columns -- and every token tile
    // streams the weight tile again.  Which wins depends on the size of the weights: for narrow models (a few MB per
    // layer) three or more token tiles per weight tile run faster than one or two wide ones above 48 rows (measured at
    // 96, 192 and 448 rows); for a 94 MB layer one tile of 112 rows beats three of 48 by 20 % of the step, and in
    // between two tiles are slightly ahead.  The caller passes the count for 49..128 rows (few_tiles).  Above 128 rows
    // it stays at three or more -- unless the pass runs its large products through the many-row kernel (gemm_wide.cu),
    // where the token rows are the MMA's M (many_rows): then as few tiles of at most 128 rows as hold them.
    if (pair && M > 48 && M <= 128) m_tiles = std::max(m_tiles, std::max(1, std::min(few_tiles, 3)));
    if (pair && M > 128 && !many_rows) m_tiles = std::max(m_tiles, 3);
    const int per = (M + m_tiles - 1) / m_tiles;
    return std::max(16, (per + 15) / 16 * 16);
}

GemmPlan plan_gemm(int M, int N, int K, size_t max_partial_bytes, bool pair) {
    GemmPlan p;
    p.pair = pair ? 1 : 0;
    p.TB = gemm_token_tile(M, pair);
    p.BN = pair ? 2 * p.TB : p.TB;
    p.m_tiles = (M + p.TB - 1) / p.TB;
    p.out_tiles = (N + BM - 1) / BM;
    const int num_kb = (K + BK - 1) / BK;
    const int tiles = p.out_tiles * p.m_tiles;
    // Enough CTAs to cover the 148 SMs about twice, each keeping at least two k-blocks.
    int s = std::max(1, (296 + tiles / 2) / tiles);
    s = std::min(s, std::max(1, num_kb / 2));
    while (s > 1 && (size_t)s * M * N * sizeof(float) > max_partial_bytes) --s;
    p.splits = s;
    const int kb_per = (num_kb + s - 1) / s;
    // Two CTAs per SM when the tile is small (about 110 KB each), otherwise one deep ring.
    const int budget = p.BN <= 64 ? 100 * 1024 : 190 * 1024;
    int st = budget / stage_bytes_for(p.BN);
    st = std::max(2, std::min(st, 8));
    st = std::min(st, std::max(2, kb_per));
    p.stages = st;
    p.smem_bytes = smem_for(p.BN, st);
    return p;
}

tasc_status gemm_set_attributes() {
    TASC_CUDA_TRY(cudaFuncSetAttribute(gemm_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    return TASC_OK;
}

tasc_status launch_gemm_bf16(const CUtensorMap* tmW, const CUtensorMap* tmX, float* partials, int M, int N, int K,
                             const GemmPlan& plan, int* status, cudaStream_t stream) {
    if (M <= 0 || N <= 0 || K <= 0) return TASC_EINVAL;
    GemmArgs a;
    a.partials = partials; a.M = M; a.N = N; a.K = K;
    a.num_kb = (K + BK - 1) / BK; a.splits = plan.splits; a.m_tiles = plan.m_tiles; a.BN = plan.BN; a.stages = plan.stages; a.pair = plan.pair;
    a.status = status;
    const int grid = plan.out_tiles * plan.splits * plan.m_tiles;
    ProfScope ps(K_GEMM, stream);
    gemm_bf16_kernel<<<grid, GEMM_THREADS, plan.smem_bytes, stream>>>(*tmW, *tmX, a);
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

}  // namespace tasc
