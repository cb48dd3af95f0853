// Verify attention for bf16 models on the warp-level tensor-core path: the R = k+1 new query rows of a
// sequence times the g query heads that share one KV head (G = g * R rows) against the paged KV cache.
//
// The kernel is bound by streaming K and V from HBM once; the tensor cores only have to keep up with
// that stream, which a float32 SIMT formulation cannot do beyond a few sequences.  A CTA owns one
// (sequence, KV head, key range): the key range of a sequence is split over several CTAs because the
// batch alone cannot fill 148 SMs.  K/V tiles of 64 keys arrive through a ring of 2-8 stages in swizzled shared
// memory: one TMA box load per 16-token page (every page of a KV head is one contiguous run), issued by one
// thread and signalled on an mbarrier; pools with another page size use 16-byte cp.async copies instead;
// warp w computes the 16-row slab w of S = Q K^T and O += P V with mma.sync m16n8k16 (ldmatrix
// fragments, V through ldmatrix.trans) and keeps an online softmax per row in registers.
//
// Precision: K and V are bf16 as stored.  Q (pre-scaled by log2(e) / sqrt(head_dim)) and the
// probabilities P are float32 values carried as hi + lo bf16 pairs, two MMAs each, so the only rounding
// in the attention is the KV cache's own.  Softmax statistics and O are float32.
//
// Merge (only when the key range is split): the splits of one (sequence, KV head) are the CTAs of a
// thread-block cluster.  Each parks its unnormalised O and (max, sum) in its shared memory; after a cluster
// barrier CTA r merges every S-th row from the S copies (distributed shared memory reads, rank order) and
// writes it as (hi, lo) bf16 in the layout the O-projection GEMM loads.  Nothing goes through global memory.
#include "kernels.h"

#include <algorithm>
#include <cstring>
#include <map>
#include <mutex>

namespace tasc {

namespace {

constexpr int TKEYS = 64;

struct AttnArgs {
    const float* q;                    // [M][n_q * hd], RoPE applied
    const __nv_bfloat16* kp;
    const __nv_bfloat16* vp;
    const int32_t* block_table;
    int max_pages, page_size;
    long long n_pages;
    const int* seq_pos0;
    const int* seq_rows;
    __nv_bfloat16* out;                // (hi, lo) activation buffer, row length n_q * hd
    int TB;
    int R, n_q, n_kv, splits, stages;  // R: rows per sequence in this pass
    int Rs, n_sub;                     // a CTA takes Rs of them (sub-block blockIdx.z % n_sub); R = Rs * n_sub
    int hs, n_hsplit;                  // a CTA takes hs of the g query heads of its KV head (blockIdx.y % n_hsplit); g = hs * n_hsplit
    int use_tma;                       // K/V tiles by TMA box loads (16-token pages); otherwise by cp.async
    int* status;
    float scale_log2e;
};

// Byte offset of 16-byte chunk `chunk` of row `row` in a 64-row bf16 tile (the Q tile: ROWS rows).  The layout is
// the one a TMA box load with hardware swizzling produces, so that K/V tiles can arrive either way: rows of at most
// 128 bytes (head_dim 128 = two column halves of 64, stored one after the other), 16-byte chunks XOR-ed with the
// row index (128-byte swizzle; 64-byte swizzle for head_dim 32).  The XOR also keeps the eight rows of an ldmatrix
// phase on distinct banks.  Tile bases are 1024-byte aligned.
template <int HD, int ROWS = 64>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    if (HD == 128) return (uint32_t)((chunk >> 3) * (ROWS * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
    if (HD == 64) return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4));
    return (uint32_t)(row * 64 + ((chunk ^ ((row >> 1) & 3)) << 4));
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// two floats -> packed bf16 pair (hi) and the packed pair of the residuals (lo)
__device__ __forceinline__ void pack_hilo(float x, float y, uint32_t& hi, uint32_t& lo) {
    __nv_bfloat16 hx, lx, hy, ly;
    split_bf16(x, hx, lx);
    split_bf16(y, hy, ly);
    hi = (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(lx) | ((uint32_t)__bfloat16_as_ushort(ly) << 16);
}

// Largest ring depth of the K/V tile pipeline (the host picks 2..max per launch).  A CTA streams its key range
// alone, so the bytes it keeps in flight (ring depth x 8-32 KB per tile) over the memory latency are its
// bandwidth; a shallower ring lets two CTAs share an SM when many (sequence, KV head) pairs are in flight.
template <int HD, int NS> struct Ring { static constexpr int MAX_STAGES = HD >= 128 ? (NS > 4 ? 4 : 5) : 8; };

// Warp groups of an eight-warp CTA whose query tile has n_slabs slabs and whose key range has n_tiles tiles.  With a
// single slab four groups work on four key tiles at once whatever the ring depth allows behind them: a ring of one
// filling per group (the next tiles requested only once these are used) still beats two groups with a tile in flight
// (ceil(T/4) x 3 us against ceil(T/2) x 2 us for T tiles of 128-wide heads).  With more slabs the SM's mma.sync pipes are
// busy anyway, and each group keeps two ring stages (one computing, one in flight) unless the whole range fits at once.
__host__ __device__ inline int warp_groups(int n_slabs, int stages, int n_tiles) {
    int ng = 8 / n_slabs;
    ng = ng >= 4 ? 4 : (ng >= 2 ? 2 : 1);
    if (n_slabs == 1) {
        while (ng > 1 && stages / ng < 1) ng >>= 1;
        return ng;
    }
    while (ng > 1 && stages / ng < 2 && !(stages / ng >= 1 && n_tiles <= (stages / ng) * ng)) ng >>= 1;
    return ng;
}

__device__ __forceinline__ void cp_async_wait_dyn(int n) {      // wait until at most n groups are pending
    switch (n) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        case 6: cp_async_wait<6>(); break;
        default: cp_async_wait<7>(); break;
    }
}

// NS = number of 16-row slabs the padded query tile has (4 or 8); the CTA always has eight warps.
template <int HD, int NS>
__global__ void __launch_bounds__(256)
attn_mma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttnArgs a) {
    constexpr int NW = 8;                        // warps
    constexpr int GP = NS * 16;                  // padded query rows
    constexpr int CH = HD / 8;                   // 16-byte chunks per row
    constexpr int THREADS = NW * 32;
    constexpr int TILE_BYTES = TKEYS * HD * 2;
    const int STAGES = a.stages;                 // ring depth of this launch, 2 .. Ring<HD, NS>::MAX_STAGES
    extern __shared__ uint8_t sm_raw[];
    uint8_t* sm = sm_raw + ((1024u - (smem_u32(sm_raw) & 1023u)) & 1023u);      // swizzled tiles sit on 1024-byte boundaries
    uint8_t* Qh = sm;
    uint8_t* Ql = Qh + GP * HD * 2;
    uint8_t* Kt = Ql + GP * HD * 2;              // [STAGES][TKEYS][HD]
    uint8_t* Vt = Kt + STAGES * TILE_BYTES;      // [STAGES][TKEYS][HD]
    constexpr int MAX_STAGED_PAGES = 1024;
    __shared__ int s_pages[MAX_STAGED_PAGES];
    __shared__ uint64_t s_full[8];               // one per ring stage: bytes of its K and V tile have landed (TMA path)

    const int sp = blockIdx.x, kh = blockIdx.y / a.n_hsplit, b = blockIdx.z / a.n_sub, rb = (blockIdx.z % a.n_sub) * a.Rs;
    const int h0 = kh * (a.n_q / a.n_kv) + (int)(blockIdx.y % a.n_hsplit) * a.hs;      // first query head of this CTA
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef TASC_TIMELINE
    struct LogAtExit { unsigned long long t0, ta, tb, tc, td, te, tf; __device__ ~LogAtExit() { if (threadIdx.x == 0) ctalog_put(t0, ta, tb, 10, tc, td, te, tf); } } log_at_exit{global_ns(), 0, 0, 0, 0, 0, 0};
#endif
    const int g = a.hs, R = a.Rs;                              // g: query heads of this CTA; R: rows of its sub-block, the first is rb
    const int G = g * R;
    const int qd = a.n_q * HD;

    // The row plan, the block table and the K/V of committed positions were written before the
    // preceding grid started, so they may be read ahead of griddepcontrol.wait.
    // A pass with more than Rs rows per sequence (prefill) is cut into sub-blocks of Rs rows; the rows before this
    // sub-block are ordinary keys to it, but they were written by the preceding grid like its own.
    const int seq_pos0 = a.seq_pos0[b];                        // committed positions: in the cache before this pass
    int rows = a.seq_rows[b] - rb;
    rows = rows < 0 ? 0 : (rows > R ? R : rows);
    const int pos0 = seq_pos0 + rb;
    if (rows == 0) {
        griddep_wait();
        griddep_launch_dependents();
        // sequence not in this step: its rows of the output are zero
        if (sp == 0) {
            for (int i = tid; i < G * (HD / 4); i += THREADS) {
                const int rho = i / (HD / 4), d4 = (i % (HD / 4)) * 4;
                const int m = b * a.R + rb + rho % R;
                const size_t row = (size_t)(m / a.TB) * (2 * a.TB) + (m % a.TB);
                const size_t col = (size_t)(h0 + rho / R) * HD + d4;
                *reinterpret_cast<uint2*>(a.out + row * qd + col) = make_uint2(0u, 0u);
                *reinterpret_cast<uint2*>(a.out + (row + a.TB) * qd + col) = make_uint2(0u, 0u);
            }
        }
        return;
    }
    const int total = pos0 + rows;               // keys visible to the last row
    // the range's 64-key tiles are dealt out evenly: every split gets floor or ceil of tiles / splits of them
    const int tiles_all = (total + TKEYS - 1) / TKEYS;
    const int t_base = tiles_all / a.splits, t_rem = tiles_all % a.splits;
    const int n_tiles = t_base + (sp < t_rem ? 1 : 0);
    const int k_begin = (sp * t_base + min(sp, t_rem)) * TKEYS;
    const int k_end = min(total, k_begin + n_tiles * TKEYS);
    const int n_slabs = (G + 15) / 16;
    // A warp owns one 16-row slab of one key tile.  With fewer slabs than warps the warps form ng = 2 or 4 groups
    // of n_slabs warps; group `grp` handles tiles grp, grp + ng, ...; the groups' results are merged in shared memory.
    const int ng = warp_groups(n_slabs, STAGES, n_tiles);
    const int slab = warp % n_slabs, grp = warp / n_slabs;
    const bool computes = grp < ng;
    const int n_super = (n_tiles + ng - 1) / ng;                 // iterations of ng tiles
    const int super_stages = STAGES / ng;

    // Page ids of this CTA's key range, staged once: the tile loads then need no dependent global read.
    const int pg_lo = k_begin / a.page_size;
    const int n_pg = n_tiles > 0 ? (k_end - 1) / a.page_size - pg_lo + 1 : 0;
    const bool pages_staged = n_pg <= MAX_STAGED_PAGES;
    const bool use_tma = a.use_tma && pages_staged;
    if (tid == 0 && use_tma) {
        for (int i = 0; i < STAGES; ++i) mbar_init(smem_u32(&s_full[i]), 1);
        fence_barrier_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (pages_staged) {
        for (int i = tid; i < n_pg; i += THREADS) {
            const int pslot = pg_lo + i;
            int page = -1;
            if (pslot < a.max_pages) page = a.block_table[(size_t)b * a.max_pages + pslot];
            s_pages[i] = (page >= 0 && page < a.n_pages) ? page : -1;      // ids outside the pool are never used as addresses
        }
    }
    __syncthreads();
    // TMA path (warp 0, one box per lane): a tile is four 16-token pages; each page of this KV head is one box (two
    // for head_dim 128) of the [pages * kv_heads * 16][head_dim] view of the pool, for K and for V.  Rows past the
    // key range re-read the range's last page and a page id outside the pool reads page 0: both are masked later,
    // and nothing unmapped is touched.  A lane that issues one copy does not wait for the other lanes' copies, so
    // the boxes of up to four tiles are requested in the time one thread needs for two.
    constexpr int HB = HD == 128 ? 2 : 1;                      // 64-column boxes per row
    constexpr int BOXES = (TKEYS / 16) * HB * 2;               // boxes of one tile: pages x halves x (K, V)
    auto load_tiles_tma = [&](int sup) {
        for (int idx = lane; idx < ng * BOXES; idx += 32) {
            const int j = idx / BOXES, r = idx % BOXES;
            const int tile = sup * ng + j;
            if (tile >= n_tiles) continue;
            const int stage = (sup % super_stages) * ng + j;
            const int pg = r / (HB * 2), h = (r >> 1) % HB, is_v = r & 1;
            const uint32_t bar = smem_u32(&s_full[stage]);
            // the expected bytes may be posted after some of them have arrived: the phase cannot end before
            // this arrival, which is the barrier's only one
            if (r == 0) mbar_expect_tx(bar, 2u * TILE_BYTES);
            int key = k_begin + tile * TKEYS + pg * 16;
            key = key < k_end ? key : k_end - 1;
            int page = s_pages[key / 16 - pg_lo];
            page = page < 0 ? 0 : page;
            const int y = (page * a.n_kv + kh) * 16;
            constexpr int BOXB = (HD >= 64 ? 128 : 64) * 16;       // bytes of one box: 16 rows of at most 128 bytes
            const uint32_t dst = smem_u32((is_v ? Vt : Kt) + stage * TILE_BYTES) + h * (TKEYS * 128) + pg * BOXB;
            tma_load_2d(dst, is_v ? &tmV : &tmK, h * 64, y, bar);
        }
    };
    // cp.async path: one row of the tile per TPR threads: a page lookup, then the thread's share of the row's chunks.
    constexpr int TPR = THREADS / TKEYS, CPT = CH / TPR;
    auto load_tile = [&](int tile, int stage) {
        const int row = tid / TPR, c0 = (tid % TPR) * CPT;
        const int key = k_begin + tile * TKEYS + row;
        const uint32_t kdst = smem_u32(Kt + stage * TILE_BYTES), vdst = smem_u32(Vt + stage * TILE_BYTES);
        size_t off = 0;
        int bytes = 0;
        if (key < k_end) {
            const int pslot = key / a.page_size;
            int page = -1;
            if (pages_staged) page = s_pages[pslot - pg_lo];
            else if (pslot < a.max_pages) {
                page = a.block_table[(size_t)b * a.max_pages + pslot];
                if (page >= a.n_pages) page = -1;
            }
            if (page >= 0) {
                off = (((size_t)page * a.n_kv + kh) * a.page_size + key % a.page_size) * HD;
                bytes = 16;
            }
        }
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            const uint32_t so = swz<HD>(row, c0 + j);
            cp_async16(kdst + so, a.kp + off + (c0 + j) * 8, bytes);     // zero-fills when bytes = 0
            cp_async16(vdst + so, a.vp + off + (c0 + j) * 8, bytes);
        }
    };
    auto load_super = [&](int sup) {                             // the ng tiles of iteration `sup`
        if (use_tma) {
            if (warp == 0) load_tiles_tma(sup);
        } else {
            for (int j = 0; j < ng; ++j)
                if (sup * ng + j < n_tiles) load_tile(sup * ng + j, (sup % super_stages) * ng + j);
            cp_async_commit();                                   // one group per iteration, empty past the end
        }
    };
    // prologue of the ring (all super_stages slots): iterations that lie wholly inside the committed prefix are
    // requested before the wait, those holding this step's new rows (written by the preceding grid) after it
    int issued = 0;
    while (issued < super_stages && issued < n_super && k_begin + (issued + 1) * ng * TKEYS <= seq_pos0) {
        load_super(issued);
        ++issued;
    }
    griddep_wait();
#ifdef TASC_TIMELINE
    log_at_exit.ta = global_ns();
#endif
    griddep_launch_dependents();

    // Q rows of this KV head's group, scaled, as (hi, lo) bf16 in swizzled shared memory.  All global reads
    // are issued before the first conversion so that their latencies overlap.
    constexpr int NQ = GP * (HD / 4) / THREADS;
    float4 qv[NQ];
#pragma unroll
    for (int j = 0; j < NQ; ++j) {
        const int i = tid + j * THREADS;
        const int rho = i / (HD / 4), d4 = (i % (HD / 4)) * 4;
        const int hl = rho / R, rr = rho % R;
        qv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (rho < G && rr < rows)
            qv[j] = *reinterpret_cast<const float4*>(a.q + (size_t)(b * a.R + rb + rr) * qd + (size_t)(h0 + hl) * HD + d4);
    }
    // the rest of the ring's prologue (tiles holding this step's new rows), requested while the Q rows are on their way
    for (; issued < super_stages; ++issued) load_super(issued);       // past the end: nothing (cp.async: an empty group)
#pragma unroll
    for (int j = 0; j < NQ; ++j) {
        const int i = tid + j * THREADS;
        const int rho = i / (HD / 4), d4 = (i % (HD / 4)) * 4;
        const float4 v = make_float4(qv[j].x * a.scale_log2e, qv[j].y * a.scale_log2e, qv[j].z * a.scale_log2e, qv[j].w * a.scale_log2e);
        uint2 h, l;
        pack_hilo(v.x, v.y, h.x, l.x);
        pack_hilo(v.z, v.w, h.y, l.y);
        const uint32_t so = swz<HD, GP>(rho, d4 >> 3) + (uint32_t)((d4 & 7) * 2);
        *reinterpret_cast<uint2*>(Qh + so) = h;
        *reinterpret_cast<uint2*>(Ql + so) = l;
    }

    // per-thread rows of the slab: r0 = lane / 4 and r0 + 8
    const int rho0 = slab * 16 + (lane >> 2), rho1 = rho0 + 8;
    const int lim0 = (rho0 < G && rho0 % R < rows) ? min(pos0 + rho0 % R, k_end - 1) : -1;   // last visible key
    const int lim1 = (rho1 < G && rho1 % R < rows) ? min(pos0 + rho1 % R, k_end - 1) : -1;
    float o[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const uint32_t qh_base = smem_u32(Qh), ql_base = smem_u32(Ql);
#ifdef TASC_TIMELINE
    log_at_exit.tc = global_ns();
#endif

    for (int sup = 0; sup < n_super; ++sup) {
        if (use_tma) {                                             // iteration `sup` has landed (bounded wait)
            for (int j = 0; j < ng; ++j)
                if (sup * ng + j < n_tiles &&
                    !mbar_wait(smem_u32(&s_full[(sup % super_stages) * ng + j]), (uint32_t)(sup / super_stages) & 1u))
                    set_status(a.status, TASC_ETIMEOUT);
        } else {
            cp_async_wait_dyn(super_stages - 1);
        }
        __syncthreads();
#ifdef TASC_TIMELINE
        if (sup == 0) log_at_exit.td = global_ns();
        if (sup == 1) log_at_exit.te = global_ns();
        if (sup == 2) log_at_exit.tf = global_ns();
#endif
        const int tile = sup * ng + grp;
        if (computes && tile < n_tiles) {
            const int stage = (sup % super_stages) * ng + grp;
            const int k0 = k_begin + tile * TKEYS;
            const uint32_t kbase = smem_u32(Kt + stage * TILE_BYTES), vbase = smem_u32(Vt + stage * TILE_BYTES);
            float s[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
            const int mi = lane >> 3, li = lane & 7;
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks) {
                uint32_t qh[4], ql[4];
                const uint32_t qo = swz<HD, GP>(slab * 16 + (mi & 1) * 8 + li, ks * 2 + (mi >> 1));
                ldsm_x4(qh_base + qo, qh);
                ldsm_x4(ql_base + qo, ql);
                // eight independent accumulators between two MMAs on the same one (hi pass, then lo pass)
                uint32_t kb[4][4];
#pragma unroll
                for (int np = 0; np < 4; ++np) ldsm_x4(kbase + swz<HD>(np * 16 + (mi >> 1) * 8 + li, ks * 2 + (mi & 1)), kb[np]);
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    mma_bf16(s[2 * np], qh, kb[np][0], kb[np][1]);
                    mma_bf16(s[2 * np + 1], qh, kb[np][2], kb[np][3]);
                }
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    mma_bf16(s[2 * np], ql, kb[np][0], kb[np][1]);
                    mma_bf16(s[2 * np + 1], ql, kb[np][2], kb[np][3]);
                }
            }
            // causal / range mask (only tiles that reach past the committed prefix or the split's end)
            if (k0 + TKEYS > pos0 + 1 || k0 + TKEYS > k_end || lim0 < 0 || lim1 < 0) {
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    const int key = k0 + nt * 8 + 2 * (lane & 3);
                    if (key > lim0) s[nt][0] = -INFINITY;
                    if (key + 1 > lim0) s[nt][1] = -INFINITY;
                    if (key > lim1) s[nt][2] = -INFINITY;
                    if (key + 1 > lim1) s[nt][3] = -INFINITY;
                }
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
                mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
            const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
            const float al0 = exp2f(m_run[0] - mu0), al1 = exp2f(m_run[1] - mu1);     // 0 while nothing was visible
            m_run[0] = mn0; m_run[1] = mn1;
            float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                s[nt][0] = exp2f(s[nt][0] - mu0); s[nt][1] = exp2f(s[nt][1] - mu0);
                s[nt][2] = exp2f(s[nt][2] - mu1); s[nt][3] = exp2f(s[nt][3] - mu1);
                ps0 += s[nt][0] + s[nt][1];
                ps1 += s[nt][2] + s[nt][3];
            }
            l_run[0] = l_run[0] * al0 + ps0;
            l_run[1] = l_run[1] * al1 + ps1;
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) { o[i][0] *= al0; o[i][1] *= al0; o[i][2] *= al1; o[i][3] *= al1; }
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                uint32_t ph[4], pl[4];
                pack_hilo(s[2 * kb][0], s[2 * kb][1], ph[0], pl[0]);
                pack_hilo(s[2 * kb][2], s[2 * kb][3], ph[1], pl[1]);
                pack_hilo(s[2 * kb + 1][0], s[2 * kb + 1][1], ph[2], pl[2]);
                pack_hilo(s[2 * kb + 1][2], s[2 * kb + 1][3], ph[3], pl[3]);
#pragma unroll
                for (int dp = 0; dp < HD / 16; dp += 2) {          // four independent accumulators per pass
                    uint32_t vb0[4], vb1[4];
                    ldsm_x4_trans(vbase + swz<HD>(kb * 16 + (mi & 1) * 8 + li, dp * 2 + (mi >> 1)), vb0);
                    ldsm_x4_trans(vbase + swz<HD>(kb * 16 + (mi & 1) * 8 + li, (dp + 1) * 2 + (mi >> 1)), vb1);
                    mma_bf16(o[2 * dp], ph, vb0[0], vb0[1]);
                    mma_bf16(o[2 * dp + 1], ph, vb0[2], vb0[3]);
                    mma_bf16(o[2 * dp + 2], ph, vb1[0], vb1[1]);
                    mma_bf16(o[2 * dp + 3], ph, vb1[2], vb1[3]);
                    mma_bf16(o[2 * dp], pl, vb0[0], vb0[1]);
                    mma_bf16(o[2 * dp + 1], pl, vb0[2], vb0[3]);
                    mma_bf16(o[2 * dp + 2], pl, vb1[0], vb1[1]);
                    mma_bf16(o[2 * dp + 3], pl, vb1[2], vb1[3]);
                }
            }
        }
        __syncthreads();
        // the slot of this iteration is free again: refill it with the iteration super_stages ahead
        if (sup + super_stages < n_super) load_super(sup + super_stages);
        else if (!use_tma) cp_async_commit();
    }
#ifdef TASC_TIMELINE
    log_at_exit.tb = global_ns();
#endif
    if (computes) {
        l_run[0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[0], 1);
        l_run[0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[0], 2);
        l_run[1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[1], 1);
        l_run[1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[1], 2);
    }
    if (ng > 1) {
        // groups 1 .. ng-1 -> shared memory (the K/V ring is idle) -> group 0 folds them into its state, in group order
        constexpr int XG = HD / 2 + 4;                          // floats per lane: O fragment, two maxima, two sums
        float* xg0 = reinterpret_cast<float*>(Kt);
        if (computes && grp > 0) {
            float* xg = xg0 + ((size_t)((grp - 1) * n_slabs + slab) * 32 + lane) * XG;
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) { xg[4 * i] = o[i][0]; xg[4 * i + 1] = o[i][1]; xg[4 * i + 2] = o[i][2]; xg[4 * i + 3] = o[i][3]; }
            xg[HD / 2] = m_run[0]; xg[HD / 2 + 1] = m_run[1]; xg[HD / 2 + 2] = l_run[0]; xg[HD / 2 + 3] = l_run[1];
        }
        __syncthreads();
        if (grp == 0) {
            for (int og = 1; og < ng; ++og) {
                const float* xg = xg0 + ((size_t)((og - 1) * n_slabs + slab) * 32 + lane) * XG;
                const float om0 = xg[HD / 2], om1 = xg[HD / 2 + 1], ol0 = xg[HD / 2 + 2], ol1 = xg[HD / 2 + 3];
                const float mn0 = fmaxf(m_run[0], om0), mn1 = fmaxf(m_run[1], om1);
                const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
                const float sa0 = exp2f(m_run[0] - mu0), sb0 = exp2f(om0 - mu0), sa1 = exp2f(m_run[1] - mu1), sb1 = exp2f(om1 - mu1);
#pragma unroll
                for (int i = 0; i < HD / 8; ++i) {
                    o[i][0] = o[i][0] * sa0 + xg[4 * i] * sb0;     o[i][1] = o[i][1] * sa0 + xg[4 * i + 1] * sb0;
                    o[i][2] = o[i][2] * sa1 + xg[4 * i + 2] * sb1; o[i][3] = o[i][3] * sa1 + xg[4 * i + 3] * sb1;
                }
                l_run[0] = l_run[0] * sa0 + ol0 * sb0; l_run[1] = l_run[1] * sa1 + ol1 * sb1;
                m_run[0] = mn0; m_run[1] = mn1;
            }
        }
    }
    const bool writer = computes && grp == 0;                  // holds the CTA's result for its slab

    if (a.splits == 1) {
        // the whole key range was here: normalise and write the rows straight to the O-projection's input
        if (writer) {
            const float inv0 = l_run[0] > 0.f ? 1.0f / l_run[0] : 0.f, inv1 = l_run[1] > 0.f ? 1.0f / l_run[1] : 0.f;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int rho = half ? rho1 : rho0;
                if (rho >= G) continue;
                const int hl = rho / R, rr = rho % R;
                const float inv = (rr < rows) ? (half ? inv1 : inv0) : 0.f;
                const int m = b * a.R + rb + rr;
                const size_t row = (size_t)(m / a.TB) * (2 * a.TB) + (m % a.TB);
                const size_t col = (size_t)(h0 + hl) * HD + 2 * (lane & 3);
#pragma unroll
                for (int nt = 0; nt < HD / 8; ++nt) {
                    uint32_t h, l;
                    pack_hilo(o[nt][2 * half] * inv, o[nt][2 * half + 1] * inv, h, l);
                    *reinterpret_cast<uint32_t*>(a.out + row * qd + col + nt * 8) = h;
                    *reinterpret_cast<uint32_t*>(a.out + (row + a.TB) * qd + col + nt * 8) = l;
                }
            }
        }
        return;
    }

    // The key range was split over the S CTAs of this cluster: every CTA parks its unnormalised rows
    // (O, running maximum, running sum) in its own shared memory (the K/V ring is idle); after a cluster
    // barrier CTA r merges the rows rho = r, r + S, ... from all S copies, in rank order, and writes them.
    constexpr int XS = HD + 4;                                 // floats per parked row: O[HD], max, sum, pad
    float* xo = reinterpret_cast<float*>(Kt);
    __syncthreads();                                           // the warp groups' exchange area is inside the ring too
    if (writer) {
        float* r0p = xo + (size_t)rho0 * XS + 2 * (lane & 3);
        float* r1p = xo + (size_t)rho1 * XS + 2 * (lane & 3);
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) {
            *reinterpret_cast<float2*>(r0p + nt * 8) = make_float2(o[nt][0], o[nt][1]);
            *reinterpret_cast<float2*>(r1p + nt * 8) = make_float2(o[nt][2], o[nt][3]);
        }
        if ((lane & 3) == 0) {
            *reinterpret_cast<float2*>(xo + (size_t)rho0 * XS + HD) = make_float2(m_run[0], l_run[0]);
            *reinterpret_cast<float2*>(xo + (size_t)rho1 * XS + HD) = make_float2(m_run[1], l_run[1]);
        }
    }
    cluster_arrive();
    cluster_wait();
    const int S = a.splits, rank = (int)cluster_ctarank();
    const uint32_t xo_addr = smem_u32(xo);
    uint32_t peer[8];
#pragma unroll
    for (int sidx = 0; sidx < 8; ++sidx) peer[sidx] = cluster_map(xo_addr, (uint32_t)(sidx < S ? sidx : 0));
    const int my_rows = rank < G ? (G - rank + S - 1) / S : 0;
    for (int i = tid; i < my_rows * (HD / 4); i += THREADS) {
        const int rho = rank + (i / (HD / 4)) * S, d4 = (i % (HD / 4)) * 4;
        const int hl = rho / R, rr = rho % R;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (rr < rows) {
            float2 ml[8];
            float4 ov[8];
#pragma unroll
            for (int sidx = 0; sidx < 8; ++sidx)
                if (sidx < S) {                                 // all remote reads are issued before the first is used
                    const uint32_t rowa = peer[sidx] + (uint32_t)(rho * XS) * 4u;
                    ml[sidx] = ld_cluster_f2(rowa + HD * 4u);
                    ov[sidx] = ld_cluster_f4(rowa + (uint32_t)d4 * 4u);
                }
            float mstar = -INFINITY;
#pragma unroll
            for (int sidx = 0; sidx < 8; ++sidx)
                if (sidx < S) mstar = fmaxf(mstar, ml[sidx].x);
            float den = 0.f;
#pragma unroll
            for (int sidx = 0; sidx < 8; ++sidx)
                if (sidx < S && ml[sidx].x != -INFINITY) {      // a split without visible keys holds zeros
                    const float w = exp2f(ml[sidx].x - mstar);
                    den += w * ml[sidx].y;
                    acc.x += w * ov[sidx].x; acc.y += w * ov[sidx].y; acc.z += w * ov[sidx].z; acc.w += w * ov[sidx].w;
                }
            const float inv = den > 0.f ? 1.0f / den : 0.f;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        }
        const int m = b * a.R + rb + rr;
        const size_t row = (size_t)(m / a.TB) * (2 * a.TB) + (m % a.TB);
        const size_t col = (size_t)(h0 + hl) * HD + d4;
        uint2 h, l;
        pack_hilo(acc.x, acc.y, h.x, l.x);
        pack_hilo(acc.z, acc.w, h.y, l.y);
        *reinterpret_cast<uint2*>(a.out + row * qd + col) = h;
        *reinterpret_cast<uint2*>(a.out + (row + a.TB) * qd + col) = l;
    }
    // peers may still be reading this CTA's parked rows
    cluster_arrive();
    cluster_wait();
}

inline size_t attn_smem_bytes(int hd, int gp, int stages) {
    return 1024 + (size_t)2 * gp * hd * 2 + (size_t)2 * stages * TKEYS * hd * 2;      // 1024: alignment slack
}

template <int HD, int NS>
tasc_status prepare_inst() {
    static bool done[64] = {false};
    int dev = 0;
    TASC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return TASC_EINVAL;
    if (!done[dev]) {
        TASC_CUDA_TRY(cudaFuncSetAttribute(attn_mma_kernel<HD, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        done[dev] = true;
    }
    return TASC_OK;
}

// Clusters of `splits` CTAs (ring depth `stages`) the device holds at once; 0 if the query fails.
template <int HD, int NS>
int fit_inst(int splits, int stages) {
    if (prepare_inst<HD, NS>() != TASC_OK) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)splits, 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = attn_smem_bytes(HD, NS * 16, stages);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)splits;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, attn_mma_kernel<HD, NS>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

int fit_any(int hd, int nw, int splits, int stages) {
    static std::mutex mu;
    static std::map<long long, int> cache;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    const long long key = ((((long long)dev * 256 + hd) * 16 + nw) * 16 + splits) * 16 + stages;
    std::lock_guard<std::mutex> lk(mu);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    int n = 0;
    if (nw == 4) n = hd == 32 ? fit_inst<32, 4>(splits, stages) : hd == 64 ? fit_inst<64, 4>(splits, stages) : fit_inst<128, 4>(splits, stages);
    else n = hd == 32 ? fit_inst<32, 8>(splits, stages) : hd == 64 ? fit_inst<64, 8>(splits, stages) : fit_inst<128, 8>(splits, stages);
    cache[key] = n;
    return n;
}

template <int HD, int NS>
tasc_status launch_inst(const AttnArgs& a, const CUtensorMap& tmK, const CUtensorMap& tmV, int B, cudaStream_t stream) {
    constexpr int GP = NS * 16;
    if (a.stages < 2 || a.stages > Ring<HD, NS>::MAX_STAGES) return TASC_EINVAL;
    const size_t smem = attn_smem_bytes(HD, GP, a.stages);
    tasc_status pst = prepare_inst<HD, NS>();
    if (pst != TASC_OK) return pst;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.splits, (unsigned)(a.n_kv * a.n_hsplit), (unsigned)B);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    int n_at = 1;
    if (a.splits > 1) {                            // the key-range splits of one (sequence, KV head) form a cluster
        at[n_at].id = cudaLaunchAttributeClusterDimension;
        at[n_at].val.clusterDim.x = (unsigned)a.splits;
        at[n_at].val.clusterDim.y = 1;
        at[n_at].val.clusterDim.z = 1;
        ++n_at;
    }
    cfg.attrs = at;
    cfg.numAttrs = n_at;
    ProfScope ps(K_ATT_SPLIT, stream);
    TASC_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_mma_kernel<HD, NS>, tmK, tmV, a));
    return TASC_OK;
}

}  // namespace

int attention_mma_row_pad(int G) { return G <= 64 ? 64 : 128; }

// Query heads per CTA, key-range splits per (sequence, head group) (1..8, the CTAs of a cluster) and ring depth, from a
// small cost model in microseconds: a CTA needs about 2.5 us to start (Q staging, first tiles) plus one tile time per
// iteration (its warp groups take `ng` tiles per iteration; a shallow ring adds memory stalls), the clusters run in as
// many waves as the device's cluster occupancy dictates (one straggling cluster costs a whole wave), and splitting
// adds the cluster exchange and merge.  With few sequences the g query heads that share a KV head are dealt out to
// several CTAs (each re-reads that head's K/V from L2, which is cheap next to leaving most SMs idle): fewer query rows
// per CTA mean fewer slabs, so more warp groups work on different key tiles at once.
AttnPlan plan_attention_mma(int B, int n_kv, int hd, int g, int rows, int max_ctx) {
    // The launch shape is fixed before the lengths are known (and stays fixed in a captured graph): it is chosen
    // for three quarters of the context the cache can hold; shorter ranges leave the last splits idle.
    const int n_tiles = std::max(1, ((max_ctx * 3) / 4 + TKEYS - 1) / TKEYS);
    // Measured (microseconds): one iteration of a warp group over a 64-key tile, and the time the SM's mma.sync
    // pipes need per tile and 16-row slab when all warps have work (the lower bound once several groups run).
    const float t_tile = hd >= 128 ? 2.0f : (hd >= 64 ? 1.3f : 0.8f);
    const float t_pipe = hd >= 128 ? 0.6f : (hd >= 64 ? 0.3f : 0.15f);
    AttnPlan best = {1, 2, g};
    float best_cost = 1e30f;
    // Candidates: all g heads of a KV head in one CTA; and, for few sequences with 128-wide heads (where one warp needs
    // 2 us per key tile), the largest share of the heads whose rows still fill a single 16-row slab.  (Measured: on the
    // 1.5B shape at one sequence 2 of 6 heads per CTA shorten the step by 4 %; 64-wide heads and larger batches lose.)
    int hs_slab = g;
    while (hs_slab > 1 && (g % hs_slab || hs_slab * rows > 16)) --hs_slab;
    const bool may_split = hd >= 128 && B * n_kv <= 4 && hs_slab * rows <= 16;
    for (int hs = g; hs >= 1; --hs) {
        if (g % hs) continue;
        if (hs != g && !(may_split && hs == hs_slab)) continue;
        const int G = hs * rows;
        if (G > 128) continue;
        const int nw = G <= 64 ? 4 : 8, n_slabs = (G + 15) / 16;       // nw: slabs of the padded query tile (kernel instance)
        const int max_stages = hd >= 128 ? (nw > 4 ? 4 : 5) : 8;
        const int depths[2] = {max_stages, max_stages >= 8 ? 4 : 3};
        const int groups = B * n_kv * (g / hs);                       // clusters of the launch
        for (int di = 0; di < 2; ++di) {
            const int stages = depths[di];
            for (int s = 1; s <= 8 && s <= n_tiles; ++s) {
                int fit = fit_any(hd, nw, s, stages);
                if (fit <= 0) fit = std::max(1, 148 / s);               // no device to ask: assume one CTA per SM
                const int waves = (groups + fit - 1) / fit;
                const int tiles_cta = (n_tiles + s - 1) / s;
                const int ng = warp_groups(n_slabs, stages, tiles_cta);
                const int iters = (tiles_cta + ng - 1) / ng;
                const float stall = di == 0 ? 0.f : 0.25f * t_tile;      // a shallow ring hides less latency
                const float loop = std::max(iters * (t_tile + stall), tiles_cta * n_slabs * t_pipe);
                const float merge = s > 1 ? 0.5f + 0.25f * s : 0.f;      // cluster barrier + one round of remote reads
                // a grid that takes (nearly) every SM keeps the next kernel's CTAs from starting early
                const float crowd = groups * s > 128 ? 3.0f : 0.f;
                // every head group re-reads its KV head's keys: L2 traffic, about 0.1 us per extra pass over a tile
                const float reread = 0.1f * tiles_cta * (float)(g / hs - 1) / (float)std::max(1, g / hs);
                const float cost = waves * (2.5f + loop) + merge + crowd + reread;
                if (cost < best_cost - 1e-6f) { best_cost = cost; best = AttnPlan{s, stages, hs}; }
            }
        }
    }
    return best;
}

tasc_status launch_attention_mma(const float* qbuf, const __nv_bfloat16* k_pages, const __nv_bfloat16* v_pages,
                                 const int32_t* block_table, int max_pages, int page_size, long long n_pages,
                                 const RowPlan& rp, __nv_bfloat16* out, int TB, int B, int R, int n_q, int n_kv, int hd,
                                 const AttnPlan& plan, int* status, cudaStream_t stream) {
    const int n_splits = plan.splits;
    // up to 16 rows per sequence (a verify step) are one block; longer passes (prefill) are cut into blocks of 16
    const int Rs = R <= 16 ? R : 16;
    if (R % Rs) return TASC_EINVAL;
    const int n_sub = R / Rs;
    const int g = n_q / n_kv, hs = plan.heads;
    if (hs < 1 || g % hs) return TASC_EINVAL;
    const int G = hs * Rs;
    if (G > 128 || (hd != 32 && hd != 64 && hd != 128) || n_splits < 1 || n_splits > 8) return TASC_EINVAL;
    const int GP = attention_mma_row_pad(G);
    AttnArgs a;
    a.q = qbuf; a.kp = k_pages; a.vp = v_pages; a.block_table = block_table;
    a.max_pages = max_pages; a.page_size = page_size; a.n_pages = n_pages;
    a.seq_pos0 = rp.seq_pos0; a.seq_rows = rp.seq_rows;
    a.out = out; a.TB = TB;
    a.hs = hs; a.n_hsplit = g / hs;
    a.R = R; a.Rs = Rs; a.n_sub = n_sub; a.n_q = n_q; a.n_kv = n_kv; a.splits = n_splits; a.stages = plan.stages;
    a.scale_log2e = 1.4426950408889634f / sqrtf((float)hd);
    a.status = status;
    // 16-token pages arrive as TMA boxes; any other page size takes the cp.async path of the same kernel
    a.use_tma = page_size == 16 ? 1 : 0;
    CUtensorMap tmK, tmV;
    memset(&tmK, 0, sizeof(tmK));
    memset(&tmV, 0, sizeof(tmV));
    if (a.use_tma) {
        const uint64_t rows = (uint64_t)n_pages * n_kv * 16;
        tasc_status st;
        if ((st = encode_tmap_kv(&tmK, k_pages, rows, hd)) != TASC_OK) return st;
        if ((st = encode_tmap_kv(&tmV, v_pages, rows, hd)) != TASC_OK) return st;
    }
    if (GP == 64) {
        if (hd == 32) return launch_inst<32, 4>(a, tmK, tmV, B * n_sub, stream);
        if (hd == 64) return launch_inst<64, 4>(a, tmK, tmV, B * n_sub, stream);
        return launch_inst<128, 4>(a, tmK, tmV, B * n_sub, stream);
    }
    if (hd == 32) return launch_inst<32, 8>(a, tmK, tmV, B * n_sub, stream);
    if (hd == 64) return launch_inst<64, 8>(a, tmK, tmV, B * n_sub, stream);
    return launch_inst<128, 8>(a, tmK, tmV, B * n_sub, stream);
}

}  // namespace tasc
