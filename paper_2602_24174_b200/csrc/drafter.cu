// On-device n-gram drafter (TASC-draft): corpus tables p_corp, context model p_prompt, exact mixture argmax.
//
// Build (once per task): for each order n = 1..n_max every window (n context tokens, next token) of
// every document is counted in an open-addressing scratch table keyed by the full 128-bit packing of
// (n, tokens) -- one 128-bit compare-and-swap claims or finds a slot, so there is no fingerprint
// matching and counts are exact.  Elements with count >= p_min are then moved into the final
// per-order structure: a context table (packed context -> offset, number of successors, total count)
// plus a flat successor array of (next, count).  Slot placement depends on thread timing, results do
// not: lookups return the same sets, and the export sorts canonically.
//
// Draft (every step): one CTA per sequence.  For each of the k drafts: warp-cooperative probes of the
// context tables of all orders at once (one warp per order, 32 slots per probe round; longest hit wins), a scan of the sequence's committed tokens for the
// longest matching suffix with its successor counts collected in a shared-memory hash, and the argmax
// of  lambda_num * c_corp(x) * T_prompt + (lambda_den - lambda_num) * c_prompt(x) * T_corp  in 64-bit
// integers with the smallest token id winning ties.
#include "kernels.h"

#include <algorithm>
#include <new>
#include <vector>

struct CtxVal {
    unsigned long long offset;   // first successor in the order's successor array
    uint32_t n_succ;
    uint32_t total;              // sum of the surviving counts
};
struct Succ {
    int32_t next;
    uint32_t count;
};
struct OrderTable {
    uint64_t* keys;              // [cap][2]
    CtxVal* vals;                // [cap]
    Succ* succ;                  // [n_succ]
    uint64_t mask;               // cap - 1
    long long n_succ;
};
struct DeviceTables {
    OrderTable t[TASC_MAX_ORDER + 1];   // index = order n
    int n_max;
    int fallback;
};

struct tasc_drafter {
    DeviceTables dt;
    int p_min, vocab, device;
};

namespace tasc {
namespace {

constexpr uint64_t VALID_BIT = 1ull << 63;
constexpr int TOK_BITS = TASC_VOCAB_BITS;
constexpr uint32_t TOK_MASK = (1u << TOK_BITS) - 1u;

struct Key { uint64_t lo, hi; };

// Field j (20 bits) at bit 20*j of the 128-bit word; the order in bits 120..122; bit 127 marks a used slot.
__host__ __device__ __forceinline__ void key_put(Key& k, int field, uint32_t tok) {
    const int bit = field * TOK_BITS;
    const uint64_t v = tok & TOK_MASK;
    if (bit + TOK_BITS <= 64) k.lo |= v << bit;
    else if (bit >= 64) k.hi |= v << (bit - 64);
    else { k.lo |= v << bit; k.hi |= v >> (64 - bit); }
}
__host__ __device__ __forceinline__ uint32_t key_get(const Key& k, int field) {
    const int bit = field * TOK_BITS;
    uint64_t v;
    if (bit + TOK_BITS <= 64) v = k.lo >> bit;
    else if (bit >= 64) v = k.hi >> (bit - 64);
    else v = (k.lo >> bit) | (k.hi << (64 - bit));
    return (uint32_t)v & TOK_MASK;
}
__host__ __device__ __forceinline__ Key key_make(int n) {
    Key k;
    k.lo = 0;
    k.hi = VALID_BIT | ((uint64_t)n << 56);
    return k;
}
__host__ __device__ __forceinline__ uint64_t key_hash(const Key& k) {
    uint64_t h = k.lo * 0x9E3779B97F4A7C15ull ^ (k.hi + 0xD6E8FEB86659FD93ull);
    h ^= h >> 32; h *= 0xD6E8FEB86659FD93ull;
    h ^= h >> 29; h *= 0x9E3779B97F4A7C15ull;
    h ^= h >> 32;
    return h;
}

// 128-bit compare-and-swap on a 16-byte aligned slot; returns the previous contents.
__device__ __forceinline__ Key cas128(uint64_t* addr, Key cmp, Key val) {
    Key old;
    asm volatile(
        "{\n\t.reg .b128 c, n, o;\n\t"
        "mov.b128 c, {%2, %3};\n\t"
        "mov.b128 n, {%4, %5};\n\t"
        "atom.global.cas.b128 o, [%6], c, n;\n\t"
        "mov.b128 {%0, %1}, o;\n\t}"
        : "=l"(old.lo), "=l"(old.hi)
        : "l"(cmp.lo), "l"(cmp.hi), "l"(val.lo), "l"(val.hi), "l"(addr)
        : "memory");
    return old;
}

// Claim or find the slot of `key`; returns the slot or ~0 when the table is full.
__device__ __forceinline__ uint64_t table_upsert(uint64_t* keys, uint64_t mask, Key key) {
    uint64_t slot = key_hash(key) & mask;
    const Key empty = {0ull, 0ull};
    for (uint64_t probe = 0; probe <= mask; ++probe) {
        const Key old = cas128(keys + 2 * slot, empty, key);
        if ((old.lo == 0 && old.hi == 0) || (old.lo == key.lo && old.hi == key.hi)) return slot;
        slot = (slot + 1) & mask;
    }
    return ~0ull;
}

// remaining[i] = number of tokens after position i inside its document, clamped to 255
__global__ void mark_remaining_kernel(const int64_t* __restrict__ offsets, int64_t n_docs, int64_t T, uint8_t* remaining) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T) return;
    int64_t lo = 0, hi = n_docs;           // last doc with offsets[doc] <= i
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (offsets[mid] <= i) lo = mid; else hi = mid;
    }
    const int64_t rem = offsets[lo + 1] - i - 1;
    remaining[i] = (uint8_t)(rem > 255 ? 255 : (rem < 0 ? 0 : rem));
}

__global__ void token_hist_kernel(const int32_t* __restrict__ tokens, int64_t T, int vocab, uint32_t* hist, int* status) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T) return;
    const int t = tokens[i];
    if (t < 0 || t >= vocab) { set_status(status, TASC_EINVAL); return; }
    atomicAdd(&hist[t], 1u);
}
__global__ void hist_argmax_kernel(const uint32_t* __restrict__ hist, int vocab, unsigned long long* best) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= vocab) return;
    atomicMax(best, ((unsigned long long)hist[i] << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i));
}

__global__ void count_kernel(const int32_t* __restrict__ tokens, const uint8_t* __restrict__ remaining, int64_t T, int n,
                             uint64_t* keys, uint32_t* counts, uint64_t mask, int* status) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T || remaining[i] < n) return;
    Key key = key_make(n);
    for (int j = 0; j <= n; ++j) key_put(key, j, (uint32_t)tokens[i + j]);   // context 0..n-1, next in field n
    const uint64_t slot = table_upsert(keys, mask, key);
    if (slot == ~0ull) { set_status(status, TASC_ECAPACITY); return; }
    atomicAdd(&counts[slot], 1u);
}

__global__ void survivors_kernel(const uint32_t* __restrict__ counts, uint64_t cap, uint32_t p_min, unsigned long long* n_surv) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool s = i < cap && counts[i] >= p_min;
    const uint32_t b = __ballot_sync(0xFFFFFFFFu, s);
    if ((threadIdx.x & 31) == 0 && b) atomicAdd(n_surv, (unsigned long long)__popc(b));
}

__device__ __forceinline__ Key context_of(Key entry, int n) {
    // clear the `next` field (field n)
    Key k = entry;
    const int bit = n * TOK_BITS;
    const uint64_t m = (uint64_t)TOK_MASK;
    if (bit + TOK_BITS <= 64) k.lo &= ~(m << bit);
    else if (bit >= 64) k.hi &= ~(m << (bit - 64));
    else { k.lo &= ~(m << bit); k.hi &= ~(m >> (64 - bit)); }
    return k;
}

__global__ void ctx_insert_kernel(const uint64_t* __restrict__ skeys, const uint32_t* __restrict__ counts, uint64_t cap,
                                  uint32_t p_min, int n, OrderTable t, int* status) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= cap || counts[i] < p_min) return;
    const Key e = {skeys[2 * i], skeys[2 * i + 1]};
    const uint64_t slot = table_upsert(t.keys, t.mask, context_of(e, n));
    if (slot == ~0ull) { set_status(status, TASC_ECAPACITY); return; }
    atomicAdd(&t.vals[slot].n_succ, 1u);
    atomicAdd(&t.vals[slot].total, counts[i]);
}
__global__ void assign_offsets_kernel(OrderTable t, unsigned long long* cursor) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i > t.mask) return;
    const uint32_t n = t.vals[i].n_succ;
    if (n) t.vals[i].offset = atomicAdd(cursor, (unsigned long long)n);
}
__global__ void succ_fill_kernel(const uint64_t* __restrict__ skeys, const uint32_t* __restrict__ counts, uint64_t cap,
                                 uint32_t p_min, int n, OrderTable t, uint32_t* fill, int* status) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= cap || counts[i] < p_min) return;
    const Key e = {skeys[2 * i], skeys[2 * i + 1]};
    const uint64_t slot = table_upsert(t.keys, t.mask, context_of(e, n));     // always found
    if (slot == ~0ull) { set_status(status, TASC_ECAPACITY); return; }
    const unsigned long long pos = t.vals[slot].offset + atomicAdd(&fill[slot], 1u);
    if (pos >= (unsigned long long)t.n_succ) { set_status(status, TASC_ECAPACITY); return; }
    Succ s;
    s.next = (int32_t)key_get(e, n);
    s.count = counts[i];
    t.succ[pos] = s;
}

// ------------------------------------------------------------------------------------------- draft
constexpr int DRAFT_THREADS = 256;

struct Best { unsigned long long score; uint32_t id; };
__device__ __forceinline__ bool better(unsigned long long s, uint32_t id, const Best& b) {
    return s > b.score || (s == b.score && id < b.id);
}
__device__ __forceinline__ Best block_best(Best v, Best* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long s = __shfl_xor_sync(0xFFFFFFFFu, v.score, o);
        const uint32_t id = __shfl_xor_sync(0xFFFFFFFFu, v.id, o);
        if (better(s, id, v)) { v.score = s; v.id = id; }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    Best r = red[0];
    for (int i = 1; i < DRAFT_THREADS / 32; ++i)
        if (better(red[i].score, red[i].id, r)) r = red[i];
    __syncthreads();
    return r;
}

// Warp-cooperative lookup of a packed context: each round the 32 lanes test 32 consecutive slots.
__device__ __forceinline__ bool warp_lookup(const OrderTable& t, Key key, CtxVal& out) {
    if (!t.keys) return false;
    const int lane = threadIdx.x & 31;
    const uint64_t h = key_hash(key);
    for (uint64_t round = 0; round * 32 <= t.mask; ++round) {
        const uint64_t slot = (h + round * 32 + lane) & t.mask;
        const ulonglong2 kv = *reinterpret_cast<const ulonglong2*>(t.keys + 2 * slot);
        const uint32_t hit = __ballot_sync(0xFFFFFFFFu, kv.x == key.lo && kv.y == key.hi);
        const uint32_t hole = __ballot_sync(0xFFFFFFFFu, kv.x == 0 && kv.y == 0);
        if (hit) {
            const int src = __ffs(hit) - 1;
            // all lanes read the value of the matching slot
            const uint64_t s = (h + round * 32 + src) & t.mask;
            out = t.vals[s];
            // a hole before the hit cannot exist: insertion stops at the first free slot
            return true;
        }
        if (hole) return false;
    }
    return false;
}

__global__ void __launch_bounds__(DRAFT_THREADS)
draft_kernel(const DeviceTables dt, const int32_t* __restrict__ tokens, int64_t stride, const int32_t* __restrict__ len,
             int k, uint32_t lam_num, uint32_t lam_den, int32_t* __restrict__ drafts, int hs_mask) {
    extern __shared__ int32_t dsm[];
    int32_t* h_tok = dsm;                                          // [hs] token or -1
    uint32_t* h_cnt = reinterpret_cast<uint32_t*>(dsm + hs_mask + 1);   // [hs] count, bit 31 = seen in the corpus list
    int32_t* s_seq = dsm + 2 * (hs_mask + 1);                      // [L] the committed tokens: every draft scans them twice
    __shared__ Best red[DRAFT_THREADS / 32];
    __shared__ int s_suffix[TASC_MAX_ORDER];     // last n_max tokens of the query, newest last
    __shared__ int s_nstar, s_tprompt;
    __shared__ int s_hit[TASC_MAX_ORDER];        // order n = index + 1 has a surviving context for the current suffix
    __shared__ CtxVal s_vals[TASC_MAX_ORDER];

    const int b = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5;
    int L = len[b];
    L = L < 0 ? 0 : (L > stride ? (int)stride : L);
    const int n_max = dt.n_max;
    const bool use_corp = lam_num > 0, use_prompt = lam_num < lam_den;

    for (int i = tid; i < L; i += DRAFT_THREADS) s_seq[i] = tokens[(int64_t)b * stride + i];
    __syncthreads();
    const int32_t* seq = s_seq;
    if (tid < TASC_MAX_ORDER) {
        const int p = L - n_max + tid;             // suffix slot tid <-> position p (only the last n_max slots are used)
        s_suffix[tid] = (tid < n_max && p >= 0) ? seq[p] : -1;
    }
    __syncthreads();

    for (int j = 0; j < k; ++j) {
        const int Lq = L + j;                      // query length so far
        const int n_avail = Lq < n_max ? Lq : n_max;
        // ---------------------------------------------------------------- p_corp: all orders are probed at once, one warp
        // per order (warp w looks up the last w + 1 tokens); the longest order that matched wins the back-off
        if (tid == 0) { s_nstar = 0; s_tprompt = 0; }
        if (warp < TASC_MAX_ORDER) {
            const int n = warp + 1;
            bool hit = false;
            CtxVal val = {0ull, 0u, 0u};
            if (use_corp && n <= n_avail) {
                Key key = key_make(n);
                for (int i = 0; i < n; ++i) key_put(key, i, (uint32_t)s_suffix[n_max - n + i]);
                hit = warp_lookup(dt.t[n], key, val);
            }
            if ((tid & 31) == 0) { s_hit[warp] = hit ? 1 : 0; s_vals[warp] = val; }
        }
        // ---------------------------------------------------------------- p_prompt: longest suffix match in the committed tokens
        if (use_prompt)
            for (int i = tid; i <= hs_mask; i += DRAFT_THREADS) { h_tok[i] = -1; h_cnt[i] = 0u; }
        __syncthreads();
        if (use_prompt) {
            auto match_len = [&](int p) {          // tokens before successor position p that agree with the query suffix
                int m = 0;
                const int lim = p < n_avail ? p : n_avail;
                while (m < lim && seq[p - 1 - m] == s_suffix[n_max - 1 - m]) ++m;
                return m;
            };
            int best = 0;
            for (int p = 1 + tid; p < L; p += DRAFT_THREADS) best = max(best, match_len(p));
            best = __reduce_max_sync(0xFFFFFFFFu, best);
            if ((tid & 31) == 0 && best > 0) atomicMax(&s_nstar, best);
            __syncthreads();
            const int nstar = s_nstar;
            if (nstar > 0) {
                for (int p = 1 + tid; p < L; p += DRAFT_THREADS) {
                    if (match_len(p) != nstar) continue;
                    const int x = seq[p];
                    uint32_t slot = ((uint32_t)x * 2654435761u) & hs_mask;
                    for (int probe = 0; probe <= hs_mask; ++probe) {
                        const int old = atomicCAS(&h_tok[slot], -1, x);
                        if (old == -1 || old == x) { atomicAdd(&h_cnt[slot], 1u); break; }
                        slot = (slot + 1) & hs_mask;
                    }
                    atomicAdd(&s_tprompt, 1);
                }
            }
            __syncthreads();
        }
        int found_n = 0;
        for (int n = n_max; n >= 1 && !found_n; --n)
            if (s_hit[n - 1]) found_n = n;
        const CtxVal cv = s_vals[found_n > 0 ? found_n - 1 : 0];
        const unsigned long long t_corp = cv.total;
        const unsigned long long t_prompt = (unsigned long long)s_tprompt;
        const bool has_corp = found_n > 0, has_prompt = t_prompt > 0;
        // ---------------------------------------------------------------- mixture argmax
        Best mine = {0ull, 0xFFFFFFFFu};
        bool any = false;
        if (has_corp) {
            const Succ* sl = dt.t[found_n].succ + cv.offset;
            const unsigned long long w_c = has_prompt ? (unsigned long long)lam_num * t_prompt : 1ull;
            const unsigned long long w_p = (unsigned long long)(lam_den - lam_num) * t_corp;
            for (uint32_t i = tid; i < cv.n_succ; i += DRAFT_THREADS) {
                const Succ s = sl[i];
                unsigned long long score = w_c * s.count;
                if (has_prompt) {
                    uint32_t slot = ((uint32_t)s.next * 2654435761u) & hs_mask;
                    for (int probe = 0; probe <= hs_mask; ++probe) {
                        const int tk = h_tok[slot];
                        if (tk == -1) break;
                        if (tk == s.next) {
                            const uint32_t c = atomicOr(&h_cnt[slot], 0x80000000u) & 0x7FFFFFFFu;
                            score += w_p * c;
                            break;
                        }
                        slot = (slot + 1) & hs_mask;
                    }
                }
                if (!any || better(score, (uint32_t)s.next, mine)) { mine.score = score; mine.id = (uint32_t)s.next; any = true; }
            }
        }
        __syncthreads();     // corpus pass has marked the shared successors
        if (has_prompt) {
            const unsigned long long w_p = has_corp ? (unsigned long long)(lam_den - lam_num) * t_corp : 1ull;
            for (int i = tid; i <= hs_mask; i += DRAFT_THREADS) {
                const int tk = h_tok[i];
                const uint32_t c = h_cnt[i];
                if (tk < 0 || (c & 0x80000000u)) continue;      // empty, or already scored with its corpus count
                const unsigned long long score = w_p * c;
                if (!any || better(score, (uint32_t)tk, mine)) { mine.score = score; mine.id = (uint32_t)tk; any = true; }
            }
        }
        if (!any) { mine.score = 0ull; mine.id = 0xFFFFFFFFu; }
        const Best win = block_best(mine, red);
        const int draft = (has_corp || has_prompt) ? (int)win.id : dt.fallback;
        if (tid == 0) {
            drafts[(int64_t)b * k + j] = draft;
            for (int i = 0; i + 1 < n_max; ++i) s_suffix[i] = s_suffix[i + 1];
            s_suffix[n_max - 1] = draft;
        }
        __syncthreads();
    }
}

void free_tables(DeviceTables& dt) {
    for (int n = 0; n <= TASC_MAX_ORDER; ++n) {
        if (dt.t[n].keys) cudaFree(dt.t[n].keys);
        if (dt.t[n].vals) cudaFree(dt.t[n].vals);
        if (dt.t[n].succ) cudaFree(dt.t[n].succ);
        dt.t[n] = OrderTable{nullptr, nullptr, nullptr, 0, 0};
    }
}

uint64_t pow2_at_least(uint64_t v) {
    uint64_t p = 64;
    while (p < v) p <<= 1;
    return p;
}

inline unsigned blocks_for(uint64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace
}  // namespace tasc

using namespace tasc;

extern "C" tasc_status tasc_drafter_build(const int32_t* corpus_tokens, const int64_t* doc_offsets, int64_t n_docs,
                                          int32_t n_max, int32_t p_min, int32_t vocab, tasc_stream stream_,
                                          tasc_drafter** out) {
    if (!out) return TASC_EINVAL;
    *out = nullptr;
    if (!doc_offsets || n_docs < 0 || n_max < 1 || n_max > TASC_MAX_ORDER || p_min < 1 || vocab < 1 ||
        vocab > (1 << TASC_VOCAB_BITS))
        return TASC_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::vector<int64_t> offs((size_t)n_docs + 1);
    TASC_CUDA_TRY(cudaMemcpyAsync(offs.data(), doc_offsets, offs.size() * sizeof(int64_t), cudaMemcpyDeviceToHost, stream));
    TASC_CUDA_TRY(cudaStreamSynchronize(stream));
    if (offs[0] != 0) return TASC_EINVAL;
    uint64_t windows[TASC_MAX_ORDER + 1] = {0};
    for (int64_t d = 0; d < n_docs; ++d) {
        const int64_t len = offs[d + 1] - offs[d];
        if (len < 0) return TASC_EINVAL;
        for (int n = 1; n <= n_max; ++n) windows[n] += (uint64_t)std::max<int64_t>(0, len - n);
    }
    const int64_t T = offs[n_docs];
    if (T > 0 && !corpus_tokens) return TASC_EINVAL;

    tasc_drafter* d = new (std::nothrow) tasc_drafter();
    if (!d) return TASC_ENOMEM;
    for (int n = 0; n <= TASC_MAX_ORDER; ++n) d->dt.t[n] = OrderTable{nullptr, nullptr, nullptr, 0, 0};
    d->dt.n_max = n_max; d->dt.fallback = 0; d->p_min = p_min; d->vocab = vocab;
    cudaGetDevice(&d->device);

    // scratch shared by all orders
    uint8_t* remaining = nullptr;
    uint32_t* hist = nullptr;
    unsigned long long* scalars = nullptr;     // [0] histogram argmax, [1] survivors, [2] cursor
    int* status = nullptr;
    uint64_t* skeys = nullptr;
    uint32_t* scounts = nullptr;
    uint32_t* fill = nullptr;
    const uint64_t scap = pow2_at_least(2 * std::max<uint64_t>(windows[1], 1));
    tasc_status rc = TASC_OK;
    auto fail = [&](tasc_status s) { rc = s; };
#define TRY_ALLOC(ptr, bytes) if (rc == TASC_OK && cudaMalloc(reinterpret_cast<void**>(&(ptr)), (bytes)) != cudaSuccess) { (void)cudaGetLastError(); fail(TASC_ENOMEM); }
    TRY_ALLOC(remaining, (size_t)std::max<int64_t>(T, 1));
    TRY_ALLOC(hist, (size_t)vocab * sizeof(uint32_t));
    TRY_ALLOC(scalars, 4 * sizeof(unsigned long long));
    TRY_ALLOC(status, sizeof(int));
    TRY_ALLOC(skeys, scap * 16);
    TRY_ALLOC(scounts, scap * 4);
    if (rc == TASC_OK) {
        cudaMemsetAsync(hist, 0, (size_t)vocab * sizeof(uint32_t), stream);
        cudaMemsetAsync(scalars, 0, 4 * sizeof(unsigned long long), stream);
        cudaMemsetAsync(status, 0, sizeof(int), stream);
        if (T > 0) {
            mark_remaining_kernel<<<blocks_for(T, 256), 256, 0, stream>>>(doc_offsets, n_docs, T, remaining);
            token_hist_kernel<<<blocks_for(T, 256), 256, 0, stream>>>(corpus_tokens, T, vocab, hist, status);
        }
        hist_argmax_kernel<<<blocks_for(vocab, 256), 256, 0, stream>>>(hist, vocab, scalars);
        int st = 0;
        unsigned long long best = 0;
        if (cudaMemcpyAsync(&st, status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaMemcpyAsync(&best, scalars, sizeof(best), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); fail(TASC_ECUDA); }
        else if (st != 0) fail(st);               // a token id outside [0, vocab)
        else d->dt.fallback = T > 0 ? (int)(0xFFFFFFFFu - (uint32_t)(best & 0xFFFFFFFFull)) : 0;
    }
    for (int n = 1; n <= n_max && rc == TASC_OK; ++n) {
        if (windows[n] == 0) continue;
        const uint64_t cap = pow2_at_least(2 * windows[n]);      // <= scap
        cudaMemsetAsync(skeys, 0, cap * 16, stream);
        cudaMemsetAsync(scounts, 0, cap * 4, stream);
        cudaMemsetAsync(scalars + 1, 0, 2 * sizeof(unsigned long long), stream);
        count_kernel<<<blocks_for(T, 256), 256, 0, stream>>>(corpus_tokens, remaining, T, n, skeys, scounts, cap - 1, status);
        survivors_kernel<<<blocks_for(cap, 256), 256, 0, stream>>>(scounts, cap, (uint32_t)p_min, scalars + 1);
        unsigned long long n_surv = 0;
        if (cudaMemcpyAsync(&n_surv, scalars + 1, sizeof(n_surv), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); fail(TASC_ECUDA); break; }
        if (n_surv == 0) continue;
        OrderTable& t = d->dt.t[n];
        const uint64_t ccap = pow2_at_least(2 * n_surv);
        t.mask = ccap - 1;
        t.n_succ = (long long)n_surv;
        TRY_ALLOC(t.keys, ccap * 16);
        TRY_ALLOC(t.vals, ccap * sizeof(CtxVal));
        TRY_ALLOC(t.succ, n_surv * sizeof(Succ));
        TRY_ALLOC(fill, ccap * sizeof(uint32_t));
        if (rc != TASC_OK) break;
        cudaMemsetAsync(t.keys, 0, ccap * 16, stream);
        cudaMemsetAsync(t.vals, 0, ccap * sizeof(CtxVal), stream);
        cudaMemsetAsync(fill, 0, ccap * sizeof(uint32_t), stream);
        ctx_insert_kernel<<<blocks_for(cap, 256), 256, 0, stream>>>(skeys, scounts, cap, (uint32_t)p_min, n, t, status);
        assign_offsets_kernel<<<blocks_for(ccap, 256), 256, 0, stream>>>(t, scalars + 2);
        succ_fill_kernel<<<blocks_for(cap, 256), 256, 0, stream>>>(skeys, scounts, cap, (uint32_t)p_min, n, t, fill, status);
        if (cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); fail(TASC_ECUDA); break; }
        cudaFree(fill);
        fill = nullptr;
    }
    if (rc == TASC_OK) {
        int st = 0;
        if (cudaMemcpyAsync(&st, status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); fail(TASC_ECUDA); }
        else if (st != 0) fail(st);
    }
#undef TRY_ALLOC
    if (fill) cudaFree(fill);
    if (remaining) cudaFree(remaining);
    if (hist) cudaFree(hist);
    if (scalars) cudaFree(scalars);
    if (status) cudaFree(status);
    if (skeys) cudaFree(skeys);
    if (scounts) cudaFree(scounts);
    if (rc != TASC_OK) {
        free_tables(d->dt);
        delete d;
        return rc;
    }
    *out = d;
    return TASC_OK;
}

extern "C" tasc_status tasc_drafter_export(const tasc_drafter* d, tasc_ngram_entry* out, int64_t cap, int64_t* n_entries,
                                           int32_t* fallback_token) {
    if (!d || !n_entries || cap < 0 || (cap > 0 && !out)) return TASC_EINVAL;
    int64_t total = 0;
    for (int n = 1; n <= d->dt.n_max; ++n) total += d->dt.t[n].n_succ;
    *n_entries = total;
    if (fallback_token) *fallback_token = d->dt.fallback;
    if (cap < total) return cap == 0 ? TASC_OK : TASC_ECAPACITY;
    int64_t w = 0;
    for (int n = 1; n <= d->dt.n_max; ++n) {
        const OrderTable& t = d->dt.t[n];
        if (!t.keys) continue;
        const uint64_t ccap = t.mask + 1;
        std::vector<uint64_t> keys(ccap * 2);
        std::vector<CtxVal> vals(ccap);
        std::vector<Succ> succ((size_t)t.n_succ);
        TASC_CUDA_TRY(cudaMemcpy(keys.data(), t.keys, ccap * 16, cudaMemcpyDeviceToHost));
        TASC_CUDA_TRY(cudaMemcpy(vals.data(), t.vals, ccap * sizeof(CtxVal), cudaMemcpyDeviceToHost));
        TASC_CUDA_TRY(cudaMemcpy(succ.data(), t.succ, succ.size() * sizeof(Succ), cudaMemcpyDeviceToHost));
        for (uint64_t s = 0; s < ccap; ++s) {
            if (!(keys[2 * s + 1] & VALID_BIT)) continue;
            const Key k = {keys[2 * s], keys[2 * s + 1]};
            for (uint32_t i = 0; i < vals[s].n_succ; ++i) {
                const uint64_t pos = vals[s].offset + i;
                if (pos >= succ.size() || w >= total) return TASC_ECAPACITY;
                tasc_ngram_entry& e = out[w++];
                e.n = n;
                for (int j = 0; j < TASC_MAX_ORDER; ++j) e.ctx[j] = j < n ? (int32_t)key_get(k, j) : -1;
                e.next = succ[pos].next;
                e.count = succ[pos].count;
            }
        }
    }
    std::sort(out, out + w, [](const tasc_ngram_entry& a, const tasc_ngram_entry& b) {
        if (a.n != b.n) return a.n < b.n;
        for (int j = 0; j < TASC_MAX_ORDER; ++j)
            if (a.ctx[j] != b.ctx[j]) return a.ctx[j] < b.ctx[j];
        return a.next < b.next;
    });
    return w == total ? TASC_OK : TASC_ECAPACITY;
}

extern "C" tasc_status tasc_drafter_destroy(tasc_drafter* d) {
    if (!d) return TASC_EINVAL;
    free_tables(d->dt);
    delete d;
    return TASC_OK;
}

extern "C" tasc_status tasc_draft(const tasc_drafter* d, const int32_t* tokens, int64_t stride, const int32_t* len,
                                  int32_t B, int32_t k, int32_t lambda_num, int32_t lambda_den, int32_t* drafts,
                                  tasc_stream stream) {
    if (!d || !tokens || !len || !drafts || B < 1 || k < 1 || k > TASC_MAX_ROWS - 1 || stride < 1 || stride > 12288 ||
        lambda_den < 1 || lambda_den > 256 || lambda_num < 0 || lambda_num > lambda_den)
        return TASC_EINVAL;
    uint64_t hs = 64;
    while (hs * 3 < (uint64_t)stride * 4) hs <<= 1;      // load factor <= 3/4
    const size_t smem = hs * 8 + (size_t)stride * sizeof(int32_t);      // hash of the context successors + the tokens
    static bool attr = false;
    if (!attr) {
        TASC_CUDA_TRY(cudaFuncSetAttribute(draft_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 184 * 1024));
        attr = true;
    }
    ProfScope ps(K_DRAFT, static_cast<cudaStream_t>(stream));
    draft_kernel<<<B, DRAFT_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(
        d->dt, tokens, stride, len, k, (uint32_t)lambda_num, (uint32_t)lambda_den, drafts, (int)(hs - 1));
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}
