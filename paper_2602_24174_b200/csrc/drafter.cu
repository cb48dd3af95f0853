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
#include "ngram_table.cuh"

#include <algorithm>
#include <cmath>
#include <mutex>
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


// Order-1 model with one successor of count 1 per context: context token c -> table[c].
__global__ void bigram_insert_kernel(const int32_t* __restrict__ table, int vocab, OrderTable t, int* status) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= vocab) return;
    const int x = table[c];
    if (x < 0 || x >= vocab) { set_status(status, TASC_EINVAL); return; }
    Key key = key_make(1);
    key_put(key, 0, (uint32_t)c);
    const uint64_t slot = table_upsert(t.keys, t.mask, key);
    if (slot == ~0ull) { set_status(status, TASC_ECAPACITY); return; }
    CtxVal v;
    v.offset = (unsigned long long)c; v.n_succ = 1u; v.total = 1u;
    t.vals[slot] = v;
    Succ sc;
    sc.next = x; sc.count = 1u;
    t.succ[c] = sc;
}

// ------------------------------------------------------------------------------------------- corpus statistics
// The statistics are functions of the multiset of counts only, so the device first turns the count table into a
// histogram of count VALUES (how many bigrams occur c times), which is exact integer work whose result does not
// depend on where the hash table put anything; one block then walks that histogram in a fixed order.
constexpr int CC_BITS = 20;                       // count values below 2^20 have a histogram bin of their own
constexpr uint32_t CC_BINS = 1u << CC_BITS;
constexpr int CC_OVERFLOW = 4096;                 // larger count values are listed individually
constexpr int STATS_THREADS = 1024;

// [0] distinct keys, [1] overflow entries, [2] sum of squared counts
__global__ void count_values_kernel(const uint32_t* __restrict__ counts, uint64_t n, uint32_t* __restrict__ bins,
                                    uint32_t* __restrict__ overflow, unsigned long long* __restrict__ scal, int* status) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t c = i < n ? counts[i] : 0u;
    unsigned long long sq = (unsigned long long)c * c;
    unsigned int nz = c ? 1u : 0u;
    if (c) {
        if (c < CC_BINS) atomicAdd(&bins[c], 1u);
        else {
            const unsigned long long at = atomicAdd(&scal[1], 1ull);
            if (at < CC_OVERFLOW) overflow[at] = c; else set_status(status, TASC_ECAPACITY);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
        nz += __shfl_xor_sync(0xFFFFFFFFu, nz, o);
    }
    if ((threadIdx.x & 31) == 0 && nz) {
        atomicAdd(&scal[0], (unsigned long long)nz);
        atomicAdd(&scal[2], sq);                   // integer sums: the order of the additions does not matter
    }
}

struct CountSummary {
    unsigned long long n_total;      // sum of the counts
    unsigned long long n_distinct;
    unsigned long long sum_sq;
    unsigned long long n_for_cdf;    // smallest number of the largest counts that reach cdf_num / cdf_den of n_total
    double sum_c_log2_c;             // sum over all keys of c log2 c
};

// One block.  bins[c] = number of keys with count c (c < 2^20), overflow[] = the counts >= 2^20.  Walks the count
// values from the largest down: thread t owns a contiguous range of bins, an exclusive scan over the threads
// gives the mass and the number of keys above its range, and the thread whose range holds the crossing of the
// coverage target finishes the count by itself.  Sums are taken in a fixed order, so the result is reproducible.
__global__ void __launch_bounds__(STATS_THREADS)
count_summary_kernel(const uint32_t* __restrict__ bins, uint32_t* __restrict__ overflow, const unsigned long long* __restrict__ scal,
                     unsigned long long cdf_num, unsigned long long cdf_den, CountSummary* out) {
    __shared__ unsigned long long s_mass[STATS_THREADS], s_keys[STATS_THREADS];
    __shared__ double s_log[STATS_THREADS];
    __shared__ uint32_t s_over[CC_OVERFLOW];
    __shared__ unsigned long long s_result, s_over_mass;
    __shared__ double s_over_log;
    const int t = threadIdx.x;
    const int n_over = (int)min(scal[1], (unsigned long long)CC_OVERFLOW);
    // the overflow list, largest first: rank by counting (a few thousand entries at most)
    for (int i = t; i < n_over; i += STATS_THREADS) {
        const uint32_t c = overflow[i];
        int rank = 0;
        for (int j = 0; j < n_over; ++j) {
            const uint32_t o = overflow[j];
            rank += (o > c || (o == c && j < i)) ? 1 : 0;
        }
        s_over[rank] = c;
    }
    __syncthreads();
    if (t == 0) {
        unsigned long long m = 0;
        double l = 0.0;
        for (int i = 0; i < n_over; ++i) { m += s_over[i]; l += (double)s_over[i] * log2((double)s_over[i]); }
        s_over_mass = m; s_over_log = l; s_result = 0ull;
    }
    // thread t owns bins hi, hi - 1, ..., lo (descending count values)
    constexpr uint32_t PER = CC_BINS / STATS_THREADS;
    const uint32_t hi = CC_BINS - 1u - (uint32_t)t * PER, lo = hi - (PER - 1u);
    unsigned long long mass = 0, keys = 0;
    double lg = 0.0;
    for (uint32_t c = hi; ; --c) {
        const uint32_t m = c ? bins[c] : 0u;
        if (m) { mass += (unsigned long long)m * c; keys += m; lg += (double)m * ((double)c * log2((double)c)); }
        if (c == lo) break;
    }
    s_mass[t] = mass; s_keys[t] = keys; s_log[t] = lg;
    __syncthreads();
    if (t == 0) {
        // serial exclusive scan over the 1,024 partial sums (fixed order)
        unsigned long long m = s_over_mass, k = (unsigned long long)n_over;
        double l = s_over_log;
        for (int i = 0; i < STATS_THREADS; ++i) {
            const unsigned long long mi = s_mass[i], ki = s_keys[i];
            l += s_log[i];
            s_mass[i] = m; s_keys[i] = k;
            m += mi; k += ki;
        }
        out->n_total = m; out->n_distinct = k; out->sum_sq = scal[2]; out->sum_c_log2_c = l;
        s_over_mass = m;                                     // total mass, for the threads below
    }
    __syncthreads();
    const unsigned long long total = s_over_mass;
    if (total == 0) { if (t == 0) out->n_for_cdf = 0; return; }
    // target: smallest run with run * den >= num * total.  128-bit products are not needed: total < 2^40, num, den <= 2^16.
    const unsigned long long need = (cdf_num * total + cdf_den - 1) / cdf_den;
    if (t == 0) {
        // crossing inside the overflow list?
        unsigned long long run = 0;
        for (int i = 0; i < n_over; ++i) {
            run += s_over[i];
            if (run >= need) { s_result = (unsigned long long)i + 1; break; }
        }
    }
    __syncthreads();
    const unsigned long long above = s_mass[t];
    if (s_result == 0 && above < need && above + mass >= need) {
        unsigned long long run = above, k = s_keys[t];
        for (uint32_t c = hi; ; --c) {
            const uint32_t m = c ? bins[c] : 0u;
            if (m) {
                if (run + (unsigned long long)m * c >= need) {
                    k += (need - run + c - 1) / c;
                    break;
                }
                run += (unsigned long long)m * c; k += m;
            }
            if (c == lo) break;
        }
        s_result = k;
    }
    __syncthreads();
    if (t == 0) out->n_for_cdf = s_result;
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

extern "C" tasc_status tasc_drafter_from_bigram(const int32_t* table, int32_t vocab, tasc_stream stream_, tasc_drafter** out) {
    if (!out) return TASC_EINVAL;
    *out = nullptr;
    if (!table || vocab < 1 || vocab > (1 << TASC_VOCAB_BITS)) return TASC_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    tasc_drafter* d = new (std::nothrow) tasc_drafter();
    if (!d) return TASC_ENOMEM;
    for (int n = 0; n <= TASC_MAX_ORDER; ++n) d->dt.t[n] = OrderTable{nullptr, nullptr, nullptr, 0, 0};
    d->dt.n_max = 1; d->dt.fallback = 0; d->p_min = 1; d->vocab = vocab;
    cudaGetDevice(&d->device);
    OrderTable& t = d->dt.t[1];
    const uint64_t cap = pow2_at_least(2 * (uint64_t)vocab);
    t.mask = cap - 1;
    t.n_succ = vocab;
    int* status = nullptr;
    tasc_status rc = TASC_OK;
    if (cudaMalloc(reinterpret_cast<void**>(&t.keys), cap * 16) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&t.vals), cap * sizeof(CtxVal)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&t.succ), (size_t)vocab * sizeof(Succ)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&status), sizeof(int)) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ENOMEM; }
    if (rc == TASC_OK) {
        cudaMemsetAsync(t.keys, 0, cap * 16, stream);
        cudaMemsetAsync(t.vals, 0, cap * sizeof(CtxVal), stream);
        cudaMemsetAsync(status, 0, sizeof(int), stream);
        bigram_insert_kernel<<<blocks_for((uint64_t)vocab, 256), 256, 0, stream>>>(table, vocab, t, status);
        int st = 0;
        if (cudaMemcpyAsync(&st, status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ECUDA; }
        else if (st != 0) rc = st;
    }
    if (status) cudaFree(status);
    if (rc != TASC_OK) {
        free_tables(d->dt);
        delete d;
        return rc;
    }
    *out = d;
    return TASC_OK;
}

extern "C" tasc_status tasc_corpus_stats(const int32_t* corpus_tokens, const int64_t* doc_offsets, int64_t n_docs, int32_t vocab,
                                         int32_t cdf_num, int32_t cdf_den, tasc_stream stream_, tasc_corpus_statistics* out) {
    if (!out || !doc_offsets || n_docs < 0 || vocab < 1 || vocab > (1 << TASC_VOCAB_BITS) || cdf_den < 1 || cdf_den > 65536 ||
        cdf_num < 1 || cdf_num > cdf_den)
        return TASC_EINVAL;
    *out = tasc_corpus_statistics{};
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::vector<int64_t> offs((size_t)n_docs + 1);
    TASC_CUDA_TRY(cudaMemcpyAsync(offs.data(), doc_offsets, offs.size() * sizeof(int64_t), cudaMemcpyDeviceToHost, stream));
    TASC_CUDA_TRY(cudaStreamSynchronize(stream));
    if (offs[0] != 0) return TASC_EINVAL;
    uint64_t pairs = 0;
    for (int64_t d = 0; d < n_docs; ++d) {
        const int64_t len = offs[d + 1] - offs[d];
        if (len < 0) return TASC_EINVAL;
        pairs += (uint64_t)std::max<int64_t>(0, len - 1);
    }
    const int64_t T = offs[n_docs];
    if (T > 0 && !corpus_tokens) return TASC_EINVAL;
    if ((uint64_t)T >= (1ull << 40)) return TASC_EINVAL;

    uint8_t* remaining = nullptr;
    uint32_t *hist = nullptr, *bins = nullptr, *overflow = nullptr, *scounts = nullptr;
    unsigned long long* scal = nullptr;      // [0..2] bigram scalars, [4..6] token scalars
    CountSummary* summ = nullptr;            // [0] bigrams, [1] tokens
    int* status = nullptr;
    uint64_t* skeys = nullptr;
    const uint64_t cap = pow2_at_least(2 * std::max<uint64_t>(pairs, 1));
    tasc_status rc = TASC_OK;
#define TRY_ALLOC(ptr, bytes) if (rc == TASC_OK && cudaMalloc(reinterpret_cast<void**>(&(ptr)), (bytes)) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ENOMEM; }
    TRY_ALLOC(remaining, (size_t)std::max<int64_t>(T, 1));
    TRY_ALLOC(hist, (size_t)vocab * sizeof(uint32_t));
    TRY_ALLOC(bins, 2 * (size_t)CC_BINS * sizeof(uint32_t));
    TRY_ALLOC(overflow, 2 * (size_t)CC_OVERFLOW * sizeof(uint32_t));
    TRY_ALLOC(scal, 8 * sizeof(unsigned long long));
    TRY_ALLOC(summ, 2 * sizeof(CountSummary));
    TRY_ALLOC(status, sizeof(int));
    TRY_ALLOC(skeys, cap * 16);
    TRY_ALLOC(scounts, cap * 4);
#undef TRY_ALLOC
    CountSummary h[2] = {};
    if (rc == TASC_OK) {
        cudaMemsetAsync(hist, 0, (size_t)vocab * sizeof(uint32_t), stream);
        cudaMemsetAsync(bins, 0, 2 * (size_t)CC_BINS * sizeof(uint32_t), stream);
        cudaMemsetAsync(scal, 0, 8 * sizeof(unsigned long long), stream);
        cudaMemsetAsync(status, 0, sizeof(int), stream);
        cudaMemsetAsync(skeys, 0, cap * 16, stream);
        cudaMemsetAsync(scounts, 0, cap * 4, stream);
        if (T > 0) {
            mark_remaining_kernel<<<blocks_for(T, 256), 256, 0, stream>>>(doc_offsets, n_docs, T, remaining);
            token_hist_kernel<<<blocks_for(T, 256), 256, 0, stream>>>(corpus_tokens, T, vocab, hist, status);
            // bigrams = the windows of the order-1 model before pruning: (token, next) inside one document
            count_kernel<<<blocks_for(T, 256), 256, 0, stream>>>(corpus_tokens, remaining, T, 1, skeys, scounts, cap - 1, status);
        }
        count_values_kernel<<<blocks_for(cap, 256), 256, 0, stream>>>(scounts, cap, bins, overflow, scal, status);
        count_values_kernel<<<blocks_for(vocab, 256), 256, 0, stream>>>(hist, (uint64_t)vocab, bins + CC_BINS, overflow + CC_OVERFLOW, scal + 4, status);
        count_summary_kernel<<<1, STATS_THREADS, 0, stream>>>(bins, overflow, scal, (unsigned long long)cdf_num, (unsigned long long)cdf_den, summ);
        count_summary_kernel<<<1, STATS_THREADS, 0, stream>>>(bins + CC_BINS, overflow + CC_OVERFLOW, scal + 4, 1ull, 1ull, summ + 1);
        int st = 0;
        if (cudaMemcpyAsync(h, summ, sizeof(h), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaMemcpyAsync(&st, status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ECUDA; }
        else if (st != 0) rc = st;
    }
    cudaFree(remaining); cudaFree(hist); cudaFree(bins); cudaFree(overflow); cudaFree(scal); cudaFree(summ);
    cudaFree(status); cudaFree(skeys); cudaFree(scounts);
    if (rc != TASC_OK) return rc;
    // the closing arithmetic on a handful of scalars: H = log2 N - (sum c log2 c) / N;  H_2 = 2 log2 N - log2 sum c^2
    auto entropy = [](const CountSummary& c) { return c.n_total ? log2((double)c.n_total) - c.sum_c_log2_c / (double)c.n_total : 0.0; };
    out->n_tokens = T;
    out->n_bigrams = (int64_t)h[0].n_total;
    out->n_unique_tokens = (int64_t)h[1].n_distinct;
    out->n_unique_bigrams = (int64_t)h[0].n_distinct;
    out->bigrams_for_cdf = (int64_t)h[0].n_for_cdf;
    out->bigram_entropy_bits = entropy(h[0]);
    out->typical_set_size = exp2(out->bigram_entropy_bits);
    out->token_entropy_bits = entropy(h[1]);
    out->token_entropy_normalised = vocab > 1 ? out->token_entropy_bits / log2((double)vocab) : 0.0;
    out->token_renyi2_bits = h[1].n_total ? 2.0 * log2((double)h[1].n_total) - log2((double)h[1].sum_sq) : 0.0;
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

extern "C" tasc_status tasc_drafter_import(const tasc_ngram_entry* entries, int64_t n_entries, int32_t n_max, int32_t vocab,
                                           int32_t fallback_token, tasc_stream stream_, tasc_drafter** out) {
    if (!out) return TASC_EINVAL;
    *out = nullptr;
    if (n_entries < 0 || (n_entries > 0 && !entries) || n_max < 1 || n_max > TASC_MAX_ORDER || vocab < 1 ||
        vocab > (1 << TASC_VOCAB_BITS) || fallback_token < 0 || fallback_token >= vocab)
        return TASC_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // the packed (context, next) keys and counts of every order, in the form the build's compaction kernels read
    std::vector<std::vector<uint64_t>> keys((size_t)n_max + 1);
    std::vector<std::vector<uint32_t>> counts((size_t)n_max + 1);
    for (int64_t i = 0; i < n_entries; ++i) {
        const tasc_ngram_entry& e = entries[i];
        if (e.n < 1 || e.n > n_max || e.next < 0 || e.next >= vocab || e.count < 1) return TASC_EINVAL;
        Key k = key_make(e.n);
        for (int j = 0; j < e.n; ++j) {
            if (e.ctx[j] < 0 || e.ctx[j] >= vocab) return TASC_EINVAL;
            key_put(k, j, (uint32_t)e.ctx[j]);
        }
        key_put(k, e.n, (uint32_t)e.next);
        keys[e.n].push_back(k.lo);
        keys[e.n].push_back(k.hi);
        counts[e.n].push_back(e.count);
    }
    tasc_drafter* d = new (std::nothrow) tasc_drafter();
    if (!d) return TASC_ENOMEM;
    for (int n = 0; n <= TASC_MAX_ORDER; ++n) d->dt.t[n] = OrderTable{nullptr, nullptr, nullptr, 0, 0};
    d->dt.n_max = n_max; d->dt.fallback = fallback_token; d->p_min = 1; d->vocab = vocab;
    cudaGetDevice(&d->device);
    tasc_status rc = TASC_OK;
    int* status = nullptr;
    unsigned long long* cursor = nullptr;
    if (cudaMalloc(reinterpret_cast<void**>(&status), sizeof(int)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&cursor), sizeof(unsigned long long)) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ENOMEM; }
    if (rc == TASC_OK) cudaMemsetAsync(status, 0, sizeof(int), stream);
    for (int n = 1; n <= n_max && rc == TASC_OK; ++n) {
        const uint64_t cnt = counts[n].size();
        if (cnt == 0) continue;
        uint64_t* skeys = nullptr;
        uint32_t *scounts = nullptr, *fill = nullptr;
        OrderTable& t = d->dt.t[n];
        const uint64_t ccap = pow2_at_least(2 * cnt);
        t.mask = ccap - 1;
        t.n_succ = (long long)cnt;
        if (cudaMalloc(reinterpret_cast<void**>(&skeys), cnt * 16) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&scounts), cnt * 4) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&fill), ccap * 4) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&t.keys), ccap * 16) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&t.vals), ccap * sizeof(CtxVal)) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&t.succ), cnt * sizeof(Succ)) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ENOMEM; }
        if (rc == TASC_OK) {
            cudaMemcpyAsync(skeys, keys[n].data(), cnt * 16, cudaMemcpyHostToDevice, stream);
            cudaMemcpyAsync(scounts, counts[n].data(), cnt * 4, cudaMemcpyHostToDevice, stream);
            cudaMemsetAsync(t.keys, 0, ccap * 16, stream);
            cudaMemsetAsync(t.vals, 0, ccap * sizeof(CtxVal), stream);
            cudaMemsetAsync(fill, 0, ccap * 4, stream);
            cudaMemsetAsync(cursor, 0, sizeof(unsigned long long), stream);
            ctx_insert_kernel<<<blocks_for(cnt, 256), 256, 0, stream>>>(skeys, scounts, cnt, 1u, n, t, status);
            assign_offsets_kernel<<<blocks_for(ccap, 256), 256, 0, stream>>>(t, cursor);
            succ_fill_kernel<<<blocks_for(cnt, 256), 256, 0, stream>>>(skeys, scounts, cnt, 1u, n, t, fill, status);
            if (cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ECUDA; }
        }
        if (skeys) cudaFree(skeys);
        if (scounts) cudaFree(scounts);
        if (fill) cudaFree(fill);
    }
    if (rc == TASC_OK) {
        int st = 0;
        if (cudaMemcpy(&st, status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ECUDA; }
        else if (st != 0) rc = st;
    }
    if (status) cudaFree(status);
    if (cursor) cudaFree(cursor);
    if (rc != TASC_OK) {
        free_tables(d->dt);
        delete d;
        return rc;
    }
    *out = d;
    return TASC_OK;
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
    {
        // the attribute belongs to the device: set once per device, under a lock (two threads may make their first call together)
        static std::mutex mu;
        static bool attr_done[64] = {false};
        int dev = 0;
        TASC_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return TASC_EINVAL;
        std::lock_guard<std::mutex> lk(mu);
        if (!attr_done[dev]) {
            TASC_CUDA_TRY(cudaFuncSetAttribute(draft_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 184 * 1024));
            attr_done[dev] = true;
        }
    }
    ProfScope ps(K_DRAFT, static_cast<cudaStream_t>(stream));
    draft_kernel<<<B, DRAFT_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(
        d->dt, tokens, stride, len, k, (uint32_t)lambda_num, (uint32_t)lambda_den, drafts, (int)(hs - 1));
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}
