// Tokenizer enrichment (TASC-tok, Section 4 of the paper) on the device.
//
// tasc_tok_enrich -- Algorithm 1: starting from the base vocabulary, every iteration counts the token n-grams
// (2 <= n <= n_max) of the task corpus as it is tokenised with the current vocabulary, scores each with the merge
// reward f_merge(t^n) = freq(t^n) * (n - 1) (Section 4.1), takes the argmax, adds it as one new token and replaces its
// occurrences (left to right, non-overlapping, inside each document) before the next iteration.  The prefix-collision
// test of the paper needs the tokens' strings; ids have none, so every candidate passes.
//   Counting is the drafter's machinery: one open-addressing table keyed by the full packing of (n, tokens), one
//   128-bit compare-and-swap per window, plus an atomic minimum of the window's position, which makes the argmax
//   unique: largest reward, then the longer n-gram, then the one that occurs first.  The documents stay at their
//   original offsets and only get shorter, so a thread per document can rewrite its document in place.
//   All iterations are enqueued without a host round trip; an iteration that finds nothing to merge (and every later
//   one) does nothing.
// tasc_tok_init_rows -- Section 4.2: the embedding / LM-head row of an added token is the mean of its constituents'
//   rows (a constituent may itself be an added token).  One thread per column walks the merges in order, so a row is
//   always complete when a later row needs it, with no synchronisation.
// tasc_tok_encode -- Appendix on byte-pair encoding: text is encoded with the added tokens matched first and greedily
//   (the longest added token whose expansion into base tokens matches the upcoming base tokens).  The added tokens'
//   expansions form a trie stored as a hash of (node, token) -> child; a thread per document walks it.
#include "kernels.h"
#include "ngram_table.cuh"

#include <algorithm>
#include <map>
#include <vector>

namespace tasc {
namespace {

constexpr int MAX_N = TASC_TOK_MAX_N;            // longest n-gram (the key holds six ids)
constexpr int POS_BITS = 28;                     // window positions are below 2^28
constexpr int LEN_BITS = 3;

struct Winner { int n; int tok[MAX_N]; int done; };

// One window (n tokens starting at i) per thread and n-gram length; rem[i] = tokens after i inside its document.
__global__ void tok_count_kernel(const int32_t* __restrict__ cur, const uint8_t* __restrict__ rem, int64_t T, int n,
                                 uint64_t* keys, uint32_t* counts, uint32_t* first, uint64_t mask, const Winner* w, int* status) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (w->done || i >= T || rem[i] < n - 1) return;
    Key key = key_make(n);
    for (int j = 0; j < n; ++j) key_put(key, j, (uint32_t)cur[i + j]);
    const uint64_t slot = table_upsert(keys, mask, key);
    if (slot == ~0ull) { set_status(status, TASC_ECAPACITY); return; }
    atomicAdd(&counts[slot], 1u);
    atomicMin(&first[slot], (uint32_t)i);
}

// reward (33 bits) | n (3 bits) | 2^28 - 1 - first position (28 bits): one unsigned maximum picks the largest
// reward, then the longer n-gram, then the earlier first occurrence
__device__ __forceinline__ unsigned long long tok_rank(uint32_t count, int n, uint32_t first) {
    const unsigned long long reward = (unsigned long long)count * (unsigned long long)(n - 1);
    return (reward << (LEN_BITS + POS_BITS)) | ((unsigned long long)n << POS_BITS) |
           (unsigned long long)(((1u << POS_BITS) - 1u) - first);
}
__device__ __forceinline__ int key_order(const Key& k) { return (int)((k.hi >> 56) & 0x7Full); }

__global__ void tok_best_kernel(const uint64_t* __restrict__ keys, const uint32_t* __restrict__ counts,
                                const uint32_t* __restrict__ first, uint64_t cap, unsigned long long* best, const Winner* w) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long r = 0;
    if (!w->done && i < cap && counts[i]) {
        const Key k = {keys[2 * i], keys[2 * i + 1]};
        r = tok_rank(counts[i], key_order(k), first[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long x = __shfl_xor_sync(0xFFFFFFFFu, r, o);
        r = x > r ? x : r;
    }
    if ((threadIdx.x & 31) == 0 && r) atomicMax(best, r);
}

// The slot whose rank equals the maximum is the iteration's n-gram t*: recorded as merge number *n_merges.
__global__ void tok_winner_kernel(const uint64_t* __restrict__ keys, const uint32_t* __restrict__ counts,
                                  const uint32_t* __restrict__ first, uint64_t cap, const unsigned long long* best,
                                  Winner* w, int32_t* merges, int* n_merges) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (w->done) return;
    const unsigned long long b = *best;
    if (b == 0ull) {                                   // no n-gram left: this and every later iteration is empty
        if (i == 0) { w->n = 0; }
        return;
    }
    if (i >= cap || !counts[i]) return;
    const Key k = {keys[2 * i], keys[2 * i + 1]};
    const int n = key_order(k);
    if (tok_rank(counts[i], n, first[i]) != b) return;
    const int at = *n_merges;                           // one thread gets here
    w->n = n;
    for (int j = 0; j < MAX_N; ++j) {
        const int t = j < n ? (int)key_get(k, j) : -1;
        w->tok[j] = t;
        merges[(size_t)at * MAX_N + j] = t;
    }
}

// After the search: close the iteration (count the merge, or mark the procedure as finished).
__global__ void tok_commit_kernel(Winner* w, int* n_merges, unsigned long long* best) {
    if (w->done) return;
    if (*best == 0ull || w->n == 0) w->done = 1;
    else *n_merges += 1;
    *best = 0ull;
}

// One thread per document: replaces the occurrences of t* (left to right, non-overlapping) by the new id, in place,
// and rewrites the document's remaining-token counts.  new_id = base_vocab + (*n_merges - 1) after the commit.
__global__ void tok_rewrite_kernel(int32_t* cur, uint8_t* rem, const int64_t* __restrict__ doc_start, int32_t* doc_len,
                                   int64_t n_docs, const Winner* w, const int* n_merges, int base_vocab) {
    const int64_t d = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= n_docs || w->done) return;
    const int n = w->n;
    const int new_id = base_vocab + *n_merges - 1;
    int t[MAX_N];
#pragma unroll
    for (int j = 0; j < MAX_N; ++j) t[j] = w->tok[j];
    int32_t* doc = cur + doc_start[d];
    uint8_t* r = rem + doc_start[d];
    const int L = doc_len[d];
    int rd = 0, wr = 0;
    while (rd < L) {
        bool hit = rd + n <= L;
        for (int j = 0; hit && j < n; ++j) hit = doc[rd + j] == t[j];
        if (hit) { doc[wr++] = new_id; rd += n; }
        else { doc[wr++] = doc[rd++]; }
    }
    if (wr == L) return;                                // nothing replaced: counts unchanged
    doc_len[d] = wr;
    for (int j = 0; j < L; ++j) {
        const int left = wr - 1 - j;
        r[j] = (uint8_t)(left < 0 ? 0 : (left > 255 ? 255 : left));
    }
}

__global__ void tok_init_docs_kernel(const int64_t* __restrict__ offsets, int64_t n_docs, int64_t* doc_start, int32_t* doc_len,
                                     uint8_t* rem) {
    const int64_t d = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= n_docs) return;
    const int64_t s = offsets[d];
    const int L = (int)(offsets[d + 1] - s);
    doc_start[d] = s;
    doc_len[d] = L;
    for (int j = 0; j < L; ++j) {
        const int left = L - 1 - j;
        rem[s + j] = (uint8_t)(left > 255 ? 255 : left);
    }
}

// Exclusive scan of the document lengths into offsets (one block; each thread owns a contiguous run of documents).
__global__ void __launch_bounds__(1024)
tok_scan_kernel(const int32_t* __restrict__ doc_len, int64_t n_docs, int64_t* offsets_out) {
    __shared__ long long part[1024];
    const int t = threadIdx.x;
    const int64_t per = (n_docs + 1023) / 1024;
    const int64_t lo = min(n_docs, (int64_t)t * per), hi = min(n_docs, lo + per);
    long long s = 0;
    for (int64_t d = lo; d < hi; ++d) s += doc_len[d];
    part[t] = s;
    __syncthreads();
    if (t == 0) {
        long long run = 0;
        for (int i = 0; i < 1024; ++i) { const long long v = part[i]; part[i] = run; run += v; }
        offsets_out[n_docs] = run;
    }
    __syncthreads();
    long long run = part[t];
    for (int64_t d = lo; d < hi; ++d) { offsets_out[d] = run; run += doc_len[d]; }
}
__global__ void tok_compact_kernel(const int32_t* __restrict__ cur, const int64_t* __restrict__ doc_start,
                                   const int32_t* __restrict__ doc_len, const int64_t* __restrict__ offsets_out,
                                   int64_t n_docs, int32_t* tokens_out) {
    const int64_t d = blockIdx.x;
    if (d >= n_docs) return;
    const int32_t* src = cur + doc_start[d];
    int32_t* dst = tokens_out + offsets_out[d];
    for (int j = threadIdx.x; j < doc_len[d]; j += blockDim.x) dst[j] = src[j];
}

// ------------------------------------------------------------------------------------------- new rows
template <typename T>
__global__ void tok_rows_kernel(const T* __restrict__ base, int base_vocab, int d, const int32_t* __restrict__ merges,
                                int n_merges, T* rows_out, int* status) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    for (int i = 0; i < n_merges; ++i) {
        float acc = 0.f;
        int n = 0;
        for (int c = 0; c < MAX_N; ++c) {
            const int t = merges[(size_t)i * MAX_N + c];
            if (t < 0) break;
            float v = 0.f;
            if (t < base_vocab) v = Num<T>::to_f(base[(size_t)t * d + j]);
            else if (t - base_vocab < i) v = Num<T>::to_f(rows_out[(size_t)(t - base_vocab) * d + j]);   // written by this thread
            else set_status(status, TASC_EINVAL);                                                      // a constituent that does not exist yet
            acc += v;
            ++n;
        }
        if (n < 2) { set_status(status, TASC_EINVAL); n = 1; }
        rows_out[(size_t)i * d + j] = Num<T>::from_f(acc / (float)n);
    }
}

// ------------------------------------------------------------------------------------------- encode
struct TrieTable { const uint64_t* keys; const int32_t* child; const int32_t* token; uint64_t mask; };

__device__ __forceinline__ uint64_t trie_hash(uint64_t k) {
    k ^= k >> 33; k *= 0xFF51AFD7ED558CCDull; k ^= k >> 33; k *= 0xC4CEB9FE1A85EC53ull; k ^= k >> 33;
    return k;
}
// child of `node` along `tok`, or -1
__device__ __forceinline__ int trie_step(const TrieTable& t, int node, int tok) {
    const uint64_t key = ((uint64_t)(uint32_t)node << 32) | (uint64_t)(uint32_t)tok | (1ull << 63);
    uint64_t slot = trie_hash(key) & t.mask;
    for (uint64_t probe = 0; probe <= t.mask; ++probe) {
        const uint64_t k = t.keys[slot];
        if (k == key) return t.child[slot];
        if (k == 0ull) return -1;
        slot = (slot + 1) & t.mask;
    }
    return -1;
}

// One thread per document: at every position the longest added token whose expansion matches, else the base token.
// Output in place of a scratch copy at the document's original offset; lengths to doc_len.
__global__ void tok_encode_kernel(const int32_t* __restrict__ tokens, const int64_t* __restrict__ offsets, int64_t n_docs,
                                  TrieTable trie, int32_t* scratch, int64_t* doc_start, int32_t* doc_len) {
    const int64_t d = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= n_docs) return;
    const int64_t s = offsets[d];
    const int L = (int)(offsets[d + 1] - s);
    const int32_t* doc = tokens + s;
    int32_t* out = scratch + s;
    int i = 0, w = 0;
    while (i < L) {
        int node = 0, best_tok = -1, best_len = 0;
        for (int j = i; j < L; ++j) {
            node = trie_step(trie, node, doc[j]);
            if (node < 0) break;
            const int tk = trie.token[node];
            if (tk >= 0) { best_tok = tk; best_len = j - i + 1; }
        }
        if (best_tok >= 0) { out[w++] = best_tok; i += best_len; }
        else { out[w++] = doc[i++]; }
    }
    doc_start[d] = s;
    doc_len[d] = w;
}

tasc_status compact_docs(const int32_t* cur, const int64_t* doc_start, const int32_t* doc_len, int64_t n_docs,
                         int32_t* tokens_out, int64_t* offsets_out, cudaStream_t stream) {
    tok_scan_kernel<<<1, 1024, 0, stream>>>(doc_len, n_docs, offsets_out);
    if (n_docs > 0) tok_compact_kernel<<<(unsigned)n_docs, 64, 0, stream>>>(cur, doc_start, doc_len, offsets_out, n_docs, tokens_out);
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

}  // namespace
}  // namespace tasc

using namespace tasc;

extern "C" tasc_status tasc_tok_enrich(const int32_t* corpus_tokens, const int64_t* doc_offsets, int64_t n_docs,
                                       int32_t base_vocab, int32_t budget, int32_t n_max, int32_t* merges,
                                       int32_t* n_merges, int32_t* tokens_out, int64_t* offsets_out, tasc_stream stream_) {
    if (!doc_offsets || !merges || !n_merges || !offsets_out || n_docs < 0 || base_vocab < 1 || budget < 0 || n_max < 2 ||
        n_max > MAX_N || (int64_t)base_vocab + budget > (1 << TASC_VOCAB_BITS) || n_docs >= (1ll << 31))
        return TASC_EINVAL;
    *n_merges = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::vector<int64_t> offs((size_t)n_docs + 1);
    TASC_CUDA_TRY(cudaMemcpyAsync(offs.data(), doc_offsets, offs.size() * sizeof(int64_t), cudaMemcpyDeviceToHost, stream));
    TASC_CUDA_TRY(cudaStreamSynchronize(stream));
    if (offs[0] != 0) return TASC_EINVAL;
    uint64_t windows = 0;
    for (int64_t d = 0; d < n_docs; ++d) {
        const int64_t len = offs[d + 1] - offs[d];
        if (len < 0 || len >= (1ll << 31)) return TASC_EINVAL;
        for (int n = 2; n <= n_max; ++n) windows += (uint64_t)std::max<int64_t>(0, len - n + 1);
    }
    const int64_t T = offs[n_docs];
    if (T >= (1ll << POS_BITS)) return TASC_EINVAL;
    if (T > 0 && (!corpus_tokens || !tokens_out)) return TASC_EINVAL;

    int32_t* cur = nullptr;
    uint8_t* rem = nullptr;
    int64_t* doc_start = nullptr;
    int32_t* doc_len = nullptr;
    uint64_t* keys = nullptr;
    uint32_t *counts = nullptr, *first = nullptr;
    unsigned long long* best = nullptr;
    Winner* win = nullptr;
    int* dn = nullptr;                         // [0] number of merges, [1] status
    const uint64_t cap = pow2_at_least(2 * std::max<uint64_t>(windows, 1));
    tasc_status rc = TASC_OK;
#define TRY_ALLOC(ptr, bytes) if (rc == TASC_OK && cudaMalloc(reinterpret_cast<void**>(&(ptr)), (bytes)) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ENOMEM; }
    TRY_ALLOC(cur, (size_t)std::max<int64_t>(T, 1) * 4);
    TRY_ALLOC(rem, (size_t)std::max<int64_t>(T, 1));
    TRY_ALLOC(doc_start, (size_t)std::max<int64_t>(n_docs, 1) * 8);
    TRY_ALLOC(doc_len, (size_t)std::max<int64_t>(n_docs, 1) * 4);
    TRY_ALLOC(keys, cap * 16);
    TRY_ALLOC(counts, cap * 4);
    TRY_ALLOC(first, cap * 4);
    TRY_ALLOC(best, 8);
    TRY_ALLOC(win, sizeof(Winner));
    TRY_ALLOC(dn, 2 * sizeof(int));
#undef TRY_ALLOC
    int h_dn[2] = {0, 0};
    if (rc == TASC_OK) {
        cudaMemsetAsync(best, 0, 8, stream);
        cudaMemsetAsync(win, 0, sizeof(Winner), stream);
        cudaMemsetAsync(dn, 0, 2 * sizeof(int), stream);
        cudaMemsetAsync(merges, 0xFF, (size_t)budget * MAX_N * sizeof(int32_t), stream);
        if (T > 0) cudaMemcpyAsync(cur, corpus_tokens, (size_t)T * 4, cudaMemcpyDeviceToDevice, stream);
        if (n_docs > 0) tok_init_docs_kernel<<<blocks_for((uint64_t)n_docs, 128), 128, 0, stream>>>(doc_offsets, n_docs, doc_start, doc_len, rem);
        for (int it = 0; it < budget && T > 0; ++it) {
            cudaMemsetAsync(keys, 0, cap * 16, stream);
            cudaMemsetAsync(counts, 0, cap * 4, stream);
            cudaMemsetAsync(first, 0xFF, cap * 4, stream);
            for (int n = 2; n <= n_max; ++n)
                tok_count_kernel<<<blocks_for((uint64_t)T, 256), 256, 0, stream>>>(cur, rem, T, n, keys, counts, first, cap - 1, win, dn + 1);
            tok_best_kernel<<<blocks_for(cap, 256), 256, 0, stream>>>(keys, counts, first, cap, best, win);
            tok_winner_kernel<<<blocks_for(cap, 256), 256, 0, stream>>>(keys, counts, first, cap, best, win, merges, dn);
            tok_commit_kernel<<<1, 1, 0, stream>>>(win, dn, best);
            tok_rewrite_kernel<<<blocks_for((uint64_t)n_docs, 128), 128, 0, stream>>>(cur, rem, doc_start, doc_len, n_docs, win, dn, base_vocab);
        }
        if (cudaGetLastError() != cudaSuccess) rc = TASC_ECUDA;
        if (rc == TASC_OK) rc = compact_docs(cur, doc_start, doc_len, n_docs, tokens_out, offsets_out, stream);
        if (rc == TASC_OK && (cudaMemcpyAsync(h_dn, dn, sizeof(h_dn), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
                              cudaStreamSynchronize(stream) != cudaSuccess)) { (void)cudaGetLastError(); rc = TASC_ECUDA; }
        if (rc == TASC_OK && h_dn[1] != 0) rc = h_dn[1];
    }
    cudaFree(cur); cudaFree(rem); cudaFree(doc_start); cudaFree(doc_len); cudaFree(keys); cudaFree(counts); cudaFree(first);
    cudaFree(best); cudaFree(win); cudaFree(dn);
    if (rc == TASC_OK) *n_merges = h_dn[0];
    return rc;
}

extern "C" tasc_status tasc_tok_init_rows(const void* matrix, int32_t dtype, int32_t base_vocab, int32_t d,
                                          const int32_t* merges, int32_t n_merges, void* rows_out, int32_t* device_status,
                                          tasc_stream stream_) {
    if (!matrix || !merges || !rows_out || !device_status || base_vocab < 1 || d < 1 || n_merges < 0 ||
        (dtype != TASC_F32 && dtype != TASC_BF16))
        return TASC_EINVAL;
    if (n_merges == 0) return TASC_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const unsigned blocks = (unsigned)((d + 127) / 128);
    if (dtype == TASC_F32)
        tok_rows_kernel<float><<<blocks, 128, 0, stream>>>(static_cast<const float*>(matrix), base_vocab, d, merges, n_merges,
                                                           static_cast<float*>(rows_out), device_status);
    else
        tok_rows_kernel<__nv_bfloat16><<<blocks, 128, 0, stream>>>(static_cast<const __nv_bfloat16*>(matrix), base_vocab, d, merges,
                                                                   n_merges, static_cast<__nv_bfloat16*>(rows_out), device_status);
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}

extern "C" tasc_status tasc_tok_encode(const int32_t* tokens, const int64_t* doc_offsets, int64_t n_docs, int32_t base_vocab,
                                       const int32_t* merges, int32_t n_merges, int32_t* tokens_out, int64_t* offsets_out,
                                       tasc_stream stream_) {
    if (!doc_offsets || !offsets_out || n_docs < 0 || base_vocab < 1 || n_merges < 0 || (n_merges > 0 && !merges)) return TASC_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // the added tokens' expansions into base tokens, then the trie over them (host: a few thousand short sequences)
    std::vector<int32_t> hm((size_t)n_merges * MAX_N);
    int64_t T = 0;
    if (n_merges > 0) TASC_CUDA_TRY(cudaMemcpyAsync(hm.data(), merges, hm.size() * 4, cudaMemcpyDeviceToHost, stream));
    TASC_CUDA_TRY(cudaMemcpyAsync(&T, doc_offsets + n_docs, sizeof(int64_t), cudaMemcpyDeviceToHost, stream));
    TASC_CUDA_TRY(cudaStreamSynchronize(stream));
    if (T < 0 || (T > 0 && (!tokens || !tokens_out))) return TASC_EINVAL;
    constexpr size_t MAX_EXPANSION = 4096;
    std::vector<std::vector<int32_t>> exp((size_t)n_merges);
    for (int i = 0; i < n_merges; ++i) {
        for (int c = 0; c < MAX_N; ++c) {
            const int t = hm[(size_t)i * MAX_N + c];
            if (t < 0) break;
            if (t < base_vocab) exp[i].push_back(t);
            else if (t - base_vocab < i) exp[i].insert(exp[i].end(), exp[t - base_vocab].begin(), exp[t - base_vocab].end());
            else return TASC_EINVAL;
            if (exp[i].size() > MAX_EXPANSION) return TASC_ECAPACITY;
        }
        if (exp[i].size() < 2) return TASC_EINVAL;
    }
    std::map<std::pair<int, int>, int> edges;          // (node, token) -> child
    std::vector<int32_t> node_token(1, -1);
    for (int i = 0; i < n_merges; ++i) {
        int node = 0;
        for (int32_t t : exp[i]) {
            auto it = edges.find({node, t});
            if (it == edges.end()) {
                it = edges.emplace(std::make_pair(node, (int)t), (int)node_token.size()).first;
                node_token.push_back(-1);
            }
            node = it->second;
        }
        if (node_token[node] < 0) node_token[node] = base_vocab + i;     // two added tokens with one expansion: the earlier one
    }
    const uint64_t cap = pow2_at_least(2 * std::max<uint64_t>(edges.size(), 1));
    std::vector<uint64_t> hk(cap, 0ull);
    std::vector<int32_t> hc(cap, -1);
    auto mix = [](uint64_t k) { k ^= k >> 33; k *= 0xFF51AFD7ED558CCDull; k ^= k >> 33; k *= 0xC4CEB9FE1A85EC53ull; k ^= k >> 33; return k; };
    for (const auto& e : edges) {
        const uint64_t key = ((uint64_t)(uint32_t)e.first.first << 32) | (uint64_t)(uint32_t)e.first.second | (1ull << 63);
        uint64_t slot = mix(key) & (cap - 1);
        while (hk[slot] != 0ull) slot = (slot + 1) & (cap - 1);
        hk[slot] = key;
        hc[slot] = e.second;
    }
    uint64_t* d_keys = nullptr;
    int32_t *d_child = nullptr, *d_tok = nullptr, *scratch = nullptr, *doc_len = nullptr;
    int64_t* doc_start = nullptr;
    tasc_status rc = TASC_OK;
#define TRY_ALLOC(ptr, bytes) if (rc == TASC_OK && cudaMalloc(reinterpret_cast<void**>(&(ptr)), (bytes)) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ENOMEM; }
    TRY_ALLOC(d_keys, cap * 8);
    TRY_ALLOC(d_child, cap * 4);
    TRY_ALLOC(d_tok, node_token.size() * 4);
    TRY_ALLOC(scratch, (size_t)std::max<int64_t>(T, 1) * 4);
    TRY_ALLOC(doc_len, (size_t)std::max<int64_t>(n_docs, 1) * 4);
    TRY_ALLOC(doc_start, (size_t)std::max<int64_t>(n_docs, 1) * 8);
#undef TRY_ALLOC
    if (rc == TASC_OK) {
        cudaMemcpyAsync(d_keys, hk.data(), cap * 8, cudaMemcpyHostToDevice, stream);
        cudaMemcpyAsync(d_child, hc.data(), cap * 4, cudaMemcpyHostToDevice, stream);
        cudaMemcpyAsync(d_tok, node_token.data(), node_token.size() * 4, cudaMemcpyHostToDevice, stream);
        TrieTable trie = {d_keys, d_child, d_tok, cap - 1};
        if (n_docs > 0)
            tok_encode_kernel<<<blocks_for((uint64_t)n_docs, 128), 128, 0, stream>>>(tokens, doc_offsets, n_docs, trie, scratch, doc_start, doc_len);
        if (cudaGetLastError() != cudaSuccess) rc = TASC_ECUDA;
        if (rc == TASC_OK) rc = compact_docs(scratch, doc_start, doc_len, n_docs, tokens_out, offsets_out, stream);
        if (cudaStreamSynchronize(stream) != cudaSuccess) { (void)cudaGetLastError(); rc = TASC_ECUDA; }   // the host tables must outlive the copies
    }
    cudaFree(d_keys); cudaFree(d_child); cudaFree(d_tok); cudaFree(scratch); cudaFree(doc_len); cudaFree(doc_start);
    return rc;
}
