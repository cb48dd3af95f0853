// Packed n-gram keys and the open-addressing table they live in: shared by the drafter's corpus tables, the corpus
// statistics and the tokenizer enrichment.  A key is the full 128-bit packing of (order, up to six 20-bit token ids),
// claimed or found with one 128-bit compare-and-swap, so matches are exact (no fingerprints).
#pragma once

#include "common.cuh"

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

inline uint64_t pow2_at_least(uint64_t v) {
    uint64_t p = 64;
    while (p < v) p <<= 1;
    return p;
}

inline unsigned blocks_for(uint64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace
}  // namespace tasc
