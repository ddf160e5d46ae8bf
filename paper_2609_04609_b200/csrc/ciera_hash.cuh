// Hash128 of a block of exponents: the per-block fingerprint that the sender of Algorithm 1 keeps in
// HashCache.  Section 3.1 asks for 128 bits made of two 64-bit SplitMix64-based hashes that do not
// depend on each other.
//
// The paper fixes no more than that.  The construction used here:
//   mix(z)  = the SplitMix64 output function;
//   a block of L exponent bytes is read as ceil(L / 8) little-endian 64-bit words x_j (the last
//   one zero-padded);  H_i = mix(L + sum_j mix(s_i + (j + 1) * g_i + x_j))  (mod 2^64);
//   Hash128 = (H_1, H_2) with s_1 = 0, g_1 = 0x9E3779B97F4A7C15 (the SplitMix64 increment) and
//   s_2 = 0x6A09E667F3BCC908, g_2 = 0xD1342543DE82EF95 (a second odd increment: on a common increment
//   the two halves would share every collision made by moving a word and shifting it by the distance
//   times the increment).
// The per-word terms are summed, so the threads holding a block's words can be combined in any
// order.
#pragma once

#include "ciera_internal.cuh"

namespace ciera {

constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kGamma2 = 0xD1342543DE82EF95ull;
constexpr uint64_t kSeed1 = 0x0000000000000000ull;
constexpr uint64_t kSeed2 = 0x6A09E667F3BCC908ull;

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

// the two terms of word x, the j-th word of its block
__device__ __forceinline__ void hash_word_terms(uint32_t j, uint64_t x, uint64_t& a, uint64_t& b) {
    a = mix64(kSeed1 + (uint64_t)(j + 1u) * kGamma + x);
    b = mix64(kSeed2 + (uint64_t)(j + 1u) * kGamma2 + x);
}

// the block's two hashes from the sums of its words' terms
__device__ __forceinline__ ulonglong2 hash_finish(uint64_t sum_a, uint64_t sum_b, uint32_t L) {
    return make_ulonglong2((unsigned long long)mix64(sum_a + L), (unsigned long long)mix64(sum_b + L));
}

}  // namespace ciera
