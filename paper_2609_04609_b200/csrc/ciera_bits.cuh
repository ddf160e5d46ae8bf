// Per-thread register work on "pieces": runs of consecutive values owned by one thread.
//
// Split and merge follow the paper's Section 3.1 (a value is sign, exponent and mantissa bits;
// the exponent travels apart from sign-plus-mantissa) on the IEEE binary32 / bfloat16 layouts:
//   bf16: bit 15 sign, bits 14:7 exponent, bits 6:0 mantissa  -> sm byte  = sign<<7  | mantissa
//   fp32: bit 31 sign, bits 30:23 exponent, bits 22:0 mantissa -> sm 24bit = sign<<23 | mantissa
// Everything is done on packed 32-bit words with shifts, three-input logic and byte permutes,
// four values at a time.
//
// Thread -> value layout inside a tile of 8192 values (512 consumer threads):
//   bf16: two pieces of 8 values per thread, piece p of thread t = values [4096 p + 8 t, +8).
//         Every access of a warp is then one contiguous run: 16 B / lane on the weights,
//         8 B / lane on the byte-wide streams (exponents, sign-plus-mantissa).
//   fp32: one piece of 16 values per thread, values [16 t, +16): 64 B of weights, 16 B of
//         exponents, 48 B of sign-plus-mantissa per lane.
// With blocks of 16 values and more a piece never straddles a block, so a piece has one "my
// exponents changed" bit; the tile has 1024 (bf16) or 512 (fp32) such bits.  With smaller blocks
// a piece holds 1 to 16 whole blocks and has one bit for each.
#pragma once

#include "ciera_internal.cuh"

namespace ciera {

// ---- 8- and 16-byte accesses ---------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream16(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ uint2 ld_stream8(const void* p) { return __ldcs(reinterpret_cast<const uint2*>(p)); }
__device__ __forceinline__ void st_stream16(void* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }
__device__ __forceinline__ void st_stream8(void* p, uint2 v) { __stcs(reinterpret_cast<uint2*>(p), v); }
__device__ __forceinline__ uint4 ld_shared16(const void* p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"((uint32_t)__cvta_generic_to_shared(p)));
    return v;
}
__device__ __forceinline__ uint2 ld_shared8(const void* p) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"((uint32_t)__cvta_generic_to_shared(p)));
    return v;
}
__device__ __forceinline__ void st_shared16(void* p, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v.x),
                 "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ void st_shared8(void* p, uint2 v) {
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v.x), "r"(v.y)
                 : "memory");
}
// memory spaces a piece is read from / written to
struct Global {
    static __device__ __forceinline__ uint4 ld16(const uint8_t* p) { return ld_stream16(p); }
    static __device__ __forceinline__ uint2 ld8(const uint8_t* p) { return ld_stream8(p); }
    static __device__ __forceinline__ void st16(uint8_t* p, uint4 v) { st_stream16(p, v); }
    static __device__ __forceinline__ void st8(uint8_t* p, uint2 v) { st_stream8(p, v); }
    static __device__ __forceinline__ uint32_t ld1(const uint8_t* p) { return __ldcs(p); }
    static __device__ __forceinline__ uint32_t ld2(const uint8_t* p) { return __ldcs(reinterpret_cast<const uint16_t*>(p)); }
    static __device__ __forceinline__ uint32_t ld4(const uint8_t* p) { return __ldcs(reinterpret_cast<const uint32_t*>(p)); }
};
struct Shared {
    static __device__ __forceinline__ uint4 ld16(const uint8_t* p) { return ld_shared16(p); }
    static __device__ __forceinline__ uint2 ld8(const uint8_t* p) { return ld_shared8(p); }
    static __device__ __forceinline__ void st16(uint8_t* p, uint4 v) { st_shared16(p, v); }
    static __device__ __forceinline__ void st8(uint8_t* p, uint2 v) { st_shared8(p, v); }
    static __device__ __forceinline__ uint32_t ld1(const uint8_t* p) {
        uint32_t v;
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)));
        return v;
    }
    static __device__ __forceinline__ uint32_t ld2(const uint8_t* p) {
        uint32_t v;
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)));
        return v;
    }
    static __device__ __forceinline__ uint32_t ld4(const uint8_t* p) {
        uint32_t v;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)));
        return v;
    }
};

// (x & mask) | (y & ~mask): one three-input logic operation
__device__ __forceinline__ uint32_t bitselect(uint32_t mask, uint32_t x, uint32_t y) { return (x & mask) | (y & ~mask); }

// ---- bf16 --------------------------------------------------------------------------------
// Four values a = v0 | v1 << 16, b = v2 | v3 << 16.  Gather their low bytes (e0 m6..m0) and high
// bytes (s e7..e1) with two byte permutes; then
//   sm byte  = (high & 0x80) | (low & 0x7F)            exponent byte = (high << 1) | (low >> 7)
// for all four at once (the shifts leak across byte lanes only into bits that are masked off).
__device__ __forceinline__ void bf16_split4(uint32_t a, uint32_t b, uint32_t& e, uint32_t& sm) {
    const uint32_t lo = __byte_perm(a, b, 0x6420), hi = __byte_perm(a, b, 0x7531);
    sm = bitselect(0x7F7F7F7Fu, lo, hi);
    e = bitselect(0xFEFEFEFEu, hi << 1, lo >> 7);
}
// four exponent bytes + four sm bytes -> two words of two bf16 each
__device__ __forceinline__ void bf16_merge4(uint32_t e, uint32_t s, uint32_t& a, uint32_t& b) {
    const uint32_t lo = bitselect(0x7F7F7F7Fu, s, e << 7);  // e0 m6..m0
    const uint32_t hi = bitselect(0x80808080u, s, e >> 1);  // s e7..e1
    a = __byte_perm(lo, hi, 0x5140);
    b = __byte_perm(lo, hi, 0x7362);
}

// ---- fp32 --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t fp32_exp4(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
    uint32_t t01 = __byte_perm(w0 << 1, w1 << 1, 0x0073);  // byte0 = exp(w0), byte1 = exp(w1)
    uint32_t t23 = __byte_perm(w2 << 1, w3 << 1, 0x0073);
    return __byte_perm(t01, t23, 0x5410);
}
// sign << 23 | mantissa in bits 23:0 (bits 31:24 are don't-care for the packing below)
__device__ __forceinline__ uint32_t fp32_sm(uint32_t w) { return bitselect(0x007FFFFFu, w, w >> 8); }
// four 24-bit sm values -> three little-endian words
__device__ __forceinline__ void fp32_pack4(uint32_t s0, uint32_t s1, uint32_t s2, uint32_t s3, uint32_t& o0,
                                           uint32_t& o1, uint32_t& o2) {
    o0 = __byte_perm(s0, s1, 0x4210);
    o1 = __byte_perm(s1, s2, 0x5421);
    o2 = __byte_perm(s2, s3, 0x6542);
}
// three words -> four sm values in bits 23:0 (bits 31:24 don't-care)
__device__ __forceinline__ void fp32_unpack4(uint32_t o0, uint32_t o1, uint32_t o2, uint32_t& s0, uint32_t& s1,
                                             uint32_t& s2, uint32_t& s3) {
    s0 = o0;
    s1 = __byte_perm(o0, o1, 0x0543);
    s2 = __byte_perm(o1, o2, 0x0432);
    s3 = o2 >> 8;
}
// exponent in bits 7:0 of e (higher bits don't-care), sm in bits 23:0 of s
__device__ __forceinline__ uint32_t fp32_merge(uint32_t e, uint32_t s) {
    return bitselect(0x007FFFFFu, s, bitselect(0x7F800000u, e << 23, s << 8));
}

// ---- byte-granular access to a short run of exponent / sm bytes held in words ---------------
template <int NB>
__device__ __forceinline__ void load_bytes_partial(uint32_t* w, const uint8_t* src, int nbytes) {
#pragma unroll
    for (int i = 0; i < NB / 4; ++i) w[i] = 0;
#pragma unroll
    for (int i = 0; i < NB; ++i)
        if (i < nbytes) w[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
}
template <int NB>
__device__ __forceinline__ void store_bytes_partial(uint8_t* dst, const uint32_t* w, int nbytes) {
#pragma unroll
    for (int i = 0; i < NB; ++i)
        if (i < nbytes) dst[i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
}


// ---- flags of fine blocks ------------------------------------------------------------------
// bit 7 of every byte of the result tells whether that byte of d is non-zero
__device__ __forceinline__ uint32_t nonzero_bytes(uint32_t d) {
    return (((d & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | d) & 0x80808080u;
}
// d0, d1 = new exponents ^ cached exponents of eight consecutive values (one byte each): one flag
// per value, value 0 in bit 0.  The non-zero marks of d0 go to bits 0, 8, 16, 24 and those of d1 to
// bits 4, 12, 20, 28; one multiply then gathers bit 8i into bit 24 + i and bit 8i + 4 into bit
// 28 + i (all partial products land on distinct bits below 32, so nothing carries).
__device__ __forceinline__ uint32_t value_flags8(uint32_t d0, uint32_t d1) {
    const uint32_t t = (nonzero_bytes(d0) >> 7) | (nonzero_bytes(d1) >> 3);
    return (t * 0x01020408u) >> 24;
}
// d = the same for four values: one flag per block of 2^log2b values (log2b = 1, 2: two, one flag)
__device__ __forceinline__ uint32_t word_block_flags(uint32_t d, uint32_t log2b) {
    if (log2b == 1) return ((d & 0xFFFFu) != 0u ? 1u : 0u) | ((d >> 16) != 0u ? 2u : 0u);
    return d != 0u ? 1u : 0u;
}

// ---- pieces --------------------------------------------------------------------------------
template <int DT>
struct Piece;

// bf16: 8 values = 16 B of weights, 8 exponent bytes, 8 sm bytes
template <>
struct Piece<CIERA_BF16> {
    static constexpr int kValues = 8;
    static constexpr int kLog2Values = 3;
    static constexpr int kPerThread = 2;  // pieces per thread
    static constexpr int kExpWords = 2;
    static constexpr int kSmWords = 2;
    // first value (inside the tile) of piece p of consumer thread tid
    static __device__ __forceinline__ uint32_t start(uint32_t tid, int p) {
        return (uint32_t)p * (kTileValues / 2) + tid * 8u;
    }

    uint32_t e[kExpWords];
    uint32_t s[kSmWords];

    template <class M>
    __device__ __forceinline__ void split_full(const uint8_t* w) {
        const uint4 a = M::ld16(w);
        bf16_split4(a.x, a.y, e[0], s[0]);
        bf16_split4(a.z, a.w, e[1], s[1]);
    }
    // the first nvalid (< 8) values; the others read as +0.0 (exponent 0)
    __device__ __forceinline__ void split_partial(const uint8_t* w, int nvalid) {
        uint32_t x[4] = {0, 0, 0, 0};
        const uint16_t* p = reinterpret_cast<const uint16_t*>(w);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvalid) x[i >> 1] |= (uint32_t)p[i] << (16 * (i & 1));
        bf16_split4(x[0], x[1], e[0], s[0]);
        bf16_split4(x[2], x[3], e[1], s[1]);
    }
    template <class M>
    __device__ __forceinline__ void load_exp_full(const uint8_t* src) {
        const uint2 v = M::ld8(src);
        e[0] = v.x; e[1] = v.y;
    }
    template <class M>
    __device__ __forceinline__ void store_exp_full(uint8_t* dst) const { M::st8(dst, make_uint2(e[0], e[1])); }
    __device__ __forceinline__ void load_exp_partial(const uint8_t* src, int nvalid) { load_bytes_partial<8>(e, src, nvalid); }
    __device__ __forceinline__ void store_exp_partial(uint8_t* dst, int nvalid) const { store_bytes_partial<8>(dst, e, nvalid); }
    template <class M>
    __device__ __forceinline__ void load_sm_full(const uint8_t* src) {
        const uint2 v = M::ld8(src);
        s[0] = v.x; s[1] = v.y;
    }
    template <class M>
    __device__ __forceinline__ void store_sm_full(uint8_t* dst) const { M::st8(dst, make_uint2(s[0], s[1])); }
    __device__ __forceinline__ void load_sm_partial(const uint8_t* src, int nvalid) { load_bytes_partial<8>(s, src, nvalid); }
    __device__ __forceinline__ void store_sm_partial(uint8_t* dst, int nvalid) const { store_bytes_partial<8>(dst, s, nvalid); }
    template <class M>
    __device__ __forceinline__ void merge_store_full(uint8_t* w) const {
        uint4 a;
        bf16_merge4(e[0], s[0], a.x, a.y);
        bf16_merge4(e[1], s[1], a.z, a.w);
        M::st16(w, a);
    }
    __device__ __forceinline__ void merge_store_partial(uint8_t* w, int nvalid) const {
        uint32_t x[4];
        bf16_merge4(e[0], s[0], x[0], x[1]);
        bf16_merge4(e[1], s[1], x[2], x[3]);
        uint16_t* p = reinterpret_cast<uint16_t*>(w);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvalid) p[i] = (uint16_t)(x[i >> 1] >> (16 * (i & 1)));
    }
    __device__ __forceinline__ bool differs(const Piece& o) const { return ((e[0] ^ o.e[0]) | (e[1] ^ o.e[1])) != 0; }
    // one flag per block of 2^log2b values (log2b <= 3), lowest block first
    __device__ __forceinline__ uint32_t block_flags(const Piece& o, uint32_t log2b) const {
        if (log2b >= 3) return differs(o) ? 1u : 0u;
        if (log2b == 0) return value_flags8(e[0] ^ o.e[0], e[1] ^ o.e[1]);
        const uint32_t per_word = 4u >> log2b;
        return word_block_flags(e[0] ^ o.e[0], log2b) | (word_block_flags(e[1] ^ o.e[1], log2b) << per_word);
    }
};

// fp32: 16 values = 64 B of weights, 16 exponent bytes, 48 sm bytes
template <>
struct Piece<CIERA_FP32> {
    static constexpr int kValues = 16;
    static constexpr int kLog2Values = 4;
    static constexpr int kPerThread = 1;
    static constexpr int kExpWords = 4;
    static constexpr int kSmWords = 12;
    static __device__ __forceinline__ uint32_t start(uint32_t tid, int) { return tid * 16u; }

    uint32_t e[kExpWords];
    uint32_t s[kSmWords];

    __device__ __forceinline__ void from_words(const uint32_t* x) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[i] = fp32_exp4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
            fp32_pack4(fp32_sm(x[4 * i]), fp32_sm(x[4 * i + 1]), fp32_sm(x[4 * i + 2]), fp32_sm(x[4 * i + 3]),
                       s[3 * i], s[3 * i + 1], s[3 * i + 2]);
        }
    }
    template <class M>
    __device__ __forceinline__ void split_full(const uint8_t* w) {
        uint32_t x[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 v = M::ld16(w + 16 * i);
            x[4 * i] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
        }
        from_words(x);
    }
    __device__ __forceinline__ void split_partial(const uint8_t* w, int nvalid) {
        uint32_t x[16];
        const uint32_t* p = reinterpret_cast<const uint32_t*>(w);
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = i < nvalid ? p[i] : 0u;
        from_words(x);
    }
    template <class M>
    __device__ __forceinline__ void load_exp_full(const uint8_t* src) {
        const uint4 v = M::ld16(src);
        e[0] = v.x; e[1] = v.y; e[2] = v.z; e[3] = v.w;
    }
    template <class M>
    __device__ __forceinline__ void store_exp_full(uint8_t* dst) const { M::st16(dst, make_uint4(e[0], e[1], e[2], e[3])); }
    __device__ __forceinline__ void load_exp_partial(const uint8_t* src, int nvalid) { load_bytes_partial<16>(e, src, nvalid); }
    __device__ __forceinline__ void store_exp_partial(uint8_t* dst, int nvalid) const { store_bytes_partial<16>(dst, e, nvalid); }
    template <class M>
    __device__ __forceinline__ void load_sm_full(const uint8_t* src) {
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint4 v = M::ld16(src + 16 * i);
            s[4 * i] = v.x; s[4 * i + 1] = v.y; s[4 * i + 2] = v.z; s[4 * i + 3] = v.w;
        }
    }
    template <class M>
    __device__ __forceinline__ void store_sm_full(uint8_t* dst) const {
#pragma unroll
        for (int i = 0; i < 3; ++i) M::st16(dst + 16 * i, make_uint4(s[4 * i], s[4 * i + 1], s[4 * i + 2], s[4 * i + 3]));
    }
    __device__ __forceinline__ void load_sm_partial(const uint8_t* src, int nvalid) { load_bytes_partial<48>(s, src, 3 * nvalid); }
    __device__ __forceinline__ void store_sm_partial(uint8_t* dst, int nvalid) const { store_bytes_partial<48>(dst, s, 3 * nvalid); }
    __device__ __forceinline__ void merge_words(uint32_t* x) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t s0, s1, s2, s3;
            fp32_unpack4(s[3 * i], s[3 * i + 1], s[3 * i + 2], s0, s1, s2, s3);
            x[4 * i] = fp32_merge(e[i], s0);
            x[4 * i + 1] = fp32_merge(e[i] >> 8, s1);
            x[4 * i + 2] = fp32_merge(e[i] >> 16, s2);
            x[4 * i + 3] = fp32_merge(e[i] >> 24, s3);
        }
    }
    template <class M>
    __device__ __forceinline__ void merge_store_full(uint8_t* w) const {
        uint32_t x[16];
        merge_words(x);
#pragma unroll
        for (int i = 0; i < 4; ++i) M::st16(w + 16 * i, make_uint4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]));
    }
    __device__ __forceinline__ void merge_store_partial(uint8_t* w, int nvalid) const {
        uint32_t x[16];
        merge_words(x);
        uint32_t* p = reinterpret_cast<uint32_t*>(w);
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nvalid) p[i] = x[i];
    }
    __device__ __forceinline__ bool differs(const Piece& o) const {
        return ((e[0] ^ o.e[0]) | (e[1] ^ o.e[1]) | (e[2] ^ o.e[2]) | (e[3] ^ o.e[3])) != 0;
    }
    // one flag per block of 2^log2b values (log2b <= 3), lowest block first
    __device__ __forceinline__ uint32_t block_flags(const Piece& o, uint32_t log2b) const {
        if (log2b >= 3)
            return (((e[0] ^ o.e[0]) | (e[1] ^ o.e[1])) != 0 ? 1u : 0u) | (((e[2] ^ o.e[2]) | (e[3] ^ o.e[3])) != 0 ? 2u : 0u);
        if (log2b == 0)
            return value_flags8(e[0] ^ o.e[0], e[1] ^ o.e[1]) | (value_flags8(e[2] ^ o.e[2], e[3] ^ o.e[3]) << 8);
        const uint32_t per_word = 4u >> log2b;
        uint32_t f = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) f |= word_block_flags(e[i] ^ o.e[i], log2b) << (per_word * i);
        return f;
    }
};

// fp16: 8 values = 16 B of weights, 8 exponent bytes in the caches, and on the wire 11 bytes of
// sign-plus-mantissa (8 x 11 bits, value j at bits [11 j, 11 j + 11)) and 5 bytes of exponents
// (8 x 5 bits).  Thread -> value layout as for bf16.
template <>
struct Piece<CIERA_FP16> {
    static constexpr int kValues = 8;
    static constexpr int kLog2Values = 3;
    static constexpr int kPerThread = 2;
    static constexpr int kExpWords = 2;
    static __device__ __forceinline__ uint32_t start(uint32_t tid, int p) {
        return (uint32_t)p * (kTileValues / 2) + tid * 8u;
    }

    uint32_t e[2];  // 8 exponents, one byte each (0..31)
    uint32_t s[3];  // 88 bits of sign-plus-mantissa

    // w = eight fp16 values, two per word
    __device__ __forceinline__ void split_words(const uint32_t w[4]) {
        // p[i] = the two values' 11-bit fields side by side (22 bits): mantissa bits 9:0 stay, the sign
        // (bit 15) moves to bit 10, the second value's mantissa (bits 25:16) to 20:11, its sign (bit 31) to 21
        uint32_t e2[4], p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t t5 = w[i] >> 5, t10 = w[i] >> 10;
            e2[i] = t10 & 0x001F001Fu;
            p[i] = (w[i] & 0x000003FFu) | (t5 & 0x001FFC00u) | (t10 & 0x00200000u);
        }
        e[0] = __byte_perm(e2[0], e2[1], 0x6420);
        e[1] = __byte_perm(e2[2], e2[3], 0x6420);
        s[0] = p[0] | (p[1] << 22);
        s[1] = (p[1] >> 10) | (p[2] << 12);
        s[2] = (p[2] >> 20) | (p[3] << 2);
    }
    __device__ __forceinline__ void merge_words(uint32_t w[4]) const {
        uint32_t f[8];
        f[0] = s[0] & 0x7FFu;
        f[1] = (s[0] >> 11) & 0x7FFu;
        f[2] = ((s[0] >> 22) | (s[1] << 10)) & 0x7FFu;
        f[3] = (s[1] >> 1) & 0x7FFu;
        f[4] = (s[1] >> 12) & 0x7FFu;
        f[5] = ((s[1] >> 23) | (s[2] << 9)) & 0x7FFu;
        f[6] = (s[2] >> 2) & 0x7FFu;
        f[7] = (s[2] >> 13) & 0x7FFu;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t ex = (e[i >> 2] >> (8 * (i & 3))) & 0x1Fu;
            const uint32_t v = (f[i] & 0x3FFu) | ((f[i] & 0x400u) << 5) | (ex << 10);
            if (i & 1)
                w[i >> 1] |= v << 16;
            else
                w[i >> 1] = v;
        }
    }
    template <class M>
    __device__ __forceinline__ void split_full(const uint8_t* src) {
        const uint4 v = M::ld16(src);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        split_words(w);
    }
    // the first nvalid (< 8) values; the others read as +0.0
    __device__ __forceinline__ void split_partial(const uint8_t* src, int nvalid) {
        const uint16_t* p = reinterpret_cast<const uint16_t*>(src);
        uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvalid) w[i >> 1] |= (uint32_t)p[i] << (16 * (i & 1));
        split_words(w);
    }
    template <class M>
    __device__ __forceinline__ void merge_store_full(uint8_t* dst) const {
        uint32_t w[4];
        merge_words(w);
        M::st16(dst, make_uint4(w[0], w[1], w[2], w[3]));
    }
    __device__ __forceinline__ void merge_store_partial(uint8_t* dst, int nvalid) const {
        uint32_t w[4];
        merge_words(w);
        uint16_t* d16 = reinterpret_cast<uint16_t*>(dst);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvalid) d16[i] = (uint16_t)(w[i >> 1] >> (16 * (i & 1)));
    }
    template <class M>
    __device__ __forceinline__ void load_exp_full(const uint8_t* src) {
        const uint2 v = M::ld8(src);
        e[0] = v.x; e[1] = v.y;
    }
    template <class M>
    __device__ __forceinline__ void store_exp_full(uint8_t* dst) const { M::st8(dst, make_uint2(e[0], e[1])); }
    __device__ __forceinline__ void load_exp_partial(const uint8_t* src, int nvalid) { load_bytes_partial<8>(e, src, nvalid); }
    __device__ __forceinline__ void store_exp_partial(uint8_t* dst, int nvalid) const { store_bytes_partial<8>(dst, e, nvalid); }
    __device__ __forceinline__ bool differs(const Piece& o) const { return ((e[0] ^ o.e[0]) | (e[1] ^ o.e[1])) != 0; }
    // one flag per block of 2^log2b values (log2b <= 3), lowest block first (the exponents lie one byte each, as for bf16)
    __device__ __forceinline__ uint32_t block_flags(const Piece& o, uint32_t log2b) const {
        if (log2b >= 3) return differs(o) ? 1u : 0u;
        if (log2b == 0) return value_flags8(e[0] ^ o.e[0], e[1] ^ o.e[1]);
        const uint32_t per_word = 4u >> log2b;
        return word_block_flags(e[0] ^ o.e[0], log2b) | (word_block_flags(e[1] ^ o.e[1], log2b) << per_word);
    }

    // the 8 exponents as 40 bits: low word and high byte
    __device__ __forceinline__ void pack_exponents(uint32_t& lo, uint32_t& hi) const {
        uint32_t x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = (e[i >> 2] >> (8 * (i & 3))) & 0x1Fu;
        lo = x[0] | (x[1] << 5) | (x[2] << 10) | (x[3] << 15) | (x[4] << 20) | (x[5] << 25) | (x[6] << 30);
        hi = (x[6] >> 2) | (x[7] << 3);
    }
    __device__ __forceinline__ void unpack_exponents(uint32_t lo, uint32_t hi) {
        uint32_t x[8];
#pragma unroll
        for (int i = 0; i < 6; ++i) x[i] = (lo >> (5 * i)) & 0x1Fu;
        x[6] = ((lo >> 30) | (hi << 2)) & 0x1Fu;
        x[7] = (hi >> 3) & 0x1Fu;
        e[0] = x[0] | (x[1] << 8) | (x[2] << 16) | (x[3] << 24);
        e[1] = x[4] | (x[5] << 8) | (x[6] << 16) | (x[7] << 24);
    }
    // the packed exponents of the piece from `src` (5 bytes, any alignment; nvalid < 8: fewer)
    template <class M>
    __device__ __forceinline__ void load_packed_exponents(const uint8_t* src, int nvalid) {
        const int nbytes = (5 * nvalid + 7) >> 3;
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int i = 0; i < 5; ++i) {
            if (i < nbytes) {
                const uint32_t b = M::ld1(src + i);
                if (i < 4)
                    lo |= b << (8 * i);
                else
                    hi = b;
            }
        }
        unpack_exponents(lo, hi);
    }

    // Packed sign-plus-mantissa of a piece in a section whose pieces are all complete: the four lanes
    // 4k..4k+3 share 44 bytes = 11 aligned words, lane a holds bits [88a, 88a+88) of them.
    // `section` = start of the tile's part of the section, `piece` = index of the piece in the tile.
    template <class M>
    __device__ __forceinline__ void load_sm_group(const uint8_t* section, uint32_t piece, uint32_t lane) {
        const uint32_t a = lane & 3u;
        // lane a's bits start at word {0, 2, 5, 8}, bit {0, 24, 16, 8} of the group
        const uint32_t first = (11u * a) >> 2, sh = (88u * a) & 31u;
        const uint8_t* src = section + (size_t)11 * (piece - a) + 4u * first;
        const uint32_t w0 = M::ld4(src), w1 = M::ld4(src + 4), w2 = M::ld4(src + 8);
        const uint32_t w3 = (a == 0u || a == 3u) ? 0u : M::ld4(src + 12);  // lanes 0 and 3 end inside their third word
        s[0] = sh ? (w0 >> sh) | (w1 << (32u - sh)) : w0;
        s[1] = sh ? (w1 >> sh) | (w2 << (32u - sh)) : w1;
        s[2] = (sh ? (w2 >> sh) | (w3 << (32u - sh)) : w2) & 0x00FFFFFFu;
    }
    // lane a writes words 3a, 3a+1, 3a+2 of the group (lane 3: two words), taking the low bits of the
    // next lane's first word where its own bits end inside a word.  All 32 lanes call this.
    __device__ __forceinline__ void store_sm_group(uint8_t* section, uint32_t piece, uint32_t lane) const {
        const uint32_t a = lane & 3u, sh = 8u * a;
        const uint32_t next0 = __shfl_down_sync(0xffffffffu, s[0], 1);
        uint32_t* dst = reinterpret_cast<uint32_t*>(section + (size_t)11 * (piece - a)) + 3u * a;
        dst[0] = sh ? (s[0] >> sh) | (s[1] << (32u - sh)) : s[0];
        dst[1] = sh ? (s[1] >> sh) | (s[2] << (32u - sh)) : s[1];
        if (a != 3u) dst[2] = (s[2] >> sh) | (next0 << (24u - sh));
    }
    // byte by byte (pieces of a tile with a ragged end)
    __device__ __forceinline__ void load_sm_bytes(const uint8_t* src, int nvalid) {
        s[0] = s[1] = s[2] = 0;
        const int nbytes = (11 * nvalid + 7) >> 3;
        for (int i = 0; i < nbytes; ++i) s[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
    }
    __device__ __forceinline__ void store_sm_bytes(uint8_t* dst, int nvalid) const {
        const int nbytes = (11 * nvalid + 7) >> 3;
        for (int i = 0; i < nbytes; ++i) dst[i] = (uint8_t)(s[i >> 2] >> (8 * (i & 3)));
    }
};

// number of valid values of the piece starting at value `start` in a tile of nv values
template <int DT>
__device__ __forceinline__ int piece_valid(uint32_t start, uint32_t nv) {
    return start >= nv ? 0 : (int)min((uint32_t)Piece<DT>::kValues, nv - start);
}

// Block flags of a tile from the vote bits "my piece differs" (one warp).  `pl2` = log2 of the
// values per piece.  Fills bm (one bit per block of the tile) and pre (set bits before each word);
// returns the number of changed blocks of the tile.
__device__ __forceinline__ uint32_t build_block_bitmap(const uint32_t* ballot, uint32_t* bm, uint16_t* pre,
                                                       uint32_t log2b, uint32_t pl2, uint32_t lane) {
    const uint32_t gl2 = log2b - pl2;           // log2(pieces per block)
    const uint32_t nbt = kTileValues >> log2b;  // blocks of a full tile
    if (nbt > 32 && gl2 >= 1) {
        // More than one word of block flags (2 to 16 pieces per block): lane l turns vote word l into
        // its 32 >> gl2 block flags -- fold the votes of a block onto its first bit, gather those bits --
        // the 2^gl2 lanes whose flags share a word of bm combine them, and one scan does for the tile.
        const uint32_t vote_words = (uint32_t)kTileValues >> (pl2 + 5);  // 32 or 16
        uint32_t t = lane < vote_words ? ballot[lane] : 0u;
        for (uint32_t k = 0; k < gl2; ++k) t |= t >> (1u << k);
        const uint32_t cnt = 32u >> gl2;
        uint32_t fl = 0;
        for (uint32_t j = 0; j < cnt; ++j) fl |= ((t >> (j << gl2)) & 1u) << j;
        uint32_t v = fl << ((lane * cnt) & 31u);
        for (uint32_t k = 0; k < gl2; ++k) v |= __shfl_xor_sync(0xffffffffu, v, 1u << k);
        const uint32_t nwords = nbt >> 5;  // 2 .. 16
        uint32_t word = __shfl_sync(0xffffffffu, v, (lane << gl2) & 31u);
        if (lane >= nwords) word = 0u;
        const uint32_t pc = __popc(word);
        uint32_t incl = pc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += u;
        }
        if (lane < nwords) {
            bm[lane] = word;
            pre[lane] = (uint16_t)(incl - pc);
        }
        const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
        __syncwarp();
        return total;
    }
    uint32_t run = 0;
    for (uint32_t base = 0; base < nbt; base += 32) {
        const uint32_t i = base + lane;
        bool f = false;
        if (i < nbt) {
            const uint32_t g0 = i << gl2;
            if (gl2 <= 5) {
                const uint32_t width = 1u << gl2;
                const uint32_t m = width == 32 ? 0xffffffffu : ((1u << width) - 1u);
                f = ((ballot[g0 >> 5] >> (g0 & 31)) & m) != 0;
            } else {
                const uint32_t nw = 1u << (gl2 - 5);
                uint32_t acc = 0;
                for (uint32_t j = 0; j < nw; ++j) acc |= ballot[(g0 >> 5) + j];
                f = acc != 0;
            }
        }
        const uint32_t word = __ballot_sync(0xffffffffu, f);
        if (lane == 0) {
            bm[base >> 5] = word;
            pre[base >> 5] = (uint16_t)run;
        }
        run += __popc(word);
    }
    __syncwarp();
    return run;
}

__device__ __forceinline__ TileDesc load_tile_desc(const TileDesc* t) {
    const uint4* p = reinterpret_cast<const uint4*>(t);
    uint4 a = __ldg(p), b = __ldg(p + 1), c = __ldg(p + 2);
    TileDesc d;
    d.w_off = (uint64_t)a.x | ((uint64_t)a.y << 32);
    d.c_off = (uint64_t)a.z | ((uint64_t)a.w << 32);
    d.msg_off = (uint64_t)b.x | ((uint64_t)b.y << 32);
    d.n_unit = (uint64_t)b.z | ((uint64_t)b.w << 32);
    d.unit = c.x;
    d.tile_in_unit = c.y;
    d.first_tile = c.z;
    d.n_tiles_unit = c.w;
    return d;
}

}  // namespace ciera
