// Per-thread register work: one "group" = 16 consecutive values of one thread.
//
// Split and merge follow the paper's Section 3.1 (a value is sign, exponent and mantissa bits;
// the exponent travels apart from sign-plus-mantissa) on the IEEE binary32 / bfloat16 layouts:
//   bf16: bit 15 sign, bits 14:7 exponent, bits 6:0 mantissa  -> sm byte  = sign<<7  | mantissa
//   fp32: bit 31 sign, bits 30:23 exponent, bits 22:0 mantissa -> sm 24bit = sign<<23 | mantissa
// Everything is done on packed 32-bit words with shifts, three-input logic and byte permutes,
// four values at a time, so that a group's 16 exponent bytes end up as one uint4.
#pragma once

#include "ciera_internal.cuh"

namespace ciera {

__device__ __forceinline__ uint4 ld_stream16(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void st_stream16(void* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }
__device__ __forceinline__ uint4 ld_shared16(const void* p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"((uint32_t)__cvta_generic_to_shared(p)));
    return v;
}
__device__ __forceinline__ void st_shared16(void* p, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v.x),
                 "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
// where a group's 16-byte pieces come from: global memory (streaming) or a staged shared-memory tile
struct FromGlobal {
    __device__ __forceinline__ uint4 operator()(const uint8_t* p) const { return ld_stream16(p); }
};
struct FromShared {
    __device__ __forceinline__ uint4 operator()(const uint8_t* p) const { return ld_shared16(p); }
};

// ---- bf16 --------------------------------------------------------------------------------
// a = v0 | v1 << 16, b = v2 | v3 << 16  ->  e0 | e1<<8 | e2<<16 | e3<<24
__device__ __forceinline__ uint32_t bf16_exp4(uint32_t a, uint32_t b) { return __byte_perm(a >> 7, b >> 7, 0x6420); }
__device__ __forceinline__ uint32_t bf16_sm4(uint32_t a, uint32_t b) {
    uint32_t ya = (a & 0x007F007Fu) | ((a >> 8) & 0x00800080u);
    uint32_t yb = (b & 0x007F007Fu) | ((b >> 8) & 0x00800080u);
    return __byte_perm(ya, yb, 0x6420);
}
// four exponent bytes + four sm bytes -> two words of two bf16 each
__device__ __forceinline__ void bf16_merge4(uint32_t e, uint32_t s, uint32_t& lo, uint32_t& hi) {
    uint32_t e01 = __byte_perm(e, 0u, 0x4140), e23 = __byte_perm(e, 0u, 0x4342);
    uint32_t s01 = __byte_perm(s, 0u, 0x4140), s23 = __byte_perm(s, 0u, 0x4342);
    lo = ((s01 & 0x00800080u) << 8) | (e01 << 7) | (s01 & 0x007F007Fu);
    hi = ((s23 & 0x00800080u) << 8) | (e23 << 7) | (s23 & 0x007F007Fu);
}

// ---- fp32 --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t fp32_exp4(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
    uint32_t t01 = __byte_perm(w0 << 1, w1 << 1, 0x0073);  // byte0 = exp(w0), byte1 = exp(w1)
    uint32_t t23 = __byte_perm(w2 << 1, w3 << 1, 0x0073);
    return __byte_perm(t01, t23, 0x5410);
}
__device__ __forceinline__ uint32_t fp32_sm(uint32_t w) { return ((w >> 8) & 0x00800000u) | (w & 0x007FFFFFu); }
// four 24-bit sm values -> three little-endian words
__device__ __forceinline__ void fp32_pack4(uint32_t s0, uint32_t s1, uint32_t s2, uint32_t s3, uint32_t& o0,
                                           uint32_t& o1, uint32_t& o2) {
    o0 = s0 | (s1 << 24);
    o1 = (s1 >> 8) | (s2 << 16);
    o2 = (s2 >> 16) | (s3 << 8);
}
__device__ __forceinline__ void fp32_unpack4(uint32_t o0, uint32_t o1, uint32_t o2, uint32_t& s0, uint32_t& s1,
                                             uint32_t& s2, uint32_t& s3) {
    s0 = o0 & 0x00FFFFFFu;
    s1 = (o0 >> 24) | ((o1 & 0x0000FFFFu) << 8);
    s2 = (o1 >> 16) | ((o2 & 0x000000FFu) << 16);
    s3 = o2 >> 8;
}
__device__ __forceinline__ uint32_t fp32_merge(uint32_t e, uint32_t s) {
    return ((s & 0x00800000u) << 8) | (e << 23) | (s & 0x007FFFFFu);
}

// ---- a group in registers ------------------------------------------------------------------
template <int DT>
struct Group;

template <>
struct Group<CIERA_BF16> {
    uint32_t e[4];  // 16 exponent bytes
    uint32_t s[4];  // 16 sm bytes

    // 16 values from 32 aligned bytes
    template <class Ld = FromGlobal>
    __device__ __forceinline__ void split_full(const uint8_t* w, Ld ld = Ld()) {
        uint4 a = ld(w), b = ld(w + 16);
        e[0] = bf16_exp4(a.x, a.y); e[1] = bf16_exp4(a.z, a.w); e[2] = bf16_exp4(b.x, b.y); e[3] = bf16_exp4(b.z, b.w);
        s[0] = bf16_sm4(a.x, a.y);  s[1] = bf16_sm4(a.z, a.w);  s[2] = bf16_sm4(b.x, b.y);  s[3] = bf16_sm4(b.z, b.w);
    }
    // the first nvalid (< 16) values; the others read as +0.0 (exponent 0)
    __device__ __forceinline__ void split_partial(const uint8_t* w, int nvalid) {
        uint32_t x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = 0;
        const uint16_t* p = reinterpret_cast<const uint16_t*>(w);
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nvalid) x[i >> 1] |= (uint32_t)p[i] << (16 * (i & 1));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[i] = bf16_exp4(x[2 * i], x[2 * i + 1]);
            s[i] = bf16_sm4(x[2 * i], x[2 * i + 1]);
        }
    }
    __device__ __forceinline__ void store_sm_full(uint8_t* dst) const { st_stream16(dst, make_uint4(s[0], s[1], s[2], s[3])); }
    __device__ __forceinline__ void store_sm_partial(uint8_t* dst, int nvalid) const {
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nvalid) dst[i] = (uint8_t)(s[i >> 2] >> (8 * (i & 3)));
    }
    template <class Ld = FromGlobal>
    __device__ __forceinline__ void load_sm_full(const uint8_t* src, Ld ld = Ld()) {
        uint4 v = ld(src);
        s[0] = v.x; s[1] = v.y; s[2] = v.z; s[3] = v.w;
    }
    __device__ __forceinline__ void load_sm_partial(const uint8_t* src, int nvalid) {
#pragma unroll
        for (int i = 0; i < 4; ++i) s[i] = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nvalid) s[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
    }
    __device__ __forceinline__ void merge_store_full(uint8_t* w) const {
        uint4 a, b;
        bf16_merge4(e[0], s[0], a.x, a.y); bf16_merge4(e[1], s[1], a.z, a.w);
        bf16_merge4(e[2], s[2], b.x, b.y); bf16_merge4(e[3], s[3], b.z, b.w);
        st_stream16(w, a);
        st_stream16(w + 16, b);
    }
    __device__ __forceinline__ void merge_store_partial(uint8_t* w, int nvalid) const {
        uint32_t x[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) bf16_merge4(e[i], s[i], x[2 * i], x[2 * i + 1]);
        uint16_t* p = reinterpret_cast<uint16_t*>(w);
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nvalid) p[i] = (uint16_t)(x[i >> 1] >> (16 * (i & 1)));
    }
};

template <>
struct Group<CIERA_FP32> {
    uint32_t e[4];   // 16 exponent bytes
    uint32_t s[12];  // 16 x 24-bit sm, packed little-endian

    __device__ __forceinline__ void from_words(const uint32_t* x) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[i] = fp32_exp4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
            fp32_pack4(fp32_sm(x[4 * i]), fp32_sm(x[4 * i + 1]), fp32_sm(x[4 * i + 2]), fp32_sm(x[4 * i + 3]),
                       s[3 * i], s[3 * i + 1], s[3 * i + 2]);
        }
    }
    template <class Ld = FromGlobal>
    __device__ __forceinline__ void split_full(const uint8_t* w, Ld ld = Ld()) {
        uint32_t x[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 v = ld(w + 16 * i);
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
    __device__ __forceinline__ void store_sm_full(uint8_t* dst) const {
#pragma unroll
        for (int i = 0; i < 3; ++i) st_stream16(dst + 16 * i, make_uint4(s[4 * i], s[4 * i + 1], s[4 * i + 2], s[4 * i + 3]));
    }
    __device__ __forceinline__ void store_sm_partial(uint8_t* dst, int nvalid) const {
#pragma unroll
        for (int i = 0; i < 48; ++i)
            if (i < 3 * nvalid) dst[i] = (uint8_t)(s[i >> 2] >> (8 * (i & 3)));
    }
    template <class Ld = FromGlobal>
    __device__ __forceinline__ void load_sm_full(const uint8_t* src, Ld ld = Ld()) {
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            uint4 v = ld(src + 16 * i);
            s[4 * i] = v.x; s[4 * i + 1] = v.y; s[4 * i + 2] = v.z; s[4 * i + 3] = v.w;
        }
    }
    __device__ __forceinline__ void load_sm_partial(const uint8_t* src, int nvalid) {
#pragma unroll
        for (int i = 0; i < 12; ++i) s[i] = 0;
#pragma unroll
        for (int i = 0; i < 48; ++i)
            if (i < 3 * nvalid) s[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
    }
    __device__ __forceinline__ void merge_words(uint32_t* x) const {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t s0, s1, s2, s3;
            fp32_unpack4(s[3 * i], s[3 * i + 1], s[3 * i + 2], s0, s1, s2, s3);
            x[4 * i] = fp32_merge(e[i] & 0xFFu, s0);
            x[4 * i + 1] = fp32_merge((e[i] >> 8) & 0xFFu, s1);
            x[4 * i + 2] = fp32_merge((e[i] >> 16) & 0xFFu, s2);
            x[4 * i + 3] = fp32_merge(e[i] >> 24, s3);
        }
    }
    __device__ __forceinline__ void merge_store_full(uint8_t* w) const {
        uint32_t x[16];
        merge_words(x);
#pragma unroll
        for (int i = 0; i < 4; ++i) st_stream16(w + 16 * i, make_uint4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]));
    }
    __device__ __forceinline__ void merge_store_partial(uint8_t* w, int nvalid) const {
        uint32_t x[16];
        merge_words(x);
        uint32_t* p = reinterpret_cast<uint32_t*>(w);
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nvalid) p[i] = x[i];
    }
};

// 16 exponent bytes <-> memory
__device__ __forceinline__ void load_exp_partial(uint32_t* e, const uint8_t* src, int nvalid) {
#pragma unroll
    for (int i = 0; i < 4; ++i) e[i] = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i)
        if (i < nvalid) e[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
}
__device__ __forceinline__ void store_exp_partial(uint8_t* dst, const uint32_t* e, int nvalid) {
#pragma unroll
    for (int i = 0; i < 16; ++i)
        if (i < nvalid) dst[i] = (uint8_t)(e[i >> 2] >> (8 * (i & 3)));
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
