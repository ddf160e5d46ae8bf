// fp16 (IEEE binary16: 1 sign, 5 exponent, 10 mantissa bits) through the same method (paper
// Section 3.1 speaks of "FP16 and BF16"; Section 3.2 gives sizes for any b-bit precision).
//
// On the wire an exponent takes 5 bits and a sign-plus-mantissa 11 bits (sm = sign << 10 | mantissa),
// packed without gaps: value j of a section sits at bits [j*w, (j+1)*w), bit i of a section is bit
// i & 7 of byte i >> 3; every changed block of the payload starts on a byte boundary.  The caches
// hold one byte per value, as for the other precisions.  Eight values make 11 bytes of
// sign-plus-mantissa and 5 bytes of exponents, so a piece of 8 values owns whole bytes of both.
//
// This precision takes the plain route of several launches (see ciera_multipass.cuh), one thread
// block per tile, nothing waiting on anything:
//   sender    scan (split, compare with the cache and refresh it, packed sign-plus-mantissa out, block
//             flags to the scratch) -> unit (payload offsets, bitmap, pads, totals) -> payload (packed
//             exponents of flagged blocks; their weights are read a second time)
//   receiver  the per-tile counts of changed blocks (the prefix kernel of the decode path), then one
//             block per tile: flags from the bitmap, exponents from the payload or the cache, merge.
// Blocks of 32 values and more (four pieces), so that the four lanes that share 44 bytes of packed
// sign-plus-mantissa always lie in one block.
#include "ciera_bits.cuh"
#include "ciera_multipass.cuh"

namespace ciera {

// thread -> value layout as for bf16: two pieces of 8 values per thread
__device__ __forceinline__ uint32_t h_start(uint32_t tid, int p) { return (uint32_t)p * (kTileValues / 2) + tid * 8u; }

struct HalfPiece {
    uint32_t e[2];  // 8 exponents, one byte each (0..31)
    uint32_t s[3];  // 8 x 11 bits of sign-plus-mantissa, packed (88 bits)

    // w = eight fp16 values, two per word
    __device__ __forceinline__ void split(const uint32_t w[4]) {
        uint32_t e2[4], f[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e2[i] = (w[i] >> 10) & 0x001F001Fu;
            const uint32_t sm2 = (w[i] & 0x03FF03FFu) | ((w[i] >> 5) & 0x04000400u);
            f[2 * i] = sm2 & 0xFFFFu;
            f[2 * i + 1] = sm2 >> 16;
        }
        e[0] = __byte_perm(e2[0], e2[1], 0x6420);
        e[1] = __byte_perm(e2[2], e2[3], 0x6420);
        s[0] = f[0] | (f[1] << 11) | (f[2] << 22);
        s[1] = (f[2] >> 10) | (f[3] << 1) | (f[4] << 12) | (f[5] << 23);
        s[2] = (f[5] >> 9) | (f[6] << 2) | (f[7] << 13);
    }
    __device__ __forceinline__ void merge(uint32_t w[4]) const {
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
    __device__ __forceinline__ bool differs(const uint32_t c[2]) const { return ((e[0] ^ c[0]) | (e[1] ^ c[1])) != 0; }
};

// the first nvalid (1..8) values of a piece from global memory; the others read as +0.0
__device__ __forceinline__ void load_halves(uint32_t w[4], const uint8_t* src, int nvalid) {
    if (nvalid == 8) {
        const uint4 v = ld_stream16(src);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else {
        const uint16_t* p = reinterpret_cast<const uint16_t*>(src);
        w[0] = w[1] = w[2] = w[3] = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i < nvalid) w[i >> 1] |= (uint32_t)p[i] << (16 * (i & 1));
    }
}
__device__ __forceinline__ void load_exp_bytes(uint32_t c[2], const uint8_t* src, int nvalid) {
    if (nvalid == 8) {
        const uint2 v = ld_stream8(src);
        c[0] = v.x; c[1] = v.y;
    } else {
        load_bytes_partial<8>(c, src, nvalid);
    }
}
__device__ __forceinline__ void store_exp_bytes(uint8_t* dst, const uint32_t e[2], int nvalid) {
    if (nvalid == 8)
        st_stream8(dst, make_uint2(e[0], e[1]));
    else
        store_bytes_partial<8>(dst, e, nvalid);
}

// Packed sign-plus-mantissa of a piece to/from the message.  `full_tile`: every piece of the tile is
// complete, and the four lanes 4k..4k+3 share 44 bytes = 11 aligned words: lane a holds bits
// [88a, 88a+88) of them and writes words 3a, 3a+1, 3a+2 (lane 3: two words), taking the low bits of
// the next lane's first word where its own bits end inside a word.  Otherwise byte by byte.
__device__ __forceinline__ void store_sm(uint8_t* section, uint32_t t0, const uint32_t s[3], int nvalid, bool full_tile,
                                         uint32_t lane) {
    if (full_tile) {
        const uint32_t a = lane & 3u, sh = 8u * a;
        const uint32_t next0 = __shfl_down_sync(0xffffffffu, s[0], 1);
        uint32_t* dst = reinterpret_cast<uint32_t*>(section + (size_t)11 * ((t0 >> 3) - a)) + 3u * a;
        const uint32_t w0 = sh ? (s[0] >> sh) | (s[1] << (32u - sh)) : s[0];
        const uint32_t w1 = sh ? (s[1] >> sh) | (s[2] << (32u - sh)) : s[1];
        dst[0] = w0;
        dst[1] = w1;
        if (a != 3u) dst[2] = (s[2] >> sh) | (next0 << (24u - sh));
    } else if (nvalid > 0) {
        uint8_t* dst = section + (size_t)11 * (t0 >> 3);
        const int nbytes = (11 * nvalid + 7) >> 3;
        for (int i = 0; i < nbytes; ++i) dst[i] = (uint8_t)(s[i >> 2] >> (8 * (i & 3)));
    }
}
__device__ __forceinline__ void load_sm(uint32_t s[3], const uint8_t* section, uint32_t t0, int nvalid, bool full_tile,
                                        uint32_t lane) {
    if (full_tile) {
        const uint32_t a = lane & 3u;
        // lane a's bits start at bit 88a of the group: word {0, 2, 5, 8}, bit {0, 24, 16, 8}
        const uint32_t first = (11u * a) >> 2, sh = (8u * 11u * a) & 31u;
        const uint32_t* src = reinterpret_cast<const uint32_t*>(section + (size_t)11 * ((t0 >> 3) - a)) + first;
        const uint32_t w0 = __ldcs(src), w1 = __ldcs(src + 1), w2 = __ldcs(src + 2);
        const uint32_t w3 = (a == 0u || a == 3u) ? 0u : __ldcs(src + 3);  // lanes 0 and 3 end inside their third word
        s[0] = sh ? (w0 >> sh) | (w1 << (32u - sh)) : w0;
        s[1] = sh ? (w1 >> sh) | (w2 << (32u - sh)) : w1;
        s[2] = (sh ? (w2 >> sh) | (w3 << (32u - sh)) : w2) & 0x00FFFFFFu;
    } else {
        s[0] = s[1] = s[2] = 0;
        const uint8_t* src = section + (size_t)11 * (t0 >> 3);
        const int nbytes = (11 * nvalid + 7) >> 3;
        for (int i = 0; i < nbytes; ++i) s[i >> 2] |= (uint32_t)src[i] << (8 * (i & 3));
    }
}

// ------------------------------------------------------------------------------------------
// cache := exponents(weights) (or zero)

__global__ void __launch_bounds__(kThreads)
fp16_cache_fill_kernel(const TileDesc* __restrict__ tiles, const uint8_t* __restrict__ weights, uint8_t* __restrict__ cache) {
    const TileDesc td = load_tile_desc(tiles + blockIdx.x);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t t0 = h_start(threadIdx.x, p);
        const int nvalid = t0 >= nv ? 0 : (int)min(8u, nv - t0);
        if (nvalid == 0) continue;
        HalfPiece x;
        x.e[0] = x.e[1] = 0;
        if (weights != nullptr) {
            uint32_t w[4];
            load_halves(w, weights + td.w_off + (uint64_t)t0 * 2, nvalid);
            x.split(w);
        }
        store_exp_bytes(cache + td.c_off + t0, x.e, nvalid);
    }
}

// ------------------------------------------------------------------------------------------ sender

__global__ void __launch_bounds__(kThreads)
fp16_scan_kernel(const TileDesc* __restrict__ tiles, uint32_t log2b, const uint8_t* __restrict__ weights, uint8_t* cache,
                 uint8_t* msgs, uint32_t* ws) {
    __shared__ uint32_t s_ballot[32];
    __shared__ uint32_t s_bm[kBitmapWords];
    __shared__ uint16_t s_pre[kBitmapWords];
    const uint32_t tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const TileDesc td = load_tile_desc(tiles + tile);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const bool full_tile = nv == (uint32_t)kTileValues;
    // the tile's part of the packed sign-plus-mantissa section: 11 bytes per 8 values
    uint8_t* section = msgs + td.msg_off + sm_offset(td.n_unit, log2b) + (v0 >> 3) * 11;
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t t0 = h_start(tid, p);
        const int nvalid = t0 >= nv ? 0 : (int)min(8u, nv - t0);
        HalfPiece x;
        x.e[0] = x.e[1] = x.s[0] = x.s[1] = x.s[2] = 0;
        bool diff = false;
        if (nvalid > 0) {
            uint32_t w[4], c[2];
            load_halves(w, weights + td.w_off + (uint64_t)t0 * 2, nvalid);
            x.split(w);
            load_exp_bytes(c, cache + td.c_off + t0, nvalid);
            diff = x.differs(c);
            // cache refreshed where it differs (the other pieces of a changed block hold the same bytes already)
            if (diff) store_exp_bytes(cache + td.c_off + t0, x.e, nvalid);
        }
        store_sm(section, t0, x.s, nvalid, full_tile, lane);
        const uint32_t votes = __ballot_sync(0xffffffffu, diff);
        if (lane == 0) s_ballot[p * kWarps + warp] = votes;
    }
    __syncthreads();
    if (warp == 0) {
        const uint32_t run = build_block_bitmap(s_ballot, s_bm, s_pre, log2b, 3, lane);
        if (lane < kRecWords) ws[(size_t)tile * kRecWords + lane] = lane < kFlagWords ? s_bm[lane] : run;  // flags, count (, offset)
    }
}

// one thread block per tile, every warp on its own: packed exponents of the flagged blocks
__global__ void __launch_bounds__(kThreads)
fp16_payload_kernel(const TileDesc* __restrict__ tiles, uint32_t log2b, const uint8_t* __restrict__ weights, uint8_t* msgs,
                    const uint32_t* __restrict__ ws) {
    const uint32_t tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31u;
    const uint32_t* rec = ws + (size_t)tile * kRecWords;
    uint32_t word[2];
    bool flagged[2];
    bool any = false;
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t kb = h_start(tid, p) >> log2b;
        word[p] = __ldg(rec + (kb >> 5));
        flagged[p] = (word[p] >> (kb & 31u)) & 1u;
        any |= flagged[p];
    }
    if (!__any_sync(0xffffffffu, any)) return;
    const uint32_t word_l = lane < kFlagWords ? __ldg(rec + lane) : 0u;
    const uint32_t prefix = __ldg(rec + kRecPrefix);
    const uint32_t pc = __popc(word_l);
    uint32_t incl = pc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)lane >= o) incl += t;
    }
    const uint32_t pre_l = incl - pc;
    uint32_t rank[2];
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t kb = h_start(tid, p) >> log2b;
        rank[p] = __shfl_sync(0xffffffffu, pre_l, kb >> 5) + __popc(word[p] & ((1u << (kb & 31u)) - 1u));
    }
    const TileDesc td = load_tile_desc(tiles + tile);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const uint32_t B = 1u << log2b;
    const uint32_t bpb = 5u * (B >> 3);  // bytes of a full block in the payload
    uint8_t* pay = msgs + td.msg_off + payload_offset_of(td.n_unit, CIERA_FP16, log2b) + (uint64_t)prefix * bpb;
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t t0 = h_start(tid, p);
        const int nvalid = t0 >= nv ? 0 : (int)min(8u, nv - t0);
        if (!flagged[p] || nvalid == 0) continue;
        uint32_t w[4], lo, hi;
        load_halves(w, weights + td.w_off + (uint64_t)t0 * 2, nvalid);
        HalfPiece x;
        x.split(w);
        x.pack_exponents(lo, hi);
        uint8_t* dst = pay + (uint64_t)rank[p] * bpb + 5u * ((t0 & (B - 1u)) >> 3);
        const int nbytes = (5 * nvalid + 7) >> 3;
        for (int i = 0; i < nbytes; ++i) dst[i] = (uint8_t)(i < 4 ? lo >> (8 * i) : hi);
    }
}

// ---------------------------------------------------------------------------------------- receiver

// One thread block per tile, every warp on its own (no barrier, no shared memory): a warp reads the
// tile's words of the unit's bitmap itself and ranks them with shuffles.  What does not depend on
// the flags -- the packed sign-plus-mantissa and the cached exponents of the warp's pieces -- is
// requested first, so that those loads are under way while the flags arrive.
__global__ void __launch_bounds__(kThreads)
fp16_decode_kernel(const TileDesc* __restrict__ tiles, uint32_t log2b, const uint8_t* msgs, uint8_t* cache,
                   uint8_t* __restrict__ weights, const unsigned long long* __restrict__ wire_bytes,
                   const uint32_t* __restrict__ ws_prefix, int32_t* status) {
    const uint32_t tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31u;
    const TileDesc td = load_tile_desc(tiles + tile);
    const uint64_t N = td.n_unit;
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, N - v0);
    const bool full_tile = nv == (uint32_t)kTileValues;
    const uint32_t B = 1u << log2b;
    const uint32_t nbt = kTileValues >> log2b;  // at most 256 blocks (B >= 32): 8 words of flags
    const uint32_t nblk = (nv + B - 1u) >> log2b;
    const uint8_t* msg = msgs + td.msg_off;
    const uint8_t* section = msg + sm_offset(N, log2b) + (v0 >> 3) * 11;

    // 1. loads that need no flags
    HalfPiece x[2];
    uint32_t c[2][2];
    int nvalid[2];
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t t0 = h_start(tid, p);
        nvalid[p] = t0 >= nv ? 0 : (int)min(8u, nv - t0);
        load_sm(x[p].s, section, t0, nvalid[p], full_tile, lane);
        c[p][0] = c[p][1] = 0;
        if (nvalid[p] > 0) load_exp_bytes(c[p], cache + td.c_off + t0, nvalid[p]);
    }
    // 2. the tile's block flags from the unit's bitmap, set flags before each word, their total
    uint32_t word_l = 0;
    {
        const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msg);
        const uint64_t kb0 = (uint64_t)td.tile_in_unit * nbt;
        if (nbt >= 32) {
            if (lane < (nbt >> 5) && lane * 32u < nblk) {
                word_l = bm32[(kb0 >> 5) + lane];
                const uint32_t left = nblk - lane * 32u;
                if (left < 32u) word_l &= (1u << left) - 1u;
            }
        } else if (lane == 0) {
            word_l = (bm32[kb0 >> 5] >> (kb0 & 31u)) & ((1u << nblk) - 1u);
        }
    }
    const uint64_t before = td.tile_in_unit != 0 ? ws_prefix[tile] : 0u;  // changed blocks in the unit's earlier tiles
    const uint32_t pc = __popc(word_l);
    uint32_t incl = pc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)lane >= o) incl += t;
    }
    const uint32_t pre_l = incl - pc;
    const uint32_t own = __shfl_sync(0xffffffffu, incl, 31);
    const uint32_t bpb = 5u * (B >> 3);
    const uint64_t payoff = payload_offset_of(N, CIERA_FP16, log2b);
    // integrity check by the unit's last tile: the bitmap fixes the message length
    if (wire_bytes != nullptr && status != nullptr && td.tile_in_unit == td.n_tiles_unit - 1u && tid < 32) {
        uint64_t total = (before + own) * bpb;
        const uint32_t rem = (uint32_t)(N & (B - 1u));
        const uint32_t kb = nv >> log2b;  // the short last block, if there is one
        const uint32_t last_word = __shfl_sync(0xffffffffu, word_l, (kb >> 5) & 31u);
        if (rem && ((last_word >> (kb & 31u)) & 1u)) total -= bpb - (uint32_t)block_payload_bytes(rem, CIERA_FP16);
        if (lane == 0 && wire_bytes[td.unit] != payoff + total) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
    }
    const uint8_t* pay = msg + payoff + before * bpb;
    // 3. exponents of changed blocks from the payload, merge, store
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t t0 = h_start(tid, p);
        const uint32_t kb = t0 >> log2b;
        const uint32_t word = __shfl_sync(0xffffffffu, word_l, (kb >> 5) & 31u);
        const uint32_t pre = __shfl_sync(0xffffffffu, pre_l, (kb >> 5) & 31u);
        if (nvalid[p] == 0) continue;
        const bool chg = (word >> (kb & 31u)) & 1u;
        if (chg) {
            const uint32_t rank = pre + __popc(word & ((1u << (kb & 31u)) - 1u));
            const uint8_t* src = pay + (uint64_t)rank * bpb + 5u * ((t0 & (B - 1u)) >> 3);
            const int nbytes = (5 * nvalid[p] + 7) >> 3;
            uint32_t lo = 0, hi = 0;
            for (int i = 0; i < nbytes; ++i) {
                const uint32_t b = src[i];
                if (i < 4)
                    lo |= b << (8 * i);
                else
                    hi = b;
            }
            x[p].unpack_exponents(lo, hi);
            store_exp_bytes(cache + td.c_off + t0, x[p].e, nvalid[p]);  // ExpCache[i,k] <- newExp[j]
        } else {
            x[p].e[0] = c[p][0];
            x[p].e[1] = c[p][1];
        }
        uint32_t w[4];
        x[p].merge(w);
        uint8_t* dst = weights + td.w_off + (uint64_t)t0 * 2;
        if (nvalid[p] == 8) {
            st_stream16(dst, make_uint4(w[0], w[1], w[2], w[3]));
        } else {
            uint16_t* d16 = reinterpret_cast<uint16_t*>(dst);
            for (int i = 0; i < nvalid[p]; ++i) d16[i] = (uint16_t)(w[i >> 1] >> (16 * (i & 1)));
        }
    }
}

// launchers (called from the C entry points)
int fp16_cache_fill(const ciera_plan* p, void* cache_dev, const void* weights_dev, cudaStream_t s) {
    const uint32_t nt = (uint32_t)p->tiles.size();
    fp16_cache_fill_kernel<<<nt, kThreads, 0, s>>>(p->tiles_dev, (const uint8_t*)weights_dev, (uint8_t*)cache_dev);
    count_launch();
    return check_launch();
}

int fp16_encode(const ciera_plan* p, const void* weights_dev, void* sender_cache_dev, void* messages_dev,
                uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* workspace_dev, cudaStream_t s) {
    const uint32_t nt = (uint32_t)p->tiles.size();
    uint32_t* ws = (uint32_t*)workspace_dev;
    if (nt != 0) {
        fp16_scan_kernel<<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)weights_dev,
                                                 (uint8_t*)sender_cache_dev, (uint8_t*)messages_dev, ws);
        count_launch();
        int rc = check_launch();
        if (rc) return rc;
    }
    multipass_unit_kernel<<<p->n_units, 256, 0, s>>>(p->tiles_dev, p->unit_first_dev, p->log2b, CIERA_FP16,
                                                     (uint8_t*)messages_dev, ws, (unsigned long long*)wire_bytes_dev,
                                                     changed_blocks_dev);
    count_launch();
    int rc = check_launch();
    if (rc || nt == 0) return rc;
    fp16_payload_kernel<<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)weights_dev, (uint8_t*)messages_dev,
                                                ws);
    count_launch();
    return check_launch();
}

int fp16_decode(const ciera_plan* p, const void* messages_dev, void* receiver_cache_dev, void* weights_out_dev,
                const uint64_t* wire_bytes_dev, const uint32_t* ws_prefix, int32_t* status_dev, cudaStream_t s) {
    const uint32_t nt = (uint32_t)p->tiles.size();
    fp16_decode_kernel<<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)messages_dev,
                                               (uint8_t*)receiver_cache_dev, (uint8_t*)weights_out_dev,
                                               (const unsigned long long*)wire_bytes_dev, ws_prefix, status_dev);
    count_launch();
    return check_launch();
}

}  // namespace ciera
