// Receiver side (paper Algorithm 1, receiver part; Section 3.1) as one persistent sm_100a kernel.
//
// Grid = at most as many thread blocks as fit on the GPU.  Tiles are independent here, so they
// are handed out dynamically: every producer warp draws the next tile number from a counter in
// the caller's scratch, which keeps all SMs busy to the end whatever their individual pace.
// Two roles:
//
//   producer warps  run ahead, taking the block's tiles in turn: for each tile a producer reads
//                   the tile's bits of the unit's bitmap and the number of changed blocks before
//                   the tile, works out the tile's addresses once for everybody, and fills a
//                   shared-memory stage with three bulk-async copies: the received
//                   sign-plus-mantissa tile, the span of the receiver's cached exponents that
//                   covers the tile's unchanged blocks, and the slice of the message payload that
//                   holds the tile's changed blocks (they are contiguous there, in block order);
//   16 consumer     each thread merges the exponent bytes (from the cache span, or from the
//   warps           payload slice if its block changed) and the sign-plus-mantissa of its pieces
//                   into weights and stores them; threads of changed blocks also store the new
//                   exponents to the cache (ExpCache[i,k] <- newExp[j]).
//
// The number of changed blocks before a tile is the popcount of the bitmap bits before it.  For
// units of up to kDirectBlocks blocks a producer takes it straight from the bitmap (at most four
// words per lane, fetched one tile ahead); longer units get it from a small prefix kernel that
// runs first and writes one count per tile into the caller's scratch.
#include <cstddef>

#include "ciera_bits.cuh"
#include "ciera_pipe.cuh"

namespace ciera {

constexpr int kDecProducers = 2;                               // producer warps, taking tiles in turn
constexpr int kDecodeThreads = kThreads + 32 * kDecProducers;  // consumers + producers
constexpr int kDecProducerWarp0 = kWarps;
constexpr uint32_t kNoTile = 0xffffffffu;
constexpr uint32_t kDirectWordsPerLane = 4;
constexpr uint32_t kDirectBlocks = kDecodeDirectBlocks;
static_assert(kDirectBlocks == 32u * 32u * kDirectWordsPerLane, "one fetch covers the direct range");

// kRing: slots of per-tile bookkeeping; > stages + 2 * producers + 1, since a slot is refilled
// only after its tile is done.  With fine blocks (see ciera_internal.cuh) a slot holds up to 8192
// block flags instead of 512.
template <int DT, bool FINE>
struct DecodeCfg;
template <>
struct DecodeCfg<CIERA_BF16, false> {
    static constexpr int kStages = 4;        // 4 x (8 KB sm + 8 KB cache span + 8 KB payload slice)
    static constexpr int kBlocksPerSM = 2;
    static constexpr bool kStageOut = false;  // weights leave as 16 B / lane, contiguous per warp
    static constexpr int kRing = 12;
};
template <>
struct DecodeCfg<CIERA_FP32, false> {
    static constexpr int kStages = 4;        // 4 x (24 KB sm + 8 KB + 8 KB)
    static constexpr int kBlocksPerSM = 1;
    static constexpr bool kStageOut = true;   // 64 B / lane: staged, then one bulk store per warp
    static constexpr int kRing = 12;
};
template <>
struct DecodeCfg<CIERA_FP16, false> {
    static constexpr int kStages = 4;        // 4 x (11 KB sm + 8 KB cache span + 5 KB packed payload slice)
    static constexpr int kBlocksPerSM = 2;
    static constexpr bool kStageOut = false;
    static constexpr int kRing = 12;
};
template <>
struct DecodeCfg<CIERA_BF16, true> {
    static constexpr int kStages = 4;
    static constexpr int kBlocksPerSM = 2;
    static constexpr bool kStageOut = false;
    static constexpr int kRing = 10;
};
template <>
struct DecodeCfg<CIERA_FP16, true> {
    // 4 x (11 KB sm + 8 KB cache span + 8 KB payload slice): one block per SM (two blocks with two stages each
    // measured slower: 0.70 against 0.56 ms per layer)
    static constexpr int kStages = 4;
    static constexpr int kBlocksPerSM = 1;
    static constexpr bool kStageOut = false;
    static constexpr int kRing = 10;
};
template <>
struct DecodeCfg<CIERA_FP32, true> {
    static constexpr int kStages = 4;
    static constexpr int kBlocksPerSM = 1;
    static constexpr bool kStageOut = true;
    static constexpr int kRing = 12;
};

// Per-tile bookkeeping, in a ring that the producers fill ahead of the consumers.
template <bool FINE>
struct __align__(16) DecodeRing {
    static constexpr int kBm = FINE ? kFineBitmapWords : kBitmapWords;
    TileDesc desc;                           // copied from the plan's table (asynchronously)
    // the tile's block flags; with fine blocks they are fetched straight into this array
    uint32_t bm[kBm];
    // worked out once by a producer for the 512 consumer threads:
    uint8_t* w_dst;                          // where the tile's reconstructed weights go
    uint8_t* c_ptr;                          // the tile's cached exponents
    const uint8_t* sm_src;                   // the tile's received sign-plus-mantissa
    const uint8_t* pay_src;                  // the payload slice holding the tile's changed blocks
    uint32_t nv;                             // values in the tile
    uint32_t tile;                           // the tile's number, or kNoTile: this producer has no more work
    uint32_t pay_skew;                       // fine: bytes in front of the slice in its stage (0 .. 15)
    uint32_t ws;                             // count from the scratch (units that went through the prefix kernel)
    uint32_t direct;                         // coarse: 1 = the few unchanged pieces read their cached exponents from global memory
    uint16_t pre[kBm];                       // set flags before each word
    // raw material of coarse blocks, fetched asynchronously one tile ahead:
    uint32_t raw_pre[FINE ? 4 : 32 * kDirectWordsPerLane];  // bitmap words before the tile
    uint32_t raw_own[FINE ? 4 : kBitmapWords];               // words holding the tile's own bits
};

static_assert(offsetof(DecodeRing<true>, bm) % 16 == 0 && offsetof(DecodeRing<true>, pre) % 4 == 0,
              "with blocks of one value the flags are digested 16 bytes at a time");

template <int S, int R, bool FINE>
struct DecodeCtl {
    uint64_t full[S];   // stage filled (producer arrive + bulk-copy bytes)
    uint64_t empty[S];  // all 16 consumer warps have read it
    DecodeRing<FINE> ring[R];
    int abort;
    uint32_t issued;
    uint32_t seen;
};

// Starts the asynchronous fetch of the bitmap words a producer needs for one tile into the ring
// slot `r`: the unit's words before the tile (direct units) or the tile's count from the scratch
// (long units), and the tile's own words.  Nothing is held in registers meanwhile.
template <bool FINE>
__device__ __forceinline__ void fetch_bitmap(const TileDesc& td, uint32_t tile, uint32_t log2b, const uint8_t* msgs,
                                             const uint32_t* ws_prefix, DecodeRing<FINE>* r, uint32_t lane) {
    const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msgs + td.msg_off);
    const uint64_t kb0 = ((uint64_t)td.tile_in_unit * kTileValues) >> log2b;  // first block of the tile
    const uint64_t nb = num_blocks(td.n_unit, log2b);
    const uint32_t nbt = kTileValues >> log2b;
    if (FINE) {
        // every unit of more than one tile has its counts in the scratch; the tile's own flags are
        // 128 to 1024 bytes that start on a 128-byte boundary of the slot: 16 bytes per copy,
        // never past the bitmap's padded end
        if (td.tile_in_unit != 0 && lane == 0) cp_async4(&r->ws, ws_prefix + tile);
        const uint32_t chunks = nbt >> 7;  // 8 .. 64 copies of four words
        for (uint32_t c = lane; c < chunks; c += 32) {
            const uint64_t w = (kb0 >> 5) + 4ull * c;
            if ((w << 5) < nb) cp_async16(&r->bm[4u * c], bm32 + w);
        }
        return;
    }
    if (nb <= kDirectBlocks) {
        const uint32_t nwords = (uint32_t)((kb0 + 31) >> 5);  // words holding bits before kb0
#pragma unroll
        for (uint32_t i = 0; i < kDirectWordsPerLane; ++i) {
            const uint32_t w = lane + 32u * i;
            if (w < nwords) cp_async4(&r->raw_pre[w], bm32 + w);
        }
    } else if (lane == 0) {
        cp_async4(&r->ws, ws_prefix + tile);
    }
    // the tile's own bits: nbt >= 32 -> words (kb0 >> 5) + lane; nbt < 32 -> part of one word
    const uint32_t own_words = nbt >= 32 ? (nbt >> 5) : 1u;
    if (lane < own_words) {
        const uint64_t w = (kb0 >> 5) + lane;
        if ((w << 5) < nb) cp_async4(&r->raw_own[lane], bm32 + w);  // never past the bitmap's padded end
    }
}

// Turns a completed fetch into the tile's block flags (r->bm, r->pre).  Returns the number of
// changed blocks before the tile; `own_total` gets the number of changed blocks of the tile.
template <bool FINE>
__device__ __forceinline__ uint64_t digest_bitmap(DecodeRing<FINE>* r, const TileDesc& td, uint32_t log2b, uint32_t lane,
                                                  uint32_t& own_total) {
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint64_t kb0 = v0 >> log2b;
    const uint64_t nb = num_blocks(td.n_unit, log2b);
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const uint32_t nblk = (nv + (1u << log2b) - 1u) >> log2b;  // valid blocks of this tile
    uint32_t cnt = 0;
    if (FINE && log2b == 0) {
        // blocks of one value: 256 words; lane l takes words 8 l .. 8 l + 7, one scan does for the tile
        uint32_t w[8], before8[8], sum = 0;
        uint4* const bm4 = reinterpret_cast<uint4*>(r->bm) + 2u * lane;
        const uint4 v0w = bm4[0], v1w = bm4[1];
        w[0] = v0w.x; w[1] = v0w.y; w[2] = v0w.z; w[3] = v0w.w;
        w[4] = v1w.x; w[5] = v1w.y; w[6] = v1w.z; w[7] = v1w.w;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t first = (8u * lane + (uint32_t)i) * 32u;  // the word's first block
            // flags past the tile's last block are dropped (words past the bitmap's end were not fetched)
            if (first >= nblk)
                w[i] = 0;
            else if (nblk - first < 32u)
                w[i] &= (1u << (nblk - first)) - 1u;
            before8[i] = sum;
            sum += __popc(w[i]);
        }
        uint32_t incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += t;
        }
        const uint32_t base = incl - sum;
        bm4[0] = make_uint4(w[0], w[1], w[2], w[3]);
        bm4[1] = make_uint4(w[4], w[5], w[6], w[7]);
        uint32_t* const pre32 = reinterpret_cast<uint32_t*>(r->pre) + 4u * lane;
#pragma unroll
        for (int i = 0; i < 4; ++i) pre32[i] = (base + before8[2 * i]) | ((base + before8[2 * i + 1]) << 16);
        own_total = __shfl_sync(0xffffffffu, incl, 31);
        __syncwarp();
        return td.tile_in_unit != 0 ? r->ws : 0u;
    }
    if (FINE) {
        // flags past the tile's last block are dropped (words past the bitmap's end were not fetched)
        uint32_t run = 0;
        for (uint32_t base = 0; base < (nbt >> 5); base += 32) {
            const uint32_t w = base + lane;
            uint32_t word = 0;
            if (w * 32u < nblk) {
                word = r->bm[w];
                const uint32_t left = nblk - w * 32u;
                if (left < 32u) word &= (1u << left) - 1u;
            }
            const uint32_t pc = __popc(word);
            uint32_t incl = pc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                if ((int)lane >= o) incl += t;
            }
            r->bm[w] = word;
            r->pre[w] = (uint16_t)(run + incl - pc);
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        own_total = run;
        __syncwarp();
        return td.tile_in_unit != 0 ? r->ws : 0u;
    }
    if (nb <= kDirectBlocks) {
        const uint32_t nfull = (uint32_t)(kb0 >> 5);
#pragma unroll
        for (uint32_t i = 0; i < kDirectWordsPerLane; ++i) {
            const uint32_t w = lane + 32u * i;
            if (w < nfull)
                cnt += __popc(r->raw_pre[w]);
            else if (w == nfull && (kb0 & 31u))
                cnt += __popc(r->raw_pre[w] & ((1u << (kb0 & 31u)) - 1u));
        }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
    } else {
        cnt = r->ws;
    }
    uint32_t word = 0;
    if (nbt >= 32) {
        if (lane < (nbt >> 5) && lane * 32u < nblk) {
            word = r->raw_own[lane];
            const uint32_t left = nblk - lane * 32u;
            if (left < 32u) word &= (1u << left) - 1u;
        }
    } else if (lane == 0) {
        word = (r->raw_own[0] >> (kb0 & 31u)) & ((1u << nblk) - 1u);
    }
    // exclusive popcount prefix over the (at most 16) words
    const uint32_t pc = __popc(word);
    uint32_t incl = pc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)lane >= o) incl += t;
    }
    if (lane < kBitmapWords) {
        r->bm[lane] = word;
        r->pre[lane] = (uint16_t)(incl - pc);
    }
    own_total = __shfl_sync(0xffffffffu, incl, 31);
    __syncwarp();
    return cnt;
}

// First and last unchanged block of a full tile (lo > hi if every block changed).  One warp;
// lane w looks at word w of the block flags.
__device__ __forceinline__ void unchanged_span(const uint32_t* bm, uint32_t log2b, uint32_t lane, uint32_t& lo,
                                               uint32_t& hi) {
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nwords = nbt >= 32 ? (nbt >> 5) : 1u;
    const uint32_t valid = nbt >= 32 ? 0xffffffffu : ((1u << nbt) - 1u);
    const uint32_t zeros = lane < nwords ? (~bm[lane] & valid) : 0u;
    const uint32_t have = __ballot_sync(0xffffffffu, zeros != 0);
    if (!have) {
        lo = 1;
        hi = 0;
        return;
    }
    const uint32_t wf = (uint32_t)__ffs(have) - 1u, wl = 31u - (uint32_t)__clz(have);
    const uint32_t zf = __shfl_sync(0xffffffffu, zeros, wf), zl = __shfl_sync(0xffffffffu, zeros, wl);
    lo = wf * 32u + (uint32_t)__ffs(zf) - 1u;
    hi = wl * 32u + 31u - (uint32_t)__clz(zl);
}

// The same for fine blocks (32 to 256 words of flags; lane l looks at words l, l + 32, ...).
__device__ __forceinline__ void unchanged_span_fine(const uint32_t* bm, uint32_t log2b, uint32_t lane, uint32_t& lo,
                                                    uint32_t& hi) {
    const uint32_t nwords = kTileValues >> (log2b + 5);
    uint32_t first = 0xffffffffu, last = 0;
    bool any = false;
    for (uint32_t w = lane; w < nwords; w += 32) {
        const uint32_t zeros = ~bm[w];
        if (zeros) {
            if (!any) first = w * 32u + (uint32_t)__ffs(zeros) - 1u;
            last = w * 32u + 31u - (uint32_t)__clz(zeros);
            any = true;
        }
    }
    if (!__any_sync(0xffffffffu, any)) {
        lo = 1;
        hi = 0;
        return;
    }
    lo = __reduce_min_sync(0xffffffffu, first);
    hi = __reduce_max_sync(0xffffffffu, last);
}

// Exponents of the changed blocks of one piece, fine blocks: `km` holds the piece's block flags,
// `src` points at the exponents of its first changed block; they replace the cached exponents in
// x.e value by value.  Only the first nvalid values exist.
// (fp16: a changed block's exponents lie five bits each in 1, 2, 3 or 5 bytes for 1, 2, 4 or 8 values; the piece's
// changed blocks take 8 bytes at most, read byte by byte -- never past the last block's bytes -- into one 64-bit
// word from which every value of a changed block picks its field.)
template <int DT, class M>
__device__ __forceinline__ void gather_changed(Piece<DT>& x, uint32_t km, uint32_t log2b, const uint8_t* src, int nvalid) {
    constexpr int kV = Piece<DT>::kValues;
    if constexpr (DT == CIERA_FP16) {
        const uint32_t B = 1u << log2b;
        const uint32_t block_bytes = (uint32_t)payload_bytes_of_blocks<DT>(1, log2b);
        // bytes of the piece's changed blocks (a short last block of the unit carries fewer)
        uint32_t nbytes = 0;
#pragma unroll
        for (int j = 0; j < kV; ++j) {
            if (j < (kV >> log2b) && ((km >> j) & 1u)) {
                const int len = min((int)B, nvalid - (j << log2b));
                nbytes += len > 0 ? (5u * (uint32_t)len + 7u) >> 3 : 0u;
            }
        }
        unsigned long long v = 0;
#pragma unroll
        for (uint32_t k = 0; k < 8u; ++k)
            if (k < nbytes) v |= (unsigned long long)M::ld1(src + k) << (8u * k);
#pragma unroll
        for (int i = 0; i < kV; ++i) {
            const uint32_t j = (uint32_t)i >> log2b;
            if (((km >> j) & 1u) && i < nvalid) {
                const uint32_t at = 8u * block_bytes * (uint32_t)__popc(km & ((1u << j) - 1u)) + 5u * ((uint32_t)i & (B - 1u));
                const uint32_t b = (uint32_t)(v >> at) & 31u;
                const uint32_t sel = (i & 3) == 0 ? 0x3214u : (i & 3) == 1 ? 0x3240u : (i & 3) == 2 ? 0x3410u : 0x4210u;
                x.e[i >> 2] = __byte_perm(x.e[i >> 2], b, sel);
            }
        }
        return;
    }
    if (nvalid == kV && log2b != 0) {
        // a complete piece of blocks of 2, 4 or 8 values: a changed block's exponents come with one load
        // (the payload holds whole blocks up to here, so `src` is a multiple of the block size)
        if (log2b == 3) {
#pragma unroll
            for (int j = 0; j < kV / 8; ++j) {
                if ((km >> j) & 1u) {
                    const uint2 v = M::ld8(src);
                    src += 8;
                    x.e[2 * j] = v.x;
                    x.e[2 * j + 1] = v.y;
                }
            }
        } else if (log2b == 2) {
#pragma unroll
            for (int j = 0; j < kV / 4; ++j) {
                if ((km >> j) & 1u) {
                    x.e[j] = M::ld4(src);
                    src += 4;
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < kV / 2; ++j) {
                if ((km >> j) & 1u) {
                    const uint32_t h = M::ld2(src);
                    src += 2;
                    x.e[j >> 1] = __byte_perm(x.e[j >> 1], h, (j & 1) ? 0x5410u : 0x3254u);
                }
            }
        }
        return;
    }
    uint32_t cnt = 0;
#pragma unroll
    for (int i = 0; i < Piece<DT>::kValues; ++i) {
        if ((km >> ((uint32_t)i >> log2b)) & 1u) {
            if (i < nvalid) {
                const uint32_t b = M::ld1(src + cnt);
                // byte (i & 3) of the word <- b
                const uint32_t sel = (i & 3) == 0 ? 0x3214u : (i & 3) == 1 ? 0x3240u : (i & 3) == 2 ? 0x3410u : 0x4210u;
                x.e[i >> 2] = __byte_perm(x.e[i >> 2], b, sel);
            }
            ++cnt;
        }
    }
}

// Bytes of one shared-memory stage: the tile's sign-plus-mantissa, the span of cached exponents
// (one byte per value), the payload slice (every block changed at most) and, where the slice need
// not start on a 16-byte boundary (fine blocks, fp16), 16 bytes of slack.  Used by the kernel and by
// the host when it sizes the dynamic shared memory.
template <int DT, bool FINE>
__host__ __device__ constexpr uint32_t decode_stage_bytes() {
    return (uint32_t)sm_bytes_of_values<DT>(kTileValues) + (uint32_t)kTileValues +
           (FINE ? (uint32_t)kTileValues : (uint32_t)payload_bytes_of_blocks<DT>(kTileValues >> 5, 5)) +
           ((FINE || DT == CIERA_FP16) ? 16u : 0u);
}

template <int DT, bool FINE>
__global__ void __launch_bounds__(kDecodeThreads, DecodeCfg<DT, FINE>::kBlocksPerSM)
decode_kernel(const TileDesc* __restrict__ tiles, uint32_t n_tiles, uint32_t log2b, const uint8_t* msgs, uint8_t* cache,
              uint8_t* __restrict__ weights, const unsigned long long* __restrict__ wire_bytes,
              const uint32_t* __restrict__ ws_prefix, unsigned int* ticket, int32_t* status) {
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;  // (not used for fp16)
    constexpr bool kHalf = DT == CIERA_FP16;    // packed sections: see Piece<CIERA_FP16>
    using Cfg = DecodeCfg<DT, FINE>;
    constexpr int S = Cfg::kStages;
    constexpr int kDecRing = Cfg::kRing;
    static_assert(S % kDecProducers == 0, "every producer cycles through stages of its own");
    static_assert(kDecRing > S + 2 * kDecProducers + 1, "a slot is refilled only after its tile is done");
    constexpr bool kStageOut = Cfg::kStageOut;
    constexpr uint32_t kSmTile = (uint32_t)sm_bytes_of_values<DT>(kTileValues);  // sign-plus-mantissa of a tile
    constexpr bool kSkew = FINE || kHalf;  // the payload slice need not start on a 16-byte boundary
    constexpr uint32_t kStageBytes = decode_stage_bytes<DT, FINE>();  // + cache span + payload slice
    constexpr uint32_t kOutBytes = kStageOut ? kTileValues * VB : 0u;  // reconstructed tile, staged for bulk stores
    constexpr uint32_t kWarpOutBytes = 32 * P::kValues * VB;           // one warp's contiguous slice of it
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* const s_out = smem + (size_t)S * kStageBytes;
    using Ring = DecodeRing<FINE>;
    using Ctl = DecodeCtl<S, kDecRing, FINE>;
    Ctl* ctl = reinterpret_cast<Ctl*>(s_out + kOutBytes);

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    volatile int* abort = &ctl->abort;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kWarps);
        }
        ctl->abort = 0;
        ctl->issued = 0;
        ctl->seen = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp >= kDecProducerWarp0) {
        // ---------------------------------------------------------------- producers (all lanes)
        // producer p fills the slots p, p + P, p + 2P, ... of the block's sequence (jj counts them),
        // each with the tile whose number it draws from the counter
        const uint32_t pidx = warp - kDecProducerWarp0;
        auto seq = [&](uint32_t jj) { return pidx + jj * kDecProducers; };  // place in the block's sequence
        auto draw = [&]() {
            uint32_t t = 0;
            if (lane == 0) t = atomicAdd(ticket, 1u);
            t = __shfl_sync(0xffffffffu, t, 0);
            return t < n_tiles ? t : kNoTile;
        };
        // software pipeline through the ring: tile number and descriptor two slots ahead, bitmap
        // words one slot ahead, both by per-thread asynchronous copies (groups D_j and B_j, committed
        // in the order D_0 D_1 B_0 | D_2 B_1 | D_3 B_2 | ...)
        auto fetch_desc = [&](uint32_t jj, uint32_t tile) {
            Ring* r = &ctl->ring[seq(jj) % kDecRing];
            if (lane == 0) r->tile = tile;
            if (tile != kNoTile && lane < 3)
                cp_async16(reinterpret_cast<uint8_t*>(&r->desc) + 16u * lane,
                           reinterpret_cast<const uint8_t*>(tiles + tile) + 16u * lane);
            cp_async_commit();
        };
        uint32_t t_cur = draw(), t_nxt = draw();
        fetch_desc(0, t_cur);
        fetch_desc(1, t_nxt);
        cp_async_wait<1>();  // D_0
        __syncwarp();
        if (t_cur != kNoTile)
            fetch_bitmap(ctl->ring[seq(0) % kDecRing].desc, t_cur, log2b, msgs, ws_prefix, &ctl->ring[seq(0) % kDecRing], lane);
        cp_async_commit();
        for (uint32_t jj = 0;; ++jj) {
            const uint32_t k = seq(jj);
            const uint32_t stage = k % S;
            // make sure the slot two ahead is free before refilling it: its previous tile is done once
            // the stage of slot k is free (slots are used in order, the ring is longer than that)
            bool ok = true;
            if (k >= (uint32_t)S) ok = mbar_wait(&ctl->empty[stage], ((k / S) & 1u) ^ 1u, abort, status);
            if (!__all_sync(0xffffffffu, ok)) break;
            if (t_cur == kNoTile) {  // no work left: tell the consumers and stop
                if (lane == 0) mbar_arrive(&ctl->full[stage]);
                break;
            }
            const uint32_t t_nn = t_nxt != kNoTile ? draw() : kNoTile;
            fetch_desc(jj + 2u, t_nn);
            cp_async_wait<1>();  // everything but D_{jj+2}: D_{jj+1} and B_jj have landed
            __syncwarp();
            if (t_nxt != kNoTile) {
                Ring* rn = &ctl->ring[seq(jj + 1u) % kDecRing];
                fetch_bitmap(rn->desc, t_nxt, log2b, msgs, ws_prefix, rn, lane);
            }
            cp_async_commit();

            Ring* r = &ctl->ring[k % kDecRing];
            const TileDesc td = r->desc;
            uint32_t own = 0;
            const uint64_t before = digest_bitmap(r, td, log2b, lane, own);
            const uint64_t N = td.n_unit;
            const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
            const uint64_t smoff = sm_offset(N, log2b);
            const uint64_t payoff = smoff + pad16(sm_section_bytes(N, DT));
            const uint8_t* msg = msgs + td.msg_off;
            const uint64_t pay_before = payload_bytes_of_blocks<DT>(before, log2b);
            const uint8_t* pay = msg + payoff + pay_before;  // this tile's slice of the payload
            uint8_t* st = smem + (size_t)stage * kStageBytes;
            const bool full_tile = N - v0 >= (uint64_t)kTileValues;
            uint32_t lo = 1, hi = 0;
            if (full_tile) {
                if (FINE)
                    unchanged_span_fine(r->bm, log2b, lane, lo, hi);
                else
                    unchanged_span(r->bm, log2b, lane, lo, hi);
            }
            // Coarse blocks (not fp32, whose output goes through bulk stores and which lost 6 % with it): the
            // cached exponents of the unchanged blocks come run by run -- lane w looks at word w of the block
            // flags and starts one bulk copy per run of unchanged blocks in it -- unless the runs are many
            // (then the one span that covers them, or, where they are few and far apart, reads by the consumers).
            bool by_runs = false;
            uint32_t my_zeros = 0, unchanged_bytes = 0;
            if (!FINE && !kStageOut && full_tile) {
                const uint32_t nbt_ = (uint32_t)kTileValues >> log2b;
                const uint32_t nwords = nbt_ >= 32u ? nbt_ >> 5 : 1u;
                if (lane < nwords) my_zeros = ~r->bm[lane] & (nbt_ >= 32u ? 0xffffffffu : (1u << nbt_) - 1u);
                const uint32_t nruns = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(my_zeros & ~(my_zeros << 1)));
                const uint32_t unchanged = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(my_zeros));
                unchanged_bytes = unchanged << log2b;
                const uint32_t span_bytes = lo <= hi ? (hi - lo + 1u) << log2b : 0u;
                const bool sparse = span_bytes != 0 && 4u * unchanged_bytes <= span_bytes;  // consumers read them
                // (fp16 with more than 32 blocks per tile: the span was faster.  Runs of less than 512 bytes on
                // average -- 32 values per block with two thirds of the blocks of a changed segment changed: copies of
                // 32 to 64 bytes -- cost more than the bytes they save: 0.295 against 0.266 ms per layer with the span;
                // a limit of 1024 bytes starts to cost with 64 values per block.)
                by_runs = !sparse && nruns <= 32u && (!kHalf || nbt_ <= 32u) && unchanged_bytes >= nruns * 512u;
            }

            if (lane == 0) {
                r->w_dst = weights + td.w_off;
                r->c_ptr = cache + td.c_off;
                r->sm_src = msg + smoff + sm_bytes_of_values<DT>(v0);
                r->pay_src = pay;
                r->nv = (uint32_t)min((uint64_t)kTileValues, N - v0);

                // integrity check by the unit's last tile: the bitmap fixes the message length
                if (wire_bytes != nullptr && status != nullptr && td.tile_in_unit == td.n_tiles_unit - 1u) {
                    const uint32_t B = 1u << log2b;
                    const uint32_t nv = (uint32_t)(N - v0);
                    uint64_t total = payload_bytes_of_blocks<DT>(before + own, log2b);
                    const uint32_t rem = nv & (B - 1u);
                    if (rem) {  // a changed short last block carries fewer bytes
                        const uint32_t kb = nv >> log2b;
                        if ((r->bm[kb >> 5] >> (kb & 31u)) & 1u)
                            total -= block_payload_bytes(B, DT) - block_payload_bytes(rem, DT);
                    }
                    if (wire_bytes[td.unit] != payoff + total) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
                }

                if (full_tile) {
                    // bulk copies move whole 16-byte pieces: with fine blocks the span of cached
                    // exponents and the payload slice are widened to such boundaries (the tile's
                    // cache is 16-byte aligned; the slice stays inside the unit's payload section,
                    // which holds at least the values up to the end of this full tile)
                    uint32_t span0 = lo << log2b, span = lo <= hi ? (hi - lo + 1u) << log2b : 0u;
                    uint32_t skew = 0, slice = (uint32_t)payload_bytes_of_blocks<DT>(own, log2b);
                    if (by_runs) {
                        span = unchanged_bytes;  // no cached exponents of changed blocks are read
                        if (!kHalf) r->direct = 0u;
                    } else if (!FINE && !kHalf) {
                        // a few unchanged blocks scattered over a long span: staging the span would mostly
                        // move cached exponents that the payload replaces anyway
                        const uint32_t unchanged = (uint32_t)kTileValues - (own << log2b);
                        const bool direct = span != 0 && 4u * unchanged <= span;
                        r->direct = direct ? 1u : 0u;
                        if (direct) span = 0;
                    }
                    if (FINE && span) {
                        const uint32_t end = (span0 + span + 15u) & ~15u;
                        span0 &= ~15u;
                        span = end - span0;
                    }
                    if (kSkew) {
                        if (slice) {
                            skew = (uint32_t)(pay_before & 15ull);
                            slice = (skew + slice + 15u) & ~15u;
                        }
                        r->pay_skew = skew;
                    }
                    mbar_arrive_expect_tx(&ctl->full[stage], kSmTile + span + slice);
                    bulk_load(st, r->sm_src, kSmTile, &ctl->full[stage]);
                    // (by_runs: the copies of the runs are started by the warp's lanes, one run each, below)
                    if (!by_runs && span) bulk_load(st + kSmTile + span0, r->c_ptr + span0, span, &ctl->full[stage]);
                    if (slice) bulk_load(st + kSmTile + kTileValues, pay - skew, slice, &ctl->full[stage]);
                } else {
                    mbar_arrive(&ctl->full[stage]);  // short tile: consumers read global memory themselves
                }
            }
            __syncwarp();
            if (by_runs) {
                // (the bytes of all runs are already part of what lane 0 told the barrier to expect)
                uint32_t zeros = my_zeros;
                while (zeros) {
                    const uint32_t s0 = (uint32_t)__ffs(zeros) - 1u;
                    const uint32_t ones = ~(zeros >> s0);  // first set bit = the run's length (none: to bit 31)
                    const uint32_t len = ones ? (uint32_t)__ffs(ones) - 1u : 32u - s0;
                    const uint32_t at = (32u * lane + s0) << log2b;
                    bulk_load(st + kSmTile + at, r->c_ptr + at, len << log2b, &ctl->full[stage]);
                    zeros &= ~((len == 32u ? 0xffffffffu : (1u << len) - 1u) << s0);
                }
                __syncwarp();
            }
            if (lane == 0) atomicMax(&ctl->issued, k + 1u);
            t_cur = t_nxt;
            t_nxt = t_nn;
        }
        cp_async_wait<0>();
        // this producer draws no more numbers: the last producer of the grid to get here hands the counter (and
        // the count of producers that got here, in the word behind it) back at zero for the next call
        if (lane == 0) {
            __threadfence();
            if (atomicAdd(ticket + 1, 1u) + 1u == gridDim.x * (uint32_t)kDecProducers) {
                __threadfence();
                ticket[0] = 0u;
                ticket[1] = 0u;
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers
        const uint32_t bmask = (1u << log2b) - 1u;
        uint32_t live = (1u << kDecProducers) - 1u;  // producers that have not sent their end marker
        for (uint32_t k = 0; live != 0; ++k) {
            if (!((live >> (k % kDecProducers)) & 1u)) continue;  // that producer's slots are over
            const uint32_t stage = k % S;
            if (!mbar_wait(&ctl->full[stage], (k / S) & 1u, abort, status)) break;
            if (tid == 0) ctl->seen = k + 1;
            const Ring* r = &ctl->ring[k % kDecRing];
            if (r->tile == kNoTile) {
                live &= ~(1u << (k % kDecProducers));
                continue;
            }
            const uint32_t nv = r->nv;
            const uint8_t* const st = smem + (size_t)stage * kStageBytes;
            uint8_t* const c_ptr = r->c_ptr;
            uint8_t* const w_dst = r->w_dst;

            if (nv == (uint32_t)kTileValues) {
                if (kStageOut) {
                    if (lane == 0) bulk_wait_read<0>();  // the warp's previous bulk store has been read out
                    __syncwarp();
                }
#pragma unroll
                for (int p = 0; p < P::kPerThread; ++p) {
                    const uint32_t t0 = P::start(tid, p);
                    const uint32_t kb = t0 >> log2b;
                    const uint32_t word = r->bm[kb >> 5];
                    // exponents: the cached ones, or -- changed block -- the ones that came in the payload
                    const uint32_t rank = r->pre[kb >> 5] + __popc(word & ((1u << (kb & 31u)) - 1u));
                    P x;
                    bool chg;
                    if constexpr (kHalf && FINE) {
                        // 11 packed bytes of sign-plus-mantissa; the piece's flags pick, block by block
                        x.template load_sm_group<Shared>(st, t0 >> 3, lane);
                        const uint32_t km = (word >> (kb & 31u)) & ((1u << (P::kValues >> log2b)) - 1u);
                        chg = km != 0;
                        x.template load_exp_full<Shared>(st + kSmTile + t0);
                        if (chg)
                            gather_changed<DT, Shared>(x, km, log2b,
                                                       st + kSmTile + kTileValues + r->pay_skew +
                                                           (size_t)payload_bytes_of_blocks<DT>(rank, log2b),
                                                       P::kValues);
                    } else if constexpr (kHalf) {
                        // 11 packed bytes of sign-plus-mantissa; 5 packed bytes of exponents if the block changed
                        x.template load_sm_group<Shared>(st, t0 >> 3, lane);
                        chg = (word >> (kb & 31u)) & 1u;
                        if (chg)
                            x.template load_packed_exponents<Shared>(
                                st + kSmTile + kTileValues + r->pay_skew + (size_t)payload_bytes_of_blocks<DT>(rank, log2b) +
                                    5u * ((t0 & bmask) >> 3),
                                P::kValues);
                        else
                            x.template load_exp_full<Shared>(st + kSmTile + t0);
                    } else if (!FINE) {
                        x.template load_sm_full<Shared>(st + (size_t)t0 * SMB);
                        chg = (word >> (kb & 31u)) & 1u;
                        const uint8_t* esrc = chg ? st + kSmTile + kTileValues + ((size_t)rank << log2b) + (t0 & bmask)
                                                  : st + kSmTile + t0;
                        if (!chg && r->direct)
                            x.template load_exp_full<Global>(c_ptr + t0);
                        else
                            x.template load_exp_full<Shared>(esrc);
                    } else {
                        // the piece's flags (they never straddle a word) pick, block by block
                        x.template load_sm_full<Shared>(st + (size_t)t0 * SMB);
                        const uint32_t km = (word >> (kb & 31u)) & ((1u << (P::kValues >> log2b)) - 1u);
                        chg = km != 0;
                        x.template load_exp_full<Shared>(st + kSmTile + t0);
                        if (chg)
                            gather_changed<DT, Shared>(x, km, log2b,
                                                       st + kSmTile + kTileValues + r->pay_skew + ((size_t)rank << log2b),
                                                       P::kValues);
                    }
                    if (chg) x.template store_exp_full<Global>(c_ptr + t0);  // ExpCache[i,k] <- newExp[j]
                    if (kStageOut)
                        x.template merge_store_full<Shared>(s_out + (size_t)t0 * VB);
                    else
                        x.template merge_store_full<Global>(w_dst + (size_t)t0 * VB);
                }
                if (kStageOut) fence_async_shared();
                __syncwarp();  // every lane has used what it read from the stage (and staged its output)
                if (lane == 0) {
                    mbar_arrive(&ctl->empty[stage]);
                    if (kStageOut) {
                        // the warp's weights are contiguous: one bulk store, coalesced by the copy engine
                        bulk_store(w_dst + (size_t)warp * kWarpOutBytes, s_out + (size_t)warp * kWarpOutBytes, kWarpOutBytes);
                        bulk_commit();
                    }
                }
            } else {
                // short tile: straight from global memory
                const uint8_t* const sm_src = r->sm_src;
                const uint8_t* const pay_src = r->pay_src;
#pragma unroll
                for (int p = 0; p < P::kPerThread; ++p) {
                    const uint32_t t0 = P::start(tid, p);
                    const int nvalid = piece_valid<DT>(t0, nv);
                    if (nvalid == 0) continue;
                    const uint32_t kb = t0 >> log2b;
                    const uint32_t word = r->bm[kb >> 5];
                    const uint32_t rank = r->pre[kb >> 5] + __popc(word & ((1u << (kb & 31u)) - 1u));
                    // coarse: the piece's block; fine: the piece's blocks, picked one by one below
                    const uint32_t km = FINE ? (word >> (kb & 31u)) & ((1u << (P::kValues >> log2b)) - 1u)
                                             : (word >> (kb & 31u)) & 1u;
                    const bool chg = km != 0;
                    const uint8_t* esrc = (chg && !FINE) ? pay_src + ((size_t)rank << log2b) + (t0 & bmask) : c_ptr + t0;
                    P x;
                    if constexpr (kHalf && FINE) {
                        x.load_sm_bytes(sm_src + (size_t)11 * (t0 >> 3), nvalid);
                        x.load_exp_partial(c_ptr + t0, nvalid);
                        if (chg) {
                            gather_changed<DT, Global>(x, km, log2b, pay_src + (size_t)payload_bytes_of_blocks<DT>(rank, log2b),
                                                       nvalid);
                            x.store_exp_partial(c_ptr + t0, nvalid);
                        }
                        if (nvalid == P::kValues)
                            x.template merge_store_full<Global>(w_dst + (size_t)t0 * VB);
                        else
                            x.merge_store_partial(w_dst + (size_t)t0 * VB, nvalid);
                    } else if constexpr (kHalf) {
                        x.load_sm_bytes(sm_src + (size_t)11 * (t0 >> 3), nvalid);
                        if (chg) {
                            x.template load_packed_exponents<Global>(
                                pay_src + (size_t)payload_bytes_of_blocks<DT>(rank, log2b) + 5u * ((t0 & bmask) >> 3), nvalid);
                            x.store_exp_partial(c_ptr + t0, nvalid);
                        } else {
                            x.load_exp_partial(c_ptr + t0, nvalid);
                        }
                        if (nvalid == P::kValues)
                            x.template merge_store_full<Global>(w_dst + (size_t)t0 * VB);
                        else
                            x.merge_store_partial(w_dst + (size_t)t0 * VB, nvalid);
                    } else if (nvalid == P::kValues) {
                        x.template load_sm_full<Global>(sm_src + (size_t)t0 * SMB);
                        x.template load_exp_full<Global>(esrc);
                        if (FINE && chg) gather_changed<DT, Global>(x, km, log2b, pay_src + ((size_t)rank << log2b), nvalid);
                        if (chg) x.template store_exp_full<Global>(c_ptr + t0);
                        x.template merge_store_full<Global>(w_dst + (size_t)t0 * VB);
                    } else {
                        x.load_sm_partial(sm_src + (size_t)t0 * SMB, nvalid);
                        x.load_exp_partial(esrc, nvalid);
                        if (FINE && chg) gather_changed<DT, Global>(x, km, log2b, pay_src + ((size_t)rank << log2b), nvalid);
                        if (chg) x.store_exp_partial(c_ptr + t0, nvalid);
                        x.merge_store_partial(w_dst + (size_t)t0 * VB, nvalid);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->empty[stage]);
            }
        }
    }

    // bulk stores of this thread (lane 0 of the consumer warps) are complete before the block ends
    if (kStageOut) bulk_wait_all<0>();
    // leave together; after an aborted run wait (bounded) for bulk copies that are still in flight
    __syncthreads();
    if (tid == 0 && ctl->abort) {
        for (uint32_t k = ctl->seen; k < ctl->issued; ++k) {
            for (uint32_t i = 0; i < kMaxBarrierPolls; ++i)
                if (mbar_try_wait(&ctl->full[k % S], (k / S) & 1u)) break;
        }
    }
}

// Changed blocks before every tile of the long units (more than kDirectBlocks blocks): one thread
// block per long unit, a running count over the unit's tiles in chunks of 256.
__global__ void __launch_bounds__(256)
decode_prefix_kernel(const TileDesc* __restrict__ tiles, const uint32_t* __restrict__ long_first_tiles, uint32_t log2b,
                     const uint8_t* __restrict__ msgs, uint32_t* __restrict__ ws_prefix) {
    __shared__ uint32_t s_warp[8];
    __shared__ uint32_t s_carry;
    const uint32_t first = long_first_tiles[blockIdx.x];
    const TileDesc td0 = load_tile_desc(tiles + first);
    const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msgs + td0.msg_off);
    const uint64_t nb = num_blocks(td0.n_unit, log2b);
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (uint32_t j0 = 0; j0 < td0.n_tiles_unit; j0 += 256u) {
        const uint32_t j = j0 + tid;
        uint32_t cnt = 0;
        if (j < td0.n_tiles_unit) {
            const uint64_t kb0 = (uint64_t)j * nbt;
            if (nbt >= 32) {
                for (uint32_t w = 0; w < (nbt >> 5); ++w) {
                    const uint64_t b0 = kb0 + 32ull * w;
                    if (b0 >= nb) break;
                    uint32_t word = __ldg(bm32 + (b0 >> 5));
                    if (nb - b0 < 32) word &= (1u << (uint32_t)(nb - b0)) - 1u;
                    cnt += __popc(word);
                }
            } else {
                const uint32_t left = (uint32_t)min((uint64_t)nbt, nb - kb0);
                cnt = __popc((__ldg(bm32 + (kb0 >> 5)) >> (kb0 & 31u)) & ((1u << left) - 1u));
            }
        }
        // exclusive scan over the 256 tiles of this chunk
        uint32_t incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += t;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        uint32_t wbase = 0;
        for (uint32_t w = 0; w < warp; ++w) wbase += s_warp[w];
        const uint32_t carry = s_carry;
        if (j < td0.n_tiles_unit) ws_prefix[first + j] = carry + wbase + incl - cnt;
        __syncthreads();
        if (tid == 255) s_carry = carry + wbase + incl;
        __syncthreads();
    }
}

// The same for fine blocks, where every unit of more than one tile comes here and a tile has 32 to
// 256 words of flags: the warps take the unit's tiles in turn and each counts a tile's flags with
// all its lanes (consecutive words, coalesced), then the counts are scanned as above.
__global__ void __launch_bounds__(256)
decode_prefix_fine_kernel(const TileDesc* __restrict__ tiles, const uint32_t* __restrict__ long_first_tiles,
                          uint32_t log2b, const uint8_t* __restrict__ msgs, uint32_t* __restrict__ ws_prefix) {
    __shared__ uint32_t s_cnt[256];
    __shared__ uint32_t s_warp[8];
    __shared__ uint32_t s_carry;
    const uint32_t first = long_first_tiles[blockIdx.x];
    const TileDesc td0 = load_tile_desc(tiles + first);
    const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msgs + td0.msg_off);
    const uint64_t nb = num_blocks(td0.n_unit, log2b);
    const uint32_t words = kTileValues >> (log2b + 5);  // words of flags per tile
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (uint32_t j0 = 0; j0 < td0.n_tiles_unit; j0 += 256u) {
        for (uint32_t t = warp; t < 256u && j0 + t < td0.n_tiles_unit; t += 8u) {
            const uint64_t w0 = (uint64_t)(j0 + t) * words;
            uint32_t c = 0;
            for (uint32_t m = lane; m < words; m += 32u) {
                const uint64_t b0 = (w0 + m) << 5;
                if (b0 < nb) {
                    uint32_t word = __ldg(bm32 + w0 + m);
                    if (nb - b0 < 32) word &= (1u << (uint32_t)(nb - b0)) - 1u;
                    c += __popc(word);
                }
            }
            c = __reduce_add_sync(0xffffffffu, c);
            if (lane == 0) s_cnt[t] = c;
        }
        __syncthreads();
        const uint32_t j = j0 + tid;
        const uint32_t cnt = j < td0.n_tiles_unit ? s_cnt[tid] : 0u;
        uint32_t incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += v;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        uint32_t wbase = 0;
        for (uint32_t w = 0; w < warp; ++w) wbase += s_warp[w];
        const uint32_t carry = s_carry;
        if (j < td0.n_tiles_unit) ws_prefix[first + j] = carry + wbase + incl - cnt;
        __syncthreads();
        if (tid == 255) s_carry = carry + wbase + incl;
        __syncthreads();
    }
}

template <int DT, bool FINE>
static size_t decode_smem_bytes() {
    using Cfg = DecodeCfg<DT, FINE>;
    constexpr int S = Cfg::kStages;
    const size_t stage = decode_stage_bytes<DT, FINE>();
    const size_t out = Cfg::kStageOut ? (size_t)kTileValues * Traits<DT>::kValueBytes : 0;
    return (size_t)S * stage + out + sizeof(DecodeCtl<S, Cfg::kRing, FINE>);
}

template <int DT, bool FINE>
static int decode_grid_limit(int* out) {
    static std::atomic<int> cached[64];  // (zero-initialised; any host thread may be the first to fill an entry)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    if (cached[dev].load(std::memory_order_acquire) == 0) {
        const size_t smem = decode_smem_bytes<DT, FINE>();
        e = cudaFuncSetAttribute(decode_kernel<DT, FINE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        int per_sm = 0, sms = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_kernel<DT, FINE>, kDecodeThreads, smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (per_sm < 1 || sms < 1) return CIERA_ERR_UNSUPPORTED;
        cached[dev].store(per_sm * sms, std::memory_order_release);
    }
    *out = cached[dev].load(std::memory_order_acquire);
    return CIERA_OK;
}

template <int DT, bool FINE>
static int launch_decode(const ciera_plan* p, const void* messages_dev, void* receiver_cache_dev, void* weights_out_dev,
                         const uint64_t* wire_bytes_dev, const uint32_t* ws_prefix, unsigned int* ticket, int32_t* status_dev,
                         cudaStream_t s) {
    int limit = 0;
    const int rc = decode_grid_limit<DT, FINE>(&limit);
    if (rc) return rc;
    const uint32_t nt = (uint32_t)p->tiles.size();
    const uint32_t grid = nt < (uint32_t)limit ? nt : (uint32_t)limit;
    decode_kernel<DT, FINE><<<grid, kDecodeThreads, decode_smem_bytes<DT, FINE>(), s>>>(
        p->tiles_dev, nt, p->log2b, (const uint8_t*)messages_dev, (uint8_t*)receiver_cache_dev, (uint8_t*)weights_out_dev,
        (const unsigned long long*)wire_bytes_dev, ws_prefix, ticket, status_dev);
    count_launch();
    return check_launch();
}

}  // namespace ciera

using namespace ciera;

static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

extern "C" int ciera_decode(const ciera_plan* p, const void* messages_dev, void* receiver_cache_dev,
                            void* weights_out_dev, const uint64_t* wire_bytes_dev, void* workspace_dev,
                            int32_t* status_dev, void* stream) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    if (!messages_dev || !receiver_cache_dev || !weights_out_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(receiver_cache_dev) || misaligned16(weights_out_dev) ||
        misaligned16(workspace_dev))
        return CIERA_ERR_MISALIGNED;
    cudaStream_t s = (cudaStream_t)stream;
    // scratch: the tile counter (found at zero, handed back at zero) behind the sender's status words (left
    // alone), and behind it the per-tile counts of the units that go through the prefix kernel
    unsigned int* ticket = (unsigned int*)((uint8_t*)workspace_dev + workspace_ticket_offset(nt));
    uint32_t* ws_prefix = (uint32_t*)((uint8_t*)workspace_dev + workspace_prefix_offset(nt));
    const uint32_t n_long = (uint32_t)p->long_units.size();
    if (n_long) {
        if (is_fine(p->log2b))
            decode_prefix_fine_kernel<<<n_long, 256, 0, s>>>(p->tiles_dev, p->long_units_dev, p->log2b,
                                                             (const uint8_t*)messages_dev, ws_prefix);
        else
            decode_prefix_kernel<<<n_long, 256, 0, s>>>(p->tiles_dev, p->long_units_dev, p->log2b,
                                                        (const uint8_t*)messages_dev, ws_prefix);
        count_launch();
        int rc = check_launch();
        if (rc) return rc;
    }
    const bool fine = is_fine(p->log2b);
    if (p->dtype == CIERA_FP16)
        return fine ? launch_decode<CIERA_FP16, true>(p, messages_dev, receiver_cache_dev, weights_out_dev, wire_bytes_dev,
                                                      ws_prefix, ticket, status_dev, s)
                    : launch_decode<CIERA_FP16, false>(p, messages_dev, receiver_cache_dev, weights_out_dev, wire_bytes_dev,
                                                       ws_prefix, ticket, status_dev, s);
    if (p->dtype == CIERA_BF16)
        return fine ? launch_decode<CIERA_BF16, true>(p, messages_dev, receiver_cache_dev, weights_out_dev, wire_bytes_dev,
                                                      ws_prefix, ticket, status_dev, s)
                    : launch_decode<CIERA_BF16, false>(p, messages_dev, receiver_cache_dev, weights_out_dev, wire_bytes_dev,
                                                       ws_prefix, ticket, status_dev, s);
    return fine ? launch_decode<CIERA_FP32, true>(p, messages_dev, receiver_cache_dev, weights_out_dev, wire_bytes_dev,
                                                  ws_prefix, ticket, status_dev, s)
                : launch_decode<CIERA_FP32, false>(p, messages_dev, receiver_cache_dev, weights_out_dev, wire_bytes_dev,
                                                   ws_prefix, ticket, status_dev, s);
}
