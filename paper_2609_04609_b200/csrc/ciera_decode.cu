// Receiver side (paper Algorithm 1, receiver part; Section 3.1) as one persistent sm_100a kernel.
//
// Grid = at most as many thread blocks as fit on the GPU; block c works on tiles c, c + G, ...
// Tiles are independent here, so no block ever waits for another.  Two roles:
//
//   producer warp   runs ahead: for each tile it reads the tile's bits of the unit's bitmap and the
//                   number of changed blocks before the tile, then assembles the tile's inputs in a
//                   shared-memory stage with bulk-async copies: the received sign-plus-mantissa
//                   tile, and the tile's exponents -- every run of unchanged blocks from the
//                   receiver's cache, every run of changed blocks from the message payload;
//   16 consumer     each thread merges 16 exponent bytes and 16 sign-plus-mantissa values from the
//   warps           stage into 16 weights and stores them; threads of changed blocks also store
//                   the new exponents to the cache (ExpCache[i,k] <- newExp[j]).
//
// The number of changed blocks before a tile is the popcount of the bitmap bits before it.  For
// units of up to kDirectBlocks blocks the producer takes it straight from the bitmap (at most four
// words per lane, fetched one tile ahead); longer units get it from a small prefix kernel that
// runs first and writes one count per tile into the caller's scratch.
#include "ciera_bits.cuh"
#include "ciera_pipe.cuh"

CIERA_PROF_READER(dec)

namespace ciera {

constexpr int kDecProducers = 2;                             // producer warps, taking tiles in turn
constexpr int kDecodeThreads = kThreads + 32 * kDecProducers;  // consumers + producers
constexpr int kDecProducerWarp0 = kWarps;
constexpr int kDecDescRing = 16;  // > stages + 2 * producers + 1: slots are refilled only after their tile is done
constexpr uint32_t kDirectWordsPerLane = 4;
constexpr uint32_t kDirectBlocks = kDecodeDirectBlocks;
static_assert(kDirectBlocks == 32u * 32u * kDirectWordsPerLane, "one fetch covers the direct range");

template <int DT>
struct DecodeCfg;
template <>
struct DecodeCfg<CIERA_BF16> {
    static constexpr int kStages = 5;  // 5 x (8 KB sm + 8 KB exponents)
};
template <>
struct DecodeCfg<CIERA_FP32> {
    static constexpr int kStages = 2;  // 2 x (24 KB sm + 8 KB exponents)
};

// Per-tile bookkeeping, in a ring that the producers fill ahead of the consumers.
struct __align__(16) DecodeRing {
    TileDesc desc;                                  // copied from the plan's table (asynchronously)
    // worked out once by a producer for the 512 consumer threads:
    uint8_t* w_dst;                                 // where the tile's reconstructed weights go
    uint8_t* c_ptr;                                 // the tile's cached exponents
    const uint8_t* sm_src;                          // the tile's received sign-plus-mantissa
    const uint8_t* pay_src;                         // start of the unit's payload section
    unsigned long long before;                      // changed blocks of the unit before the tile
    uint32_t nv;                                    // values in the tile
    uint32_t pad;
    uint32_t pre[32 * kDirectWordsPerLane];         // raw bitmap words before the tile
    uint32_t own[kBitmapWords];                     // raw words holding the tile's own bits
    uint32_t ws;                                    // count from the scratch (long units)
    uint32_t bm[kBitmapWords];                      // digested: the tile's block flags
};

template <int S>
struct DecodeCtl {
    uint64_t full[S];   // stage assembled (producer arrive + bulk-copy bytes)
    uint64_t empty[S];  // all 16 consumer warps have read it
    DecodeRing ring[kDecDescRing];
    int abort;
    uint32_t issued;
    uint32_t seen;
};

// Starts the asynchronous fetch of the bitmap words the producer needs for one tile into the
// ring slot `r`: the unit's words before the tile (direct units) or the tile's count from the
// scratch (long units), and the tile's own words.  Nothing is held in registers meanwhile.
__device__ __forceinline__ void fetch_bitmap(const TileDesc& td, uint32_t tile, uint32_t log2b, const uint8_t* msgs,
                                             const uint32_t* ws_prefix, DecodeRing* r, uint32_t lane) {
    const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msgs + td.msg_off);
    const uint64_t kb0 = ((uint64_t)td.tile_in_unit * kTileValues) >> log2b;  // first block of the tile
    const uint64_t nb = num_blocks(td.n_unit, log2b);
    const uint32_t nbt = kTileValues >> log2b;
    if (nb <= kDirectBlocks) {
        const uint32_t nwords = (uint32_t)((kb0 + 31) >> 5);  // words holding bits before kb0
#pragma unroll
        for (uint32_t i = 0; i < kDirectWordsPerLane; ++i) {
            const uint32_t w = lane + 32u * i;
            if (w < nwords) cp_async4(&r->pre[w], bm32 + w);
        }
    } else if (lane == 0) {
        cp_async4(&r->ws, ws_prefix + tile);
    }
    // the tile's own bits: nbt >= 32 -> words (kb0 >> 5) + lane; nbt < 32 -> part of one word
    const uint32_t own_words = nbt >= 32 ? (nbt >> 5) : 1u;
    if (lane < own_words) {
        const uint64_t w = (kb0 >> 5) + lane;
        if ((w << 5) < nb) cp_async4(&r->own[lane], bm32 + w);  // never past the bitmap's padded end
    }
}

// Turns a completed fetch into (changed blocks before the tile, the tile's block flags in r->bm).
__device__ __forceinline__ uint64_t digest_bitmap(DecodeRing* r, const TileDesc& td, uint32_t log2b, uint32_t lane) {
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint64_t kb0 = v0 >> log2b;
    const uint64_t nb = num_blocks(td.n_unit, log2b);
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const uint32_t nblk = (nv + (1u << log2b) - 1u) >> log2b;  // valid blocks of this tile
    uint32_t cnt = 0;
    if (nb <= kDirectBlocks) {
        const uint32_t nfull = (uint32_t)(kb0 >> 5);
#pragma unroll
        for (uint32_t i = 0; i < kDirectWordsPerLane; ++i) {
            const uint32_t w = lane + 32u * i;
            if (w < nfull)
                cnt += __popc(r->pre[w]);
            else if (w == nfull && (kb0 & 31u))
                cnt += __popc(r->pre[w] & ((1u << (kb0 & 31u)) - 1u));
        }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
    } else {
        cnt = r->ws;
    }
    uint32_t word = 0;
    if (nbt >= 32) {
        if (lane < (nbt >> 5) && lane * 32u < nblk) {
            word = r->own[lane];
            const uint32_t left = nblk - lane * 32u;
            if (left < 32u) word &= (1u << left) - 1u;
        }
    } else if (lane == 0) {
        word = (r->own[0] >> (kb0 & 31u)) & ((1u << nblk) - 1u);
    }
    if (lane < kBitmapWords) r->bm[lane] = word;
    __syncwarp();
    return cnt;
}

// Starts the bulk copies that assemble the exponent tile of a FULL tile: runs of unchanged blocks
// come from the cache, runs of changed blocks from the payload.  All 32 lanes take part; every
// lane owns the blocks lane, lane + 32, ... of each 32-block word.  Total bytes = kTileValues.
__device__ __forceinline__ void assemble_exponents(uint8_t* s_exp, const uint8_t* cache_tile, const uint8_t* payload,
                                                   uint64_t before, const uint32_t* bm, uint32_t log2b, uint64_t* bar,
                                                   uint32_t lane) {
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nwords = nbt >= 32 ? (nbt >> 5) : 1u;
    const uint32_t per = nbt >= 32 ? 32u : nbt;  // blocks per word
    uint32_t rank0 = 0;                          // changed blocks of the tile before this word
    for (uint32_t w = 0; w < nwords; ++w) {
        const uint32_t bits = bm[w];
        if (lane < per) {
            // a run starts at block 0 of the word and wherever a bit differs from its predecessor
            const uint32_t starts = (bits ^ (bits << 1)) | 1u;
            if ((starts >> lane) & 1u) {
                const uint32_t later = per == 32u ? starts >> 1 >> lane : (starts & ((1u << per) - 1u)) >> 1 >> lane;
                const uint32_t len = later ? (uint32_t)__ffs(later) : per - lane;  // blocks in the run
                const uint32_t blk = w * 32u + lane;                                // block index in the tile
                const bool chg = (bits >> lane) & 1u;
                const uint32_t rank = rank0 + __popc(bits & ((1u << lane) - 1u));
                const uint8_t* src = chg ? payload + ((before + rank) << log2b) : cache_tile + ((uint64_t)blk << log2b);
                bulk_load(s_exp + ((size_t)blk << log2b), src, len << log2b, bar);
            }
        }
        rank0 += __popc(bits);
    }
}

template <int DT>
__global__ void __launch_bounds__(kDecodeThreads, 2)
decode_kernel(const TileDesc* __restrict__ tiles, uint32_t n_tiles, uint32_t log2b, const uint8_t* msgs, uint8_t* cache,
              uint8_t* __restrict__ weights, const unsigned long long* __restrict__ wire_bytes,
              const uint32_t* __restrict__ ws_prefix, int32_t* status) {
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;
    constexpr int S = DecodeCfg<DT>::kStages;
    constexpr uint32_t kSmBytesTile = kTileValues * SMB;
    constexpr uint32_t kStageBytes = kSmBytesTile + kTileValues;
    constexpr uint32_t kOutBytes = kTileValues * VB;       // reconstructed tile, staged for bulk stores
    constexpr uint32_t kWarpOutBytes = 32 * kVPT * VB;     // one warp's contiguous slice of it
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* const s_out = smem + (size_t)S * kStageBytes;
    DecodeCtl<S>* ctl = reinterpret_cast<DecodeCtl<S>*>(s_out + kOutBytes);

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t G = gridDim.x;
    const uint32_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + G - 1u) / G : 0u;
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
        // producer p handles this block's tiles p, p + P, p + 2P, ... (index k below counts them)
        const uint32_t pidx = warp - kDecProducerWarp0;
        const uint32_t my_prod = my_tiles > pidx ? (my_tiles - pidx + kDecProducers - 1u) / kDecProducers : 0u;
        if (my_prod > 0) {
            // software pipeline through the ring: descriptor two tiles ahead, bitmap words one tile
            // ahead, both by per-thread asynchronous copies (groups D_j and B_j, committed in the
            // order D_0 D_1 B_0 | D_2 B_1 | D_3 B_2 | ...)
            // jj counts this producer's tiles; seq(jj) is the tile's place in the block's sequence
            auto seq = [&](uint32_t jj) { return pidx + jj * kDecProducers; };
            auto fetch_desc = [&](uint32_t jj) {
                if (jj < my_prod && lane < 3)
                    cp_async16(reinterpret_cast<uint8_t*>(&ctl->ring[seq(jj) % kDecDescRing].desc) + 16u * lane,
                               reinterpret_cast<const uint8_t*>(tiles + blockIdx.x + (uint64_t)seq(jj) * G) + 16u * lane);
                cp_async_commit();
            };
            fetch_desc(0);
            fetch_desc(1);
            cp_async_wait<1>();  // D_0
            __syncwarp();
            fetch_bitmap(ctl->ring[seq(0) % kDecDescRing].desc, blockIdx.x + seq(0) * G, log2b, msgs, ws_prefix,
                         &ctl->ring[seq(0) % kDecDescRing], lane);
            cp_async_commit();
            PROF_T0;
            for (uint32_t jj = 0; jj < my_prod; ++jj) {
                const uint32_t k = seq(jj);
                fetch_desc(jj + 2u);
                cp_async_wait<1>();  // everything but D_{jj+2}: D_{jj+1} and B_jj have landed
                PROF_ADD(0);
                __syncwarp();
                if (jj + 1u < my_prod) {
                    DecodeRing* rn = &ctl->ring[seq(jj + 1u) % kDecDescRing];
                    fetch_bitmap(rn->desc, blockIdx.x + seq(jj + 1u) * G, log2b, msgs, ws_prefix, rn, lane);
                }
                cp_async_commit();
                PROF_ADD(1);

                const uint32_t stage = k % S;
                bool ok = true;
                if (k >= (uint32_t)S) ok = mbar_wait(&ctl->empty[stage], ((k / S) & 1u) ^ 1u, abort, status);
                if (!__all_sync(0xffffffffu, ok)) break;
                PROF_ADD(2);

                DecodeRing* r = &ctl->ring[k % kDecDescRing];
                const TileDesc td = r->desc;
                const uint64_t before = digest_bitmap(r, td, log2b, lane);
                const uint64_t N = td.n_unit;
                const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
                const uint64_t smoff = sm_offset(N, log2b);
                const uint64_t payoff = smoff + pad16(N * SMB);
                const uint8_t* msg = msgs + td.msg_off;
                uint8_t* st = smem + (size_t)stage * kStageBytes;
                if (lane == 0) {
                    r->w_dst = weights + td.w_off;
                    r->c_ptr = cache + td.c_off;
                    r->sm_src = msg + smoff + v0 * SMB;
                    r->pay_src = msg + payoff;
                    r->before = before;
                    r->nv = (uint32_t)min((uint64_t)kTileValues, N - v0);
                }
                PROF_ADD(6);

                // integrity check by the unit's last tile: the bitmap fixes the message length
                if (wire_bytes != nullptr && status != nullptr && td.tile_in_unit == td.n_tiles_unit - 1u) {
                    uint32_t own = lane < kBitmapWords ? __popc(r->bm[lane]) : 0u;
                    own = __reduce_add_sync(0xffffffffu, own);
                    const uint32_t B = 1u << log2b;
                    const uint32_t nv = (uint32_t)(N - v0);
                    uint64_t total = (before + own) << log2b;
                    const uint32_t rem = nv & (B - 1u);
                    if (rem) {
                        const uint32_t kb = nv >> log2b;
                        if ((r->bm[kb >> 5] >> (kb & 31u)) & 1u) total -= (B - rem);
                    }
                    if (lane == 0 && wire_bytes[td.unit] != payoff + total)
                        atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
                }

                PROF_ADD(7);
                if (N - v0 >= (uint64_t)kTileValues) {
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&ctl->full[stage], kStageBytes);
                        bulk_load(st, msg + smoff + v0 * SMB, kSmBytesTile, &ctl->full[stage]);
                    }
                    __syncwarp();
                    PROF_ADD(8);
                    assemble_exponents(st + kSmBytesTile, cache + td.c_off, msg + payoff, before, r->bm, log2b,
                                       &ctl->full[stage], lane);
                } else {
                    // short tile: consumers read global memory themselves
                    if (lane == 0) mbar_arrive(&ctl->full[stage]);
                }
                if (lane == 0) atomicMax(&ctl->issued, k + 1u);
                PROF_ADD(3);
            }
            PROF_FLUSH;
            cp_async_wait<0>();
        }
    } else {
        // ---------------------------------------------------------------- consumers
        const uint32_t t0 = tid * kVPT;
        PROF_T0;
        for (uint32_t k = 0; k < my_tiles; ++k) {
            const uint32_t stage = k % S;
            if (!mbar_wait(&ctl->full[stage], (k / S) & 1u, abort, status)) break;
            PROF_ADD(4);
            if (tid == 0) ctl->seen = k + 1;
            const DecodeRing* r = &ctl->ring[k % kDecDescRing];
            const uint32_t nv = r->nv;
            const int nvalid = t0 >= nv ? 0 : (int)min(16u, nv - t0);
            const uint8_t* st = smem + (size_t)stage * kStageBytes;
            const uint32_t kb = t0 >> log2b;
            const uint32_t word = r->bm[kb >> 5];
            const bool chg = nvalid > 0 && ((word >> (kb & 31u)) & 1u);
            uint8_t* cptr = r->c_ptr + t0;
            uint8_t* const w_dst = r->w_dst;
            uint8_t* wptr = w_dst + (size_t)t0 * VB;

            Group<DT> g;
            if (nv == (uint32_t)kTileValues) {
                g.load_sm_full(st + (size_t)t0 * SMB, FromShared());
                const uint4 ev = ld_shared16(st + kSmBytesTile + t0);
                g.e[0] = ev.x; g.e[1] = ev.y; g.e[2] = ev.z; g.e[3] = ev.w;
                if (chg) st_stream16(cptr, ev);  // ExpCache[i,k] <- newExp[j]
                // the warp's 32 x 16 weights are contiguous: stage them and send them with one
                // bulk store (fully coalesced by the copy engine, no store instructions per lane)
                if (lane == 0) bulk_wait_read<0>();  // the slice's previous bulk store has been read out
                __syncwarp();
                g.merge_store_full(s_out + (size_t)t0 * VB, ToShared());
                fence_async_shared();
                __syncwarp();  // every lane has used what it read from the stage and written its part
                if (lane == 0) {
                    mbar_arrive(&ctl->empty[stage]);
                    bulk_store(w_dst + (size_t)warp * kWarpOutBytes, s_out + (size_t)warp * kWarpOutBytes, kWarpOutBytes);
                    bulk_commit();
                }
                PROF_ADD(5);
            } else {
                const unsigned long long before = r->before;
                const uint8_t* smsrc = r->sm_src + (size_t)t0 * SMB;
                const uint8_t* paysrc = r->pay_src;
                uint32_t rank = __popc(word & ((1u << (kb & 31u)) - 1u));
                for (uint32_t w = 0; w < (kb >> 5); ++w) rank += __popc(r->bm[w]);
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                if (nvalid > 0) {
                    const uint8_t* src = cptr;  // unchanged block: the cached exponents
                    if (chg)                    // changed block: its exponents are in the payload
                        src = paysrc + ((before + rank) << log2b) + (t0 & ((1u << log2b) - 1u));
                    if (nvalid == 16) {
                        g.load_sm_full(smsrc);
                        const uint4 ev = ld_stream16(src);
                        g.e[0] = ev.x; g.e[1] = ev.y; g.e[2] = ev.z; g.e[3] = ev.w;
                        if (chg) st_stream16(cptr, ev);
                        g.merge_store_full(wptr);
                    } else {
                        g.load_sm_partial(smsrc, nvalid);
                        load_exp_partial(g.e, src, nvalid);
                        if (chg) store_exp_partial(cptr, g.e, nvalid);
                        g.merge_store_partial(wptr, nvalid);
                    }
                }
            }
        }
        if (warp == 0) PROF_FLUSH;
    }

    // bulk stores of this thread (lane 0 of the consumer warps) are complete before the block ends
    bulk_wait_all<0>();
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

template <int DT>
static size_t decode_smem_bytes() {
    constexpr int S = DecodeCfg<DT>::kStages;
    return (size_t)S * (kTileValues * Traits<DT>::kSmBytes + kTileValues) + (size_t)kTileValues * Traits<DT>::kValueBytes +
           sizeof(DecodeCtl<S>);
}

template <int DT>
static int decode_grid_limit(int* out) {
    static int cached[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    if (cached[dev] == 0) {
        const size_t smem = decode_smem_bytes<DT>();
        e = cudaFuncSetAttribute(decode_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        int per_sm = 0, sms = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_kernel<DT>, kDecodeThreads, smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (per_sm < 1 || sms < 1) return CIERA_ERR_UNSUPPORTED;
        cached[dev] = per_sm * sms;
    }
    *out = cached[dev];
    return CIERA_OK;
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
    if (!messages_dev || !receiver_cache_dev || !weights_out_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(receiver_cache_dev) || misaligned16(weights_out_dev) ||
        misaligned16(workspace_dev))
        return CIERA_ERR_MISALIGNED;
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t n_long = (uint32_t)p->long_units.size();
    if (n_long) {
        if (!workspace_dev) return CIERA_ERR_INVALID_ARG;
        decode_prefix_kernel<<<n_long, 256, 0, s>>>(p->tiles_dev, p->long_units_dev, p->log2b,
                                                    (const uint8_t*)messages_dev, (uint32_t*)workspace_dev);
        count_launch();
        int rc = check_launch();
        if (rc) return rc;
    }
    int limit = 0;
    int rc = p->dtype == CIERA_BF16 ? decode_grid_limit<CIERA_BF16>(&limit) : decode_grid_limit<CIERA_FP32>(&limit);
    if (rc) return rc;
    const uint32_t grid = nt < (uint32_t)limit ? nt : (uint32_t)limit;
    if (p->dtype == CIERA_BF16)
        decode_kernel<CIERA_BF16><<<grid, kDecodeThreads, decode_smem_bytes<CIERA_BF16>(), s>>>(
            p->tiles_dev, nt, p->log2b, (const uint8_t*)messages_dev, (uint8_t*)receiver_cache_dev,
            (uint8_t*)weights_out_dev, (const unsigned long long*)wire_bytes_dev, (const uint32_t*)workspace_dev,
            status_dev);
    else
        decode_kernel<CIERA_FP32><<<grid, kDecodeThreads, decode_smem_bytes<CIERA_FP32>(), s>>>(
            p->tiles_dev, nt, p->log2b, (const uint8_t*)messages_dev, (uint8_t*)receiver_cache_dev,
            (uint8_t*)weights_out_dev, (const unsigned long long*)wire_bytes_dev, (const uint32_t*)workspace_dev,
            status_dev);
    count_launch();
    return check_launch();
}
