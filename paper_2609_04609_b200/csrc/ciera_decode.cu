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
#include "ciera_bits.cuh"
#include "ciera_pipe.cuh"

namespace ciera {

constexpr int kDecProducers = 2;                               // producer warps, taking tiles in turn
constexpr int kDecodeThreads = kThreads + 32 * kDecProducers;  // consumers + producers
constexpr int kDecProducerWarp0 = kWarps;
constexpr int kDecRing = 12;  // > stages + 2 * producers + 1: slots are refilled only after their tile is done
constexpr uint32_t kNoTile = 0xffffffffu;
constexpr uint32_t kDirectWordsPerLane = 4;
constexpr uint32_t kDirectBlocks = kDecodeDirectBlocks;
static_assert(kDirectBlocks == 32u * 32u * kDirectWordsPerLane, "one fetch covers the direct range");

template <int DT>
struct DecodeCfg;
template <>
struct DecodeCfg<CIERA_BF16> {
    static constexpr int kStages = 4;        // 4 x (8 KB sm + 8 KB cache span + 8 KB payload slice)
    static constexpr int kBlocksPerSM = 2;
    static constexpr bool kStageOut = false;  // weights leave as 16 B / lane, contiguous per warp
};
template <>
struct DecodeCfg<CIERA_FP32> {
    static constexpr int kStages = 4;        // 4 x (24 KB sm + 8 KB + 8 KB)
    static constexpr int kBlocksPerSM = 1;
    static constexpr bool kStageOut = true;   // 64 B / lane: staged, then one bulk store per warp
};

// Per-tile bookkeeping, in a ring that the producers fill ahead of the consumers.
struct __align__(16) DecodeRing {
    TileDesc desc;                           // copied from the plan's table (asynchronously)
    // worked out once by a producer for the 512 consumer threads:
    uint8_t* w_dst;                          // where the tile's reconstructed weights go
    uint8_t* c_ptr;                          // the tile's cached exponents
    const uint8_t* sm_src;                   // the tile's received sign-plus-mantissa
    const uint8_t* pay_src;                  // the payload slice holding the tile's changed blocks
    uint32_t nv;                             // values in the tile
    uint32_t tile;                           // the tile's number, or kNoTile: this producer has no more work
    uint32_t bm[kBitmapWords];               // the tile's block flags
    uint32_t pre[kBitmapWords];              // set flags before each word
    // raw material, fetched asynchronously one tile ahead:
    uint32_t raw_pre[32 * kDirectWordsPerLane];  // bitmap words before the tile
    uint32_t raw_own[kBitmapWords];              // words holding the tile's own bits
    uint32_t ws;                                 // count from the scratch (long units)
};

template <int S>
struct DecodeCtl {
    uint64_t full[S];   // stage filled (producer arrive + bulk-copy bytes)
    uint64_t empty[S];  // all 16 consumer warps have read it
    DecodeRing ring[kDecRing];
    int abort;
    uint32_t issued;
    uint32_t seen;
};

// Starts the asynchronous fetch of the bitmap words a producer needs for one tile into the ring
// slot `r`: the unit's words before the tile (direct units) or the tile's count from the scratch
// (long units), and the tile's own words.  Nothing is held in registers meanwhile.
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
__device__ __forceinline__ uint64_t digest_bitmap(DecodeRing* r, const TileDesc& td, uint32_t log2b, uint32_t lane,
                                                  uint32_t& own_total) {
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
        r->pre[lane] = incl - pc;
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

template <int DT>
__global__ void __launch_bounds__(kDecodeThreads, DecodeCfg<DT>::kBlocksPerSM)
decode_kernel(const TileDesc* __restrict__ tiles, uint32_t n_tiles, uint32_t log2b, const uint8_t* msgs, uint8_t* cache,
              uint8_t* __restrict__ weights, const unsigned long long* __restrict__ wire_bytes,
              const uint32_t* __restrict__ ws_prefix, unsigned int* ticket, int32_t* status) {
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;
    constexpr int S = DecodeCfg<DT>::kStages;
    static_assert(S % kDecProducers == 0, "every producer cycles through stages of its own");
    constexpr bool kStageOut = DecodeCfg<DT>::kStageOut;
    constexpr uint32_t kSmTile = kTileValues * SMB;                   // sign-plus-mantissa of a tile
    constexpr uint32_t kStageBytes = kSmTile + 2u * kTileValues;       // + cache span + payload slice
    constexpr uint32_t kOutBytes = kStageOut ? kTileValues * VB : 0u;  // reconstructed tile, staged for bulk stores
    constexpr uint32_t kWarpOutBytes = 32 * P::kValues * VB;           // one warp's contiguous slice of it
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* const s_out = smem + (size_t)S * kStageBytes;
    DecodeCtl<S>* ctl = reinterpret_cast<DecodeCtl<S>*>(s_out + kOutBytes);

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
            DecodeRing* r = &ctl->ring[seq(jj) % kDecRing];
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
                DecodeRing* rn = &ctl->ring[seq(jj + 1u) % kDecRing];
                fetch_bitmap(rn->desc, t_nxt, log2b, msgs, ws_prefix, rn, lane);
            }
            cp_async_commit();

            DecodeRing* r = &ctl->ring[k % kDecRing];
            const TileDesc td = r->desc;
            uint32_t own = 0;
            const uint64_t before = digest_bitmap(r, td, log2b, lane, own);
            const uint64_t N = td.n_unit;
            const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
            const uint64_t smoff = sm_offset(N, log2b);
            const uint64_t payoff = smoff + pad16(N * SMB);
            const uint8_t* msg = msgs + td.msg_off;
            const uint8_t* pay = msg + payoff + (before << log2b);  // this tile's slice of the payload
            uint8_t* st = smem + (size_t)stage * kStageBytes;
            const bool full_tile = N - v0 >= (uint64_t)kTileValues;
            uint32_t lo = 1, hi = 0;
            if (full_tile) unchanged_span(r->bm, log2b, lane, lo, hi);

            if (lane == 0) {
                r->w_dst = weights + td.w_off;
                r->c_ptr = cache + td.c_off;
                r->sm_src = msg + smoff + v0 * SMB;
                r->pay_src = pay;
                r->nv = (uint32_t)min((uint64_t)kTileValues, N - v0);

                // integrity check by the unit's last tile: the bitmap fixes the message length
                if (wire_bytes != nullptr && status != nullptr && td.tile_in_unit == td.n_tiles_unit - 1u) {
                    const uint32_t B = 1u << log2b;
                    const uint32_t nv = (uint32_t)(N - v0);
                    uint64_t total = (before + own) << log2b;
                    const uint32_t rem = nv & (B - 1u);
                    if (rem) {
                        const uint32_t kb = nv >> log2b;
                        if ((r->bm[kb >> 5] >> (kb & 31u)) & 1u) total -= (B - rem);
                    }
                    if (wire_bytes[td.unit] != payoff + total) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
                }

                if (full_tile) {
                    const uint32_t span = lo <= hi ? (hi - lo + 1u) << log2b : 0u;
                    const uint32_t slice = own << log2b;
                    mbar_arrive_expect_tx(&ctl->full[stage], kSmTile + span + slice);
                    bulk_load(st, r->sm_src, kSmTile, &ctl->full[stage]);
                    if (span)
                        bulk_load(st + kSmTile + ((size_t)lo << log2b), r->c_ptr + ((size_t)lo << log2b), span,
                                  &ctl->full[stage]);
                    if (slice) bulk_load(st + kSmTile + kTileValues, pay, slice, &ctl->full[stage]);
                } else {
                    mbar_arrive(&ctl->full[stage]);  // short tile: consumers read global memory themselves
                }
                atomicMax(&ctl->issued, k + 1u);
            }
            __syncwarp();
            t_cur = t_nxt;
            t_nxt = t_nn;
        }
        cp_async_wait<0>();
    } else {
        // ---------------------------------------------------------------- consumers
        const uint32_t bmask = (1u << log2b) - 1u;
        uint32_t live = (1u << kDecProducers) - 1u;  // producers that have not sent their end marker
        for (uint32_t k = 0; live != 0; ++k) {
            if (!((live >> (k % kDecProducers)) & 1u)) continue;  // that producer's slots are over
            const uint32_t stage = k % S;
            if (!mbar_wait(&ctl->full[stage], (k / S) & 1u, abort, status)) break;
            if (tid == 0) ctl->seen = k + 1;
            const DecodeRing* r = &ctl->ring[k % kDecRing];
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
                    const bool chg = (word >> (kb & 31u)) & 1u;
                    // exponents: the cached ones, or -- changed block -- the ones that came in the payload
                    const uint32_t rank = r->pre[kb >> 5] + __popc(word & ((1u << (kb & 31u)) - 1u));
                    const uint8_t* esrc = chg ? st + kSmTile + kTileValues + ((size_t)rank << log2b) + (t0 & bmask)
                                              : st + kSmTile + t0;
                    P x;
                    x.template load_sm_full<Shared>(st + (size_t)t0 * SMB);
                    x.template load_exp_full<Shared>(esrc);
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
                    const bool chg = (word >> (kb & 31u)) & 1u;
                    const uint32_t rank = r->pre[kb >> 5] + __popc(word & ((1u << (kb & 31u)) - 1u));
                    const uint8_t* esrc = chg ? pay_src + ((size_t)rank << log2b) + (t0 & bmask) : c_ptr + t0;
                    P x;
                    if (nvalid == P::kValues) {
                        x.template load_sm_full<Global>(sm_src + (size_t)t0 * SMB);
                        x.template load_exp_full<Global>(esrc);
                        if (chg) x.template store_exp_full<Global>(c_ptr + t0);
                        x.template merge_store_full<Global>(w_dst + (size_t)t0 * VB);
                    } else {
                        x.load_sm_partial(sm_src + (size_t)t0 * SMB, nvalid);
                        x.load_exp_partial(esrc, nvalid);
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

template <int DT>
static size_t decode_smem_bytes() {
    constexpr int S = DecodeCfg<DT>::kStages;
    const size_t stage = (size_t)kTileValues * Traits<DT>::kSmBytes + 2u * kTileValues;
    const size_t out = DecodeCfg<DT>::kStageOut ? (size_t)kTileValues * Traits<DT>::kValueBytes : 0;
    return (size_t)S * stage + out + sizeof(DecodeCtl<S>);
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
    if (!messages_dev || !receiver_cache_dev || !weights_out_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(receiver_cache_dev) || misaligned16(weights_out_dev) ||
        misaligned16(workspace_dev))
        return CIERA_ERR_MISALIGNED;
    cudaStream_t s = (cudaStream_t)stream;
    // scratch = per-tile counts for long units (4 bytes per tile), then, past 8 bytes per tile, the
    // tile counter, which starts at zero
    unsigned int* ticket = (unsigned int*)((unsigned long long*)workspace_dev + nt);
    cudaError_t me = cudaMemsetAsync(ticket, 0, 16, s);
    if (me != cudaSuccess) return record_cuda_error(me);
    const uint32_t n_long = (uint32_t)p->long_units.size();
    if (n_long) {
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
            (uint8_t*)weights_out_dev, (const unsigned long long*)wire_bytes_dev, (const uint32_t*)workspace_dev, ticket,
            status_dev);
    else
        decode_kernel<CIERA_FP32><<<grid, kDecodeThreads, decode_smem_bytes<CIERA_FP32>(), s>>>(
            p->tiles_dev, nt, p->log2b, (const uint8_t*)messages_dev, (uint8_t*)receiver_cache_dev,
            (uint8_t*)weights_out_dev, (const unsigned long long*)wire_bytes_dev, (const uint32_t*)workspace_dev, ticket,
            status_dev);
    count_launch();
    return check_launch();
}
