// Sender side (paper Algorithm 1, sender part; Section 3.1) as one persistent sm_100a kernel.
//
// Grid = G persistent thread blocks.  The plan lists the tiles of short units (up to 32 tiles)
// first.  A block first takes its share of the tiles of the longer units, spread tile by tile over
// the blocks (block c takes tiles T0 + c, T0 + c + G, ...; neighbouring tiles of a unit are then
// worked on by neighbouring blocks at about the same time, and their payload offsets come from a
// single-pass look-back over per-tile status words; this part needs all blocks resident, so a
// plan with longer units is launched cooperatively).  Then it works through the short units in runs
// of four tiles, drawing the next run's number from a counter in the scratch (every unit's first run
// goes out before any unit's second run, and so on): a tile's place in its unit's payload is then a
// running sum inside the block, which a run that does not start its unit takes over from the status
// word of the tile before it -- written many draws earlier -- and all SMs stay busy to the end
// whatever their individual pace (with whole units of 16 tiles as the piece of work drawn, the blocks
// finished up to a unit apart: 0.921 of the copy peak against 0.935).
// A thread block has four roles:
//
//   producer warp   runs ahead of the others: for each of its tiles it fetches the tile
//                   descriptor, works out the tile's addresses once for everybody, and starts two
//                   bulk-async copies into shared memory -- the weights tile into a short ring
//                   (freed as soon as the consumers have read it) and the cached-exponent tile
//                   into a longer ring (held until the tile's changed exponents have been sent);
//   16 consumer     each thread owns one or two pieces of consecutive values: split into exponent
//   warps           bytes and sign-plus-mantissa, compare with the cached exponents, vote (ballot)
//                   the "my piece changed" bit, store sign-plus-mantissa to the message and leave
//                   the new exponents where the cached ones were staged;
//   aggregator warp turns the vote bits of a tile into block flags (the unit's bitmap) and counts
//                   the tile's payload bytes; for a tile of a unit that this block works through
//                   alone it also keeps the running offset, otherwise it publishes the count as
//                   the tile's status word;
//   resolver warps  (spread tiles only) resolve the tile's exclusive offset in the unit's payload
//                   with a single-pass look-back over the status words.
// A few tiles later, when that offset is known, the consumers send the exponents of changed
// blocks from shared memory to the payload and to the cache and hand the stage back.
//
// Only the resolvers ever wait for another thread block; the aggregator never does, and the
// consumers only for a resolver that is several tiles late, so a tile's status is published as
// soon as its votes are in.
//
// The same kernel serves the sender that keeps HashCache (a 128-bit hash per block, Section 3.1 and
// Algorithm 1 as printed) instead of the previous exponents (template flag HASH): the producer then
// stages the tile's cached hashes instead of cached exponents, the consumers turn their exponents
// into hash terms and add them up over the lanes that share a block, and the aggregator finishes
// the hashes, compares them with the cached ones, refreshes HashCache and derives the block flags
// from the comparison.
#include <cstddef>
#include <type_traits>

#include "ciera_bits.cuh"
#include "ciera_hash.cuh"
#include "ciera_lookback.cuh"
#include "ciera_pipe.cuh"

namespace ciera {

constexpr int kResolvers = 2;  // resolver warps (20 warps per block: two blocks per SM at 48 registers per thread)
constexpr int kEncodeThreads = kThreads + 64 + 32 * kResolvers;  // consumers + producer + aggregator + resolvers
constexpr int kProducerWarp = kWarps;                            // 16
constexpr int kAggregatorWarp = kWarps + 1;                      // 17
constexpr int kResolverWarp0 = kWarps + 2;                       // 18 ..
constexpr int kDescRing = 16;                                    // > exponent stages + 2
constexpr int kVoteWords = 32;  // vote bits of a tile: up to 1024 pieces

// Ring depths; kDefer = consumers send a tile's changed exponents this many tiles later.  With
// fine blocks (see ciera_internal.cuh) a tile has up to 8192 block flags instead of 512, and the
// exponent ring gives up a stage to make room for them (two thread blocks share an SM).
template <int DT, bool FINE>
struct EncodeCfg;
template <>
struct EncodeCfg<CIERA_BF16, false> {
    static constexpr int kWStages = 3;  // 3 x 16 KB weights tiles
    static constexpr int kEStages = 7;  // 7 x  8 KB exponent tiles
    static constexpr int kDefer = 3;
    static constexpr int kBmWords = kBitmapWords;
};
template <>
struct EncodeCfg<CIERA_FP32, false> {
    static constexpr int kWStages = 2;  // 2 x 32 KB
    static constexpr int kEStages = 5;  // 5 x  8 KB
    static constexpr int kDefer = 3;
    static constexpr int kBmWords = kBitmapWords;
};
template <>
struct EncodeCfg<CIERA_FP16, false> {  // as bf16: 16 KB weights tiles, 8 KB exponent tiles
    static constexpr int kWStages = 3;
    static constexpr int kEStages = 7;
    static constexpr int kDefer = 3;
    static constexpr int kBmWords = kBitmapWords;
};
// (fine blocks: the exponent ring is shorter still, to make room for the warps' gather spaces; ring depths of
// 3 + 5 with the sending two tiles later measured the same as 3 + 7 and three tiles later on the headline)
template <>
struct EncodeCfg<CIERA_BF16, true> {
    static constexpr int kWStages = 3;
    static constexpr int kEStages = 5;
    static constexpr int kDefer = 2;
    static constexpr int kBmWords = kFineBitmapWords;
};
template <>
struct EncodeCfg<CIERA_FP16, true> : EncodeCfg<CIERA_BF16, true> {};  // the tile sizes of bf16
template <>
struct EncodeCfg<CIERA_FP32, true> {
    static constexpr int kWStages = 2;
    static constexpr int kEStages = 3;
    static constexpr int kDefer = 1;
    static constexpr int kBmWords = kFineBitmapWords;
};

// With HashCache the exponent ring stages no cached exponents (it only keeps the new ones until
// they are sent), so it is shorter; each of its stages has a companion with the tile's cached
// hashes and the consumers' partial sums, sized at launch from the block size.
// The template argument HASH of the kernel is 0 (exponent cache), 1 (HashCache), 2 (HashCache with
// shorter rings: with blocks of 64 values and fewer the hash stages are large, and two thread blocks
// still have to fit an SM) or 3 (as 2, and the consumers finish the blocks' hashes).
template <int DT, int HASH>
struct EncodeHashCfg;
template <>
struct EncodeHashCfg<CIERA_BF16, 1> {
    static constexpr int kWStages = 3;
    static constexpr int kEStages = 6;
    static constexpr int kDefer = 3;
    static constexpr int kBmWords = kBitmapWords;
};
template <>
struct EncodeHashCfg<CIERA_FP32, 1> {
    static constexpr int kWStages = 2;
    static constexpr int kEStages = 4;
    static constexpr int kDefer = 2;
    static constexpr int kBmWords = kBitmapWords;
};
template <>
struct EncodeHashCfg<CIERA_FP16, 1> : EncodeHashCfg<CIERA_BF16, 1> {};  // fp16: the tile sizes of bf16
template <>
struct EncodeHashCfg<CIERA_BF16, 2> {
    static constexpr int kWStages = 3;
    static constexpr int kEStages = 4;
    static constexpr int kDefer = 2;
    static constexpr int kBmWords = kBitmapWords;
};
template <>
struct EncodeHashCfg<CIERA_FP32, 2> {
    static constexpr int kWStages = 2;
    static constexpr int kEStages = 3;
    static constexpr int kDefer = 1;
    static constexpr int kBmWords = kBitmapWords;
};
template <>
struct EncodeHashCfg<CIERA_FP16, 2> : EncodeHashCfg<CIERA_BF16, 2> {};
template <int DT>
struct EncodeHashCfg<DT, 3> : EncodeHashCfg<DT, 2> {};
constexpr uint32_t kHashShortRingsLog2 = 6;  // blocks of up to 2^6 values take the shorter rings
// With 256 and more blocks in a tile (16 and 32 values per block) the consumers finish the blocks' hashes
// themselves: kernel instance HASH == 3 (see finish_hash_groups; blocks of at least two lanes' pieces).
constexpr uint32_t kHashByConsumersLog2 = 5;
template <int DT, bool FINE, int HASH>
struct EncodeCfgOf {
    using type = EncodeHashCfg<DT, HASH>;
};
template <int DT, bool FINE>
struct EncodeCfgOf<DT, FINE, 0> {
    using type = EncodeCfg<DT, FINE>;
};

// Shared-memory bytes of the cached hashes (`hold`) and of the partial sums (`part`) of one tile:
// 16 bytes per block, and 16 bytes per group of lanes that add up their terms (a block's lanes, at
// most a warp).
template <int DT>
__host__ __device__ constexpr uint32_t hash_hold_bytes(uint32_t log2b) {
    return (uint32_t)(kTileValues >> log2b) * 16u;
}
template <int DT>
__host__ __device__ constexpr uint32_t hash_part_bytes(uint32_t log2b) {
    const uint32_t nbt = (uint32_t)kTileValues >> log2b;
    const uint32_t warps = (uint32_t)kTileValues >> (5 + Piece<DT>::kLog2Values);  // warp-sized groups of pieces
    return (nbt > warps ? nbt : warps) * 16u;
}

// What the consumers need of a tile, worked out once by the producer thread instead of by each
// of the 512 consumer threads.
struct __align__(16) EncodeTileInfo {
    uint8_t* sm_dst;       // where the tile's sign-plus-mantissa goes
    uint8_t* pay_dst;      // start of the unit's payload section
    uint8_t* c_ptr;        // the tile's cached exponents (with HashCache: the cached hash of the tile's first block)
    const uint8_t* w_src;  // the tile's weights
    uint32_t nv;           // values in the tile
    uint32_t pad[3];
};

template <int SW, int SE, int BW>
struct EncodeCtl {
    uint64_t full_w[SW];    // weights tile landed
    uint64_t empty_w[SW];   // all 16 consumer warps have read it
    uint64_t full_e[SE];    // cached-exponent tile landed
    uint64_t voted[SE];     // all 16 consumer warps have left their exponents there and voted
    uint64_t summed[SE];    // aggregator has published the tile's status and block flags
    uint64_t resolved[SE];  // a resolver knows the tile's offset in the unit's payload
    uint64_t empty_e[SE];   // all 16 consumer warps have sent the tile's changed exponents
    TileDesc desc[kDescRing];
    EncodeTileInfo info[kDescRing];
    uint32_t tile_idx[kDescRing];  // table index of the tile in desc[]; kNoTile = end marker
    uint32_t seq[kDescRing];       // kSeq* bits: tile of a run that this block works through alone, first / last of the run
    uint32_t ballot[SE][kVoteWords];  // coarse blocks: "my piece differs" votes
    uint32_t bm[SE][BW];              // block flags of the tile (16-byte aligned: checked where the kernel starts)
    uint16_t pre[SE][BW];             // set flags before each word of bm
    unsigned long long agg[SE];
    unsigned long long base[SE];
    int abort;
    uint32_t issued;  // tiles whose loads have been started (producer)
    uint32_t seen;    // tiles whose loads the consumers have seen complete
};

constexpr uint32_t kNoTile = 0xffffffffu;

// How a tile relates to the run of tiles it was handed out with (a short unit's tiles go out in runs of
// kSeqRunTiles, see ciera_internal.cuh): bit 0 = the tile belongs to a run (else: a spread tile of a longer
// unit), bit 1 = first tile of its run, bit 2 = last tile of its run.
constexpr uint32_t kSeqTile = 1u, kSeqRunStart = 2u, kSeqRunEnd = 4u;

// The sequence of tiles of one thread block (see the head of this file); used by the producer.
// Runs of the short units: block b starts with runs b and b + G (no round trip to the counter stands between
// the start of the kernel and the first loads); every run taken is paid for with one draw from the counter, so
// the counter is drawn from exactly n_runs times in a launch, and the thread that makes the last draw puts it
// back to zero for the next launch.  The walk keeps two runs in hand besides the current one: the number of
// the run after next (its draw is on its way) and the table entry of the next run (its load is on its way), so
// that at the start of a run neither the counter nor the table is waited for.
struct TileWalk {
    const uint2* seq_runs;
    unsigned int* run_ticket;
    uint32_t n_tiles, n_runs, G;
    uint32_t tile, end;      // current run: next tile, one past its last tile
    uint2 next_range;        // the next run's tiles (valid if next_run < n_runs)
    uint32_t next_run;       // number of the next run
    uint32_t after_run;      // number of the run after that
    uint32_t spread_tile;    // next spread tile of this block
    bool spread;

    __device__ TileWalk(const uint2* runs, unsigned int* ticket, uint32_t nruns, uint32_t spread_first, uint32_t nt,
                        uint32_t grid, uint32_t block)
        : seq_runs(runs), run_ticket(ticket), n_tiles(nt), n_runs(nruns), G(grid), tile(0), end(0), spread(true) {
        spread_tile = spread_first + block;  // tiles of longer units start after the short units' tiles
        next_run = block;
        after_run = block + grid;
        next_range = make_uint2(0u, 0u);
        if (next_run < n_runs) next_range = __ldg(seq_runs + next_run);
    }
    __device__ uint32_t draw() {
        const uint32_t d = atomicAdd(run_ticket, 1u);
        if (d + 1u == n_runs) atomicExch(run_ticket, 0u);  // that was the launch's last draw
        return d + 2u * G;
    }
    // next tile, or kNoTile; `seq` gets the kSeq* bits of the tile
    __device__ uint32_t next(uint32_t& seq) {
        if (spread) {
            if (spread_tile < n_tiles) {
                seq = 0;
                const uint32_t t = spread_tile;
                spread_tile += G;
                return t;
            }
            spread = false;
        }
        seq = kSeqTile;
        while (tile == end) {
            if (next_run >= n_runs) return kNoTile;
            tile = next_range.x;
            end = next_range.y;
            next_run = after_run;
            if (next_run < n_runs) next_range = __ldg(seq_runs + next_run);
            after_run = draw();
            seq |= kSeqRunStart;
        }
        if (tile + 1u == end) seq |= kSeqRunEnd;
        return tile++;
    }
};

// Fine blocks: the consumers have written the block flags themselves; fills pre (set bits before
// each word) and returns the number of changed blocks of the tile (one warp).
// Lane l takes the W = nwords / 32 consecutive words l W .. l W + W - 1 (1, 2, 4 or 8), so that one scan over
// the lanes does for the whole tile.
template <int W>
__device__ __forceinline__ uint32_t scan_block_bitmap_w(const uint32_t* bm, uint16_t* pre, uint32_t lane) {
    uint32_t w[W];
    if constexpr (W >= 4) {
#pragma unroll
        for (int i = 0; i < W / 4; ++i) {
            const uint4 v = reinterpret_cast<const uint4*>(bm)[lane * (W / 4) + i];
            w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < W; ++i) w[i] = bm[lane * W + i];
    }
    uint32_t before[W], sum = 0;
#pragma unroll
    for (int i = 0; i < W; ++i) {
        before[i] = sum;
        sum += __popc(w[i]);
    }
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)lane >= o) incl += t;
    }
    const uint32_t base = incl - sum;
    if constexpr (W >= 2) {  // two 16-bit counts per store
        uint32_t* pre32 = reinterpret_cast<uint32_t*>(pre) + lane * (W / 2);
#pragma unroll
        for (int i = 0; i < W / 2; ++i) pre32[i] = (base + before[2 * i]) | ((base + before[2 * i + 1]) << 16);
    } else {
        pre[lane] = (uint16_t)base;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
    __syncwarp();
    return total;
}
__device__ __forceinline__ uint32_t scan_block_bitmap(const uint32_t* bm, uint16_t* pre, uint32_t log2b, uint32_t lane) {
    if (log2b == 0) return scan_block_bitmap_w<8>(bm, pre, lane);  // 256 words: eight per lane, one scan
    if (log2b == 1) return scan_block_bitmap_w<4>(bm, pre, lane);  // 128 words: four per lane
    const uint32_t nwords = kTileValues >> (log2b + 5);  // 32 .. 128: a scan per 32 words
    uint32_t run = 0;
    for (uint32_t base = 0; base < nwords; base += 32) {
        const uint32_t pc = __popc(bm[base + lane]);
        uint32_t incl = pc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += t;
        }
        pre[base + lane] = (uint16_t)(run + incl - pc);
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    __syncwarp();
    return run;
}

// Blocks whose hashes the consumers finish themselves (see finish_hash_groups; kernel instance HASH == 3): many
// per tile, and made of at least two lanes' pieces.
template <int DT>
__host__ __device__ __forceinline__ bool hash_finished_by_consumers(uint32_t log2b) {
    return log2b <= kHashByConsumersLog2 && log2b > (uint32_t)Piece<DT>::kLog2Values;
}

// Aggregator warp, one tile: block flags, the tile's bitmap bytes, the tile's payload byte count.
// With `publish` the count goes out at once as the tile's status word, so that later tiles never
// wait for it longer than for the votes themselves.  Waits for nothing outside the thread block.
// HashCache: block flags of a tile from the consumers' partial sums.  Lane i of a round takes one
// block: adds up the block's partial sums, finishes the two hashes, compares them with the cached
// pair and, where they differ, flags the block and stores the new pair (HashCache[i,k] <- h).
// Returns the number of flagged blocks (one warp).
template <int DT, bool BY_CONSUMERS>
__device__ __forceinline__ uint32_t hash_block_bitmap(const ulonglong2* part, const ulonglong2* hold, ulonglong2* hash_dst,
                                                      uint32_t* bm, uint16_t* pre, uint32_t log2b, uint32_t nv,
                                                      uint32_t lane) {
    constexpr uint32_t kGroupL2 = 5 + Piece<DT>::kLog2Values;  // log2(values of a warp's pieces)
    const uint32_t B = 1u << log2b;
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nblk = (nv + B - 1u) >> log2b;
    const uint32_t epb_l2 = log2b > kGroupL2 ? log2b - kGroupL2 : 0u;  // log2(partial sums per block)
    const uint8_t* const verdicts = reinterpret_cast<const uint8_t*>(part);
    // one block: true iff its hashes differ from the cached pair (which is then replaced)
    auto finish_block = [&](uint32_t i) -> bool {
        if (i >= nblk) return false;
        if (BY_CONSUMERS) return verdicts[i] != 0;  // finished, compared and stored by the consumers already
        uint64_t a = 0, b = 0;
        for (uint32_t e = 0; e < (1u << epb_l2); ++e) {
            const ulonglong2 v = part[(i << epb_l2) + e];
            a += v.x;
            b += v.y;
        }
        const ulonglong2 h = hash_finish(a, b, min(B, nv - (i << log2b)));
        const ulonglong2 old = hold[i];
        const bool f = h.x != old.x || h.y != old.y;
        if (f) hash_dst[i] = h;
        return f;
    };
    uint32_t run = 0;
    uint32_t base = 0;
    // two blocks per lane and round while there are 64 and more (their chains of multiplies overlap; four were slower)
    for (; base + 64 <= nbt; base += 64) {
        const bool f0 = finish_block(base + lane), f1 = finish_block(base + 32 + lane);
        const uint32_t w0 = __ballot_sync(0xffffffffu, f0), w1 = __ballot_sync(0xffffffffu, f1);
        if (lane == 0) {
            bm[base >> 5] = w0;
            pre[base >> 5] = (uint16_t)run;
            bm[(base >> 5) + 1] = w1;
            pre[(base >> 5) + 1] = (uint16_t)(run + __popc(w0));
        }
        run += __popc(w0) + __popc(w1);
    }
    for (; base < nbt; base += 32) {
        const uint32_t word = __ballot_sync(0xffffffffu, finish_block(base + lane));
        if (lane == 0) {
            bm[base >> 5] = word;
            pre[base >> 5] = (uint16_t)run;
        }
        run += __popc(word);
    }
    __syncwarp();
    return run;
}

// HashCache, consumers: adds up the pieces' sums of terms (a[p], b[p]: the two hashes' sums of piece
// p of this thread) over groups of 2^l2 neighbouring lanes -- the lanes whose pieces lie in one block,
// at most the warp -- and stores the group's totals as entry e0 (piece 0) and e1 (the thread's last
// piece) of `part`, two 64-bit words each.  Instead of one butterfly per sum, the first exchanges
// hand every lane fewer sums to carry on with (odd lanes keep the b's, even lanes the a's; then lanes
// with bit 1 set keep the second piece's): 6 shuffles of 64 bits for four sums over a warp, not 20.
template <int NP>
__device__ __forceinline__ void reduce_hash_terms(const uint64_t* a, const uint64_t* b, uint32_t l2, uint32_t e0, uint32_t e1,
                                                  uint64_t* part, uint32_t lane) {
    const bool odd = (lane & 1u) != 0;
    if (l2 == 0) {  // every lane a block of its own (NP = 1: a piece is a whole block at least)
        part[2 * e0] = a[0];
        part[2 * e0 + 1] = b[0];
        return;
    }
    uint64_t k0 = (odd ? b[0] : a[0]) + __shfl_xor_sync(0xffffffffu, odd ? a[0] : b[0], 1);
    if constexpr (NP == 1) {
#pragma unroll
        for (uint32_t o = 1; o < 5; ++o)
            if (o < l2) k0 += __shfl_xor_sync(0xffffffffu, k0, 1u << o);
        const uint32_t r = lane & ((1u << l2) - 1u);
        if (r < 2) part[2 * e0 + r] = k0;  // lane 0 of the group: sum of a, lane 1: sum of b
    } else {
        uint64_t k1 = (odd ? b[1] : a[1]) + __shfl_xor_sync(0xffffffffu, odd ? a[1] : b[1], 1);
        if (l2 == 1) {  // groups of two lanes
            part[2 * e0 + (odd ? 1u : 0u)] = k0;
            part[2 * e1 + (odd ? 1u : 0u)] = k1;
            return;
        }
        const bool second = (lane & 2u) != 0;
        uint64_t t = (second ? k1 : k0) + __shfl_xor_sync(0xffffffffu, second ? k0 : k1, 2);
#pragma unroll
        for (uint32_t o = 2; o < 5; ++o)
            if (o < l2) t += __shfl_xor_sync(0xffffffffu, t, 1u << o);
        const uint32_t r = lane & ((1u << l2) - 1u);
        if (r < 4) part[2 * ((r & 2u) ? e1 : e0) + (r & 1u)] = t;  // lanes 0..3: a of piece 0, b of piece 0, a, b of piece 1
    }
}

// HashCache, consumers, kernel instance HASH == 3 (blocks that lie inside one warp's pieces and span at least two
// lanes, l2 >= 1): the same reduction as reduce_hash_terms, but the lanes that end up with a block's sums
// finish the block themselves -- each finishes one 64-bit half, compares it with its cached half, and the two
// halves of a block (in neighbouring lanes) agree on the verdict with one exchange; a changed block's new hash
// goes to HashCache at once (HashCache[i,k] <- h), and one byte per block tells the aggregator the verdict.
// With 256 or 512 blocks in a tile the one aggregator warp, finishing them all by itself, set the pace of the
// whole thread block (0.82 ms per layer with 32 values per block, 1.24 ms with 16, whatever the change rate);
// with fewer blocks per tile the extra work in the consumers costs more than it saves (measured), so those
// keep the aggregator's way.
//   hold   the tile's cached hashes (two words per block), staged in shared memory
//   dst    the same in global memory
//   flags  one byte per block of the tile (written for every block below nblk)
template <int DT, int NP>
__device__ __forceinline__ void finish_hash_groups(const uint64_t* a, const uint64_t* b, uint32_t l2, uint32_t log2b,
                                                   uint32_t nv, uint32_t tid, const uint64_t* hold, uint64_t* dst,
                                                   uint8_t* flags, uint32_t lane) {
    using P = Piece<DT>;
    const bool odd = (lane & 1u) != 0;
    const uint32_t B = 1u << log2b;
    // One half of one block: `t` = the sum of the half's terms over the block (held by `leader` lanes, the half is
    // the lane's parity), `piece` = which of the thread's pieces lies in that block.  Called by all lanes together.
    auto finish_half = [&](uint64_t t, int piece, bool leader) {
        const uint32_t blk = P::start(tid, piece) >> log2b;
        const uint32_t first = blk << log2b;
        const bool mine = leader && first < nv;
        uint64_t h = 0;
        uint32_t differs = 0;
        if (mine) {
            h = mix64(t + min(B, nv - first));
            differs = h != hold[2u * blk + (odd ? 1u : 0u)] ? 1u : 0u;
        }
        differs |= __shfl_xor_sync(0xffffffffu, differs, 1);  // the block's two halves sit in neighbouring lanes
        if (mine) {
            if (differs) dst[2u * blk + (odd ? 1u : 0u)] = h;
            if (!odd) flags[blk] = (uint8_t)differs;
        }
    };
    const uint32_t r = lane & ((1u << l2) - 1u);
    uint64_t k0 = (odd ? b[0] : a[0]) + __shfl_xor_sync(0xffffffffu, odd ? a[0] : b[0], 1);
    if constexpr (NP == 1) {
#pragma unroll
        for (uint32_t o = 1; o < 5; ++o)
            if (o < l2) k0 += __shfl_xor_sync(0xffffffffu, k0, 1u << o);
        finish_half(k0, 0, r < 2u);
    } else {
        const uint64_t k1 = (odd ? b[1] : a[1]) + __shfl_xor_sync(0xffffffffu, odd ? a[1] : b[1], 1);
        if (l2 == 1) {  // a block is two lanes' pieces: every lane finishes a half of each of its two blocks
            finish_half(k0, 0, true);
            finish_half(k1, NP - 1, true);
        } else {
            const bool second = (lane & 2u) != 0;
            uint64_t t = (second ? k1 : k0) + __shfl_xor_sync(0xffffffffu, second ? k0 : k1, 2);
#pragma unroll
            for (uint32_t o = 2; o < 5; ++o)
                if (o < l2) t += __shfl_xor_sync(0xffffffffu, t, 1u << o);
            finish_half(t, second ? NP - 1 : 0, r < 4u);
        }
    }
}

// what aggregate_tile needs besides the votes when the sender keeps HashCache
struct HashTile {
    const ulonglong2* part;
    const ulonglong2* hold;
    ulonglong2* dst;
};

template <int DT, bool FINE, int HASH>
__device__ __forceinline__ uint64_t aggregate_tile(const TileDesc& td, uint32_t tile, uint32_t log2b, bool publish,
                                                   const uint32_t* ballot, uint32_t* bm, uint16_t* pre, uint8_t* msgs,
                                                   unsigned long long* tile_status, const HashTile& ht, uint32_t lane) {
    const uint64_t N = td.n_unit;
    const uint32_t B = 1u << log2b;
    const uint32_t nbt = kTileValues >> log2b;
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, N - v0);
    uint8_t* msg = msgs + td.msg_off;

    uint32_t run;
    if constexpr (HASH)
        run = hash_block_bitmap<DT, HASH == 3>(ht.part, ht.hold, ht.dst, bm, pre, log2b, nv, lane);
    else
        run = FINE ? scan_block_bitmap(bm, pre, log2b, lane)
                   : build_block_bitmap(ballot, bm, pre, log2b, Piece<DT>::kLog2Values, lane);

    // payload bytes of this tile: B per changed block, less for a changed short last block
    uint64_t agg = payload_bytes_of_blocks<DT>(run, log2b);
    const uint32_t rem = nv & (B - 1u);
    if (rem) {
        const uint32_t kb = nv >> log2b;
        if ((bm[kb >> 5] >> (kb & 31u)) & 1u) agg -= block_payload_bytes(B, DT) - block_payload_bytes(rem, DT);
    }
    if (publish) {
        // a unit's first tile knows its prefix (0) already
        const uint32_t mybits = nbt < 8 ? bm[0] : 0u;
        const unsigned long long flag = td.tile_in_unit == 0 ? kFlagPrefix : kFlagAggregate;
        if (lane == 0) st_status(tile_status + tile, flag | ((unsigned long long)mybits << kBitsShift) | agg);
    }
    // bitmap bytes of this tile (tiles of >= 8 blocks own whole bytes)
    if (FINE) {
        // at least 128 bytes per full tile, starting on a 128-byte boundary of the (16-byte aligned) slot
        const uint64_t byte0 = (uint64_t)td.tile_in_unit * (nbt >> 3);
        const uint32_t nbytes = (((nv + B - 1u) >> log2b) + 7u) >> 3;
        uint32_t* dst32 = reinterpret_cast<uint32_t*>(msg + byte0);
        // 16 bytes at a time, then the last words, then the last bytes
        const uint32_t quads = nbytes >> 4;
        for (uint32_t c = lane; c < quads; c += 32) reinterpret_cast<uint4*>(dst32)[c] = reinterpret_cast<const uint4*>(bm)[c];
        for (uint32_t w = 4u * quads + lane; w < (nbytes >> 2); w += 32) dst32[w] = bm[w];
        const uint32_t done = nbytes & ~3u;
        if (lane < nbytes - done) msg[byte0 + done + lane] = (uint8_t)(bm[done >> 2] >> (lane * 8u));
    } else if (nbt >= 8) {
        const uint64_t byte0 = (uint64_t)td.tile_in_unit * (nbt >> 3);
        const uint32_t nbytes = (((nv + B - 1u) >> log2b) + 7u) >> 3;
        for (uint32_t b = lane; b < nbytes; b += 32) msg[byte0 + b] = (uint8_t)(bm[b >> 2] >> ((b & 3u) * 8u));
    }
    return agg;
}

// payload <- exponents of changed blocks in block order; cache refreshed for the same blocks.
// Every consumer thread sends the exponents of its own pieces (left in the stage's shared-memory
// tile) if their block changed; `base` is the tile's exclusive offset in the unit's payload.
// (CACHE = false, the sender with HashCache: payload only.)
// (FULL: the tile is a full one, every piece complete.)
template <int DT, bool CACHE, bool FULL>
__device__ __forceinline__ void write_changed(const EncodeTileInfo& ti, uint32_t log2b, const uint32_t* bm,
                                              const uint16_t* pre, uint64_t base, const uint8_t* s_exp, uint32_t tid) {
    using P = Piece<DT>;
#pragma unroll
    for (int p = 0; p < P::kPerThread; ++p) {
        const uint32_t t0 = P::start(tid, p);
        const int nvalid = FULL ? (int)P::kValues : piece_valid<DT>(t0, ti.nv);
        if (nvalid == 0) continue;
        const uint32_t kb = t0 >> log2b;
        const uint32_t word = bm[kb >> 5];
        if (!((word >> (kb & 31u)) & 1u)) continue;
        const uint32_t rank = pre[kb >> 5] + __popc(word & ((1u << (kb & 31u)) - 1u));
        uint8_t* cdst = ti.c_ptr + t0;
        P x;
        x.template load_exp_full<Shared>(s_exp + t0);
        if constexpr (DT == CIERA_FP16) {
            // five packed bytes per piece (fewer for the unit's last, short piece), byte by byte
            uint8_t* pdst = ti.pay_dst + base + payload_bytes_of_blocks<DT>(rank, log2b) +
                            5u * ((t0 & ((1u << log2b) - 1u)) >> 3);
            uint32_t lo, hi;
            x.pack_exponents(lo, hi);
            const int nbytes = (5 * nvalid + 7) >> 3;
#pragma unroll
            for (int i = 0; i < 5; ++i)
                if (i < nbytes) pdst[i] = (uint8_t)(i < 4 ? lo >> (8 * i) : hi);
            if (!CACHE) continue;
            if (nvalid == P::kValues)
                x.template store_exp_full<Global>(cdst);
            else
                x.store_exp_partial(cdst, nvalid);
            continue;
        }
        uint8_t* pdst = ti.pay_dst + base + ((uint64_t)rank << log2b) + (t0 & ((1u << log2b) - 1u));
        if (nvalid == P::kValues) {
            x.template store_exp_full<Global>(pdst);
            if (CACHE) x.template store_exp_full<Global>(cdst);
        } else {
            x.store_exp_partial(pdst, nvalid);
            if (CACHE) x.store_exp_partial(cdst, nvalid);
        }
    }
}

// One block of B = 2^LB (fine) exponent bytes from shared memory to global memory; both addresses are B-aligned.
template <int LB>
__device__ __forceinline__ void copy_block(uint8_t* dst, const uint8_t* s_src) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(s_src);
    if (LB == 0) {
        uint32_t v;
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
        __stcs(dst, (uint8_t)v);
    } else if (LB == 1) {
        uint16_t v;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
        __stcs(reinterpret_cast<uint16_t*>(dst), v);
    } else if (LB == 2) {
        uint32_t v;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
        __stcs(reinterpret_cast<uint32_t*>(dst), v);
    } else {
        st_stream8(dst, ld_shared8(s_src));
    }
}

// The same duty with fine blocks.  Here the work is split evenly over the tile's block flags
// rather than by pieces: thread t takes the flags of values [16 t, 16 t + 16) (16, 8, 4 or 2
// flags), walks the set ones and sends each flagged block's exponents to the payload (its rank
// = flags set before it in the tile).
// The cache is refreshed by whole 32-byte sectors instead: two neighbouring threads cover one sector of the
// tile's cached exponents, and if either of them has a changed block both store their 16 new exponents (the
// unchanged ones among them equal the cached ones).  A store of single changed bytes would leave the sector
// partly written in the L2 cache, to be completed from DRAM before it can be written back; whole sectors cost
// the same DRAM traffic and one store instruction per thread instead of one per changed value.
// (fp16: a changed block's exponents go out five bits each, the block rounded up to whole bytes -- 1, 2, 3 or 5
// bytes for 1, 2, 4 or 8 values -- and byte by byte, since such blocks start on any byte.)
template <int DT, int LB>
__device__ __forceinline__ void write_changed_fine(const EncodeTileInfo& ti, const uint32_t* bm, const uint16_t* pre,
                                                   uint64_t base, const uint8_t* s_exp, uint32_t tid) {
    constexpr uint32_t B = 1u << LB;
    constexpr uint32_t kFlags = 16u >> LB;  // flags per thread
    const uint32_t bit0 = tid * kFlags;
    const uint32_t word = bm[bit0 >> 5], sh = bit0 & 31u;
    uint32_t bits = (word >> sh) & ((1u << kFlags) - 1u);  // never straddles a word
    const uint32_t v0 = tid * 16u;
    const uint32_t mine = bits != 0u ? 1u : 0u;
    if (mine | __shfl_xor_sync(0xffffffffu, mine, 1)) {
        if (v0 + 16u <= ti.nv) {
            st_stream16(ti.c_ptr + v0, ld_shared16(s_exp + v0));
        } else {
            for (uint32_t i = v0; i < ti.nv; ++i) ti.c_ptr[i] = s_exp[i];  // the unit's last values: never past its end
        }
    }
    if (bits == 0) return;
    const uint32_t rank = (uint32_t)pre[bit0 >> 5] + __popc(word & ((1u << sh) - 1u));
    if constexpr (DT == CIERA_FP16) {
        constexpr uint32_t kBlockBytes = (uint32_t)payload_bytes_of_blocks<DT>(1, LB);
        uint8_t* pdst = ti.pay_dst + base + (uint64_t)rank * kBlockBytes;
        while (bits) {
            const uint32_t j = (uint32_t)__ffs(bits) - 1u;
            bits &= bits - 1u;
            const uint32_t v = (bit0 + j) << LB;
            const uint32_t len = min(B, ti.nv - v);  // the unit's last block may be short
            unsigned long long packed = 0;
#pragma unroll
            for (uint32_t i = 0; i < B; ++i)
                if (i < len) packed |= (unsigned long long)(s_exp[v + i] & 31u) << (5u * i);
            const uint32_t nbytes = (5u * len + 7u) >> 3;
#pragma unroll
            for (uint32_t k = 0; k < kBlockBytes; ++k)
                if (k < nbytes) pdst[k] = (uint8_t)(packed >> (8u * k));
            pdst += kBlockBytes;
        }
        return;
    }
    uint8_t* pdst = ti.pay_dst + base + ((uint64_t)rank << LB);
    while (bits) {
        const uint32_t j = (uint32_t)__ffs(bits) - 1u;
        bits &= bits - 1u;
        const uint32_t v = (bit0 + j) << LB;  // the block's first value; < nv, since blocks past the end are never flagged
        if (ti.nv - v >= B) {
            copy_block<LB>(pdst, s_exp + v);
        } else {
            for (uint32_t i = 0; i < ti.nv - v; ++i) pdst[i] = s_exp[v + i];  // the unit's short last block
        }
        pdst += B;
    }
}

// Bytes of shared memory in which one warp gathers the changed exponents of its 512 values before they go out:
// up to 15 bytes of skew in front (the gathered run starts at the same address modulo 16 as its place in the
// payload), up to 512 bytes, rounded up to whole 16-byte pieces.
constexpr uint32_t kWarpGatherBytes = 16u + 512u + 16u;
// The gathering pays from about one changed exponent byte in four (measured with one value per block: 3.4 % changed
// 0.322 ms per layer gathered against 0.316 ms stored one by one, 50 % changed 0.429 against 0.548 ms).
constexpr uint32_t kGatherDensity = 4;

// Fine blocks, full tile.  A warp's 32 threads hold the flags of 512 consecutive values, so the changed blocks of
// the warp form one contiguous run of the unit's payload.  Instead of one scattered global store per changed
// block (measured: with one value per block and 3.4 % of the exponents changed, these byte stores cost more than
// a fifth of the kernel's time, with half of the exponents changed two thirds), the warp gathers the run in
// shared memory -- every thread walks its set flags as before, but stores into the warp's gather space -- and
// then writes it out in whole 16-byte pieces, one per lane, with single bytes only at the two ragged ends.
// The cache is refreshed by whole sectors as in write_changed_fine.
template <int LB>
__device__ __forceinline__ void write_changed_fine_full(const EncodeTileInfo& ti, const uint32_t* bm, const uint16_t* pre,
                                                        uint64_t base, const uint8_t* s_exp, uint8_t* s_gather,
                                                        uint32_t tid) {
    constexpr uint32_t kFlags = 16u >> LB;  // flags per thread
    const uint32_t lane = tid & 31u;
    const uint32_t bit0 = tid * kFlags;
    const uint32_t word = bm[bit0 >> 5], sh = bit0 & 31u;
    uint32_t bits = (word >> sh) & ((1u << kFlags) - 1u);  // never straddles a word
    const uint32_t v0 = tid * 16u;
    const uint32_t mine = bits != 0u ? 1u : 0u;
    if (mine | __shfl_xor_sync(0xffffffffu, mine, 1)) st_stream16(ti.c_ptr + v0, ld_shared16(s_exp + v0));
    // changed blocks of the tile before this thread's, before the warp's, and in the warp
    const uint32_t rank = (uint32_t)pre[bit0 >> 5] + __popc(word & ((1u << sh) - 1u));
    const uint32_t rank0 = __shfl_sync(0xffffffffu, rank, 0);
    const uint32_t total = __shfl_sync(0xffffffffu, rank + (uint32_t)__popc(bits), 31) - rank0;
    if (total == 0) return;
    uint8_t* const gdst = ti.pay_dst + base + ((uint64_t)rank0 << LB);  // where the warp's run goes
    const uint32_t skew = (uint32_t)(reinterpret_cast<uintptr_t>(gdst) & 15u);  // a multiple of the block size
    uint8_t* out = s_gather + skew + ((rank - rank0) << LB);
    while (bits) {
        const uint32_t j = (uint32_t)__ffs(bits) - 1u;
        bits &= bits - 1u;
        const uint8_t* src = s_exp + ((bit0 + j) << LB);
        if (LB == 0) {
            *out = *src;
        } else if (LB == 1) {
            *reinterpret_cast<uint16_t*>(out) = *reinterpret_cast<const uint16_t*>(src);
        } else if (LB == 2) {
            *reinterpret_cast<uint32_t*>(out) = *reinterpret_cast<const uint32_t*>(src);
        } else {
            st_shared8(out, ld_shared8(src));
        }
        out += 1u << LB;
    }
    __syncwarp();
    // write-out: piece c covers bytes [16 c, 16 c + 16) of the gather space; the run occupies [skew, skew + len)
    // (the ragged ends byte by byte, one byte per lane; whole pieces in between, one per lane)
    const uint32_t end = skew + (total << LB);
    uint8_t* const g16 = gdst - skew;
    const uint32_t head_end = min((skew + 15u) & ~15u, end);  // first 16-byte boundary at or after the run's start
    const uint32_t tail_start = max(head_end, end & ~15u);     // last 16-byte boundary at or before its end
    if (skew + lane < head_end) g16[skew + lane] = s_gather[skew + lane];
    for (uint32_t c = ((skew + 15u) >> 4) + lane; 16u * c + 16u <= end; c += 32u)
        st_stream16(g16 + 16u * c, ld_shared16(s_gather + 16u * c));
    if (tail_start + lane < end) g16[tail_start + lane] = s_gather[tail_start + lane];
    __syncwarp();  // the gather space is free again
}

template <int DT, bool FINE, int HASH>
__device__ __forceinline__ void send_changed(const EncodeTileInfo& ti, uint32_t log2b, const uint32_t* bm,
                                             const uint16_t* pre, uint64_t base, uint32_t tile_payload_bytes,
                                             const uint8_t* s_exp, uint8_t* s_gather, uint32_t tid) {
    if (!FINE) {
        // (as in the consumers' main loop: the two instances named there keep the one form that tests as it goes)
        constexpr bool kOneBody = (DT == CIERA_BF16 && HASH == 0) || (DT == CIERA_FP32 && HASH != 0);
        if (!kOneBody && ti.nv == (uint32_t)kTileValues)
            write_changed<DT, HASH == 0, true>(ti, log2b, bm, pre, base, s_exp, tid);
        else
            write_changed<DT, HASH == 0, false>(ti, log2b, bm, pre, base, s_exp, tid);
    } else if (DT != CIERA_FP16 && ti.nv == (uint32_t)kTileValues &&
               tile_payload_bytes >= (uint32_t)kTileValues / kGatherDensity) {
        // a full tile in which many exponents changed: gathered in shared memory, written out in whole pieces
        switch (log2b) {
            case 0: write_changed_fine_full<0>(ti, bm, pre, base, s_exp, s_gather, tid); break;
            case 1: write_changed_fine_full<1>(ti, bm, pre, base, s_exp, s_gather, tid); break;
            case 2: write_changed_fine_full<2>(ti, bm, pre, base, s_exp, s_gather, tid); break;
            default: write_changed_fine_full<3>(ti, bm, pre, base, s_exp, s_gather, tid); break;
        }
    } else {  // few changes (a store per changed block is cheaper than the gathering), a unit's last, short tile, or fp16
        switch (log2b) {
            case 0: write_changed_fine<DT, 0>(ti, bm, pre, base, s_exp, tid); break;
            case 1: write_changed_fine<DT, 1>(ti, bm, pre, base, s_exp, tid); break;
            case 2: write_changed_fine<DT, 2>(ti, bm, pre, base, s_exp, tid); break;
            default: write_changed_fine<DT, 3>(ti, bm, pre, base, s_exp, tid); break;
        }
    }
}

// `cache` is the sender's exponent cache or, with HASH, its HashCache; `tile_hash` (HASH only) gives
// the index of every tile's first block in it.
template <int DT, bool FINE, int HASH>
__global__ void __launch_bounds__(kEncodeThreads, 2)
encode_kernel(const TileDesc* __restrict__ tiles, uint32_t n_tiles, const uint2* __restrict__ seq_runs, uint32_t n_runs,
              uint32_t spread_first, uint32_t log2b, const uint8_t* __restrict__ weights, uint8_t* cache, uint8_t* msgs,
              unsigned long long* wire_bytes, uint32_t* changed_blocks, unsigned long long* tile_status,
              unsigned int* unit_ticket, unsigned int* blocks_done, int32_t* status,
              const unsigned long long* __restrict__ tile_hash) {
    static_assert(!(HASH && FINE), "HashCache: blocks of 16 values and more");
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;
    using Cfg = typename EncodeCfgOf<DT, FINE, HASH>::type;
    constexpr int SW = Cfg::kWStages;
    constexpr int SE = Cfg::kEStages;
    constexpr int kDefer = Cfg::kDefer;
    static_assert(kDescRing > SE + 2 && SE > kDefer, "ring depths");
    constexpr uint32_t kWBytes = kTileValues * VB;
    constexpr uint32_t kEBytes = kTileValues;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* const ring_w = smem;
    uint8_t* const ring_e = smem + (size_t)SW * kWBytes;
    using Ctl = EncodeCtl<SW, SE, Cfg::kBmWords>;
    Ctl* ctl = reinterpret_cast<Ctl*>(ring_e + (size_t)SE * kEBytes);
    // HASH: per stage of the exponent ring, the tile's cached hashes and then the partial sums
    static_assert(sizeof(Ctl) % 16 == 0, "the hash stages follow the control block");
    static_assert(offsetof(Ctl, bm) % 16 == 0 && offsetof(Ctl, pre) % 4 == 0, "block flags are read 16 bytes at a time");
    uint8_t* const ring_h = reinterpret_cast<uint8_t*>(ctl) + sizeof(Ctl);
    const uint32_t kHoldBytes = HASH ? hash_hold_bytes<DT>(log2b) : 0u;
    const uint32_t kHStage = HASH ? kHoldBytes + hash_part_bytes<DT>(log2b) : 0u;

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    volatile int* abort = &ctl->abort;
    // FINE: every consumer warp's gather space for its changed exponents (in place of the hash stages)
    uint8_t* const s_gather = ring_h + (size_t)(warp < (uint32_t)kWarps ? warp : 0u) * kWarpGatherBytes;

    if (tid == 0) {
        for (int s = 0; s < SW; ++s) {
            mbar_init(&ctl->full_w[s], 1);
            mbar_init(&ctl->empty_w[s], kWarps);
        }
        for (int s = 0; s < SE; ++s) {
            mbar_init(&ctl->full_e[s], 1);
            mbar_init(&ctl->voted[s], kWarps);
            mbar_init(&ctl->summed[s], 1);
            mbar_init(&ctl->resolved[s], 1);
            mbar_init(&ctl->empty_e[s], kWarps);
        }
        ctl->abort = 0;
        ctl->issued = 0;
        ctl->seen = 0;
        mbar_fence_init();
    }
    __syncthreads();

    // The block's tiles form a sequence k = 0, 1, 2, ... that only the producer knows in advance;
    // it closes the sequence with kResolvers end markers (one for each resolver warp), which the
    // other roles pass on to each other through the same barriers as real tiles.
    if (warp == kProducerWarp) {
        // ---------------------------------------------------------------- producer
        if (lane == 0) {
            TileWalk walk(seq_runs, unit_ticket, n_runs, spread_first, n_tiles, gridDim.x, blockIdx.x);
            uint32_t seq_nxt = 0;
            uint32_t tile_nxt = walk.next(seq_nxt);
            TileDesc nxt;
            unsigned long long hb_nxt = 0;  // HASH: index of the tile's first block in HashCache
            if (tile_nxt != kNoTile) {      // descriptors are fetched one tile ahead
                nxt = load_tile_desc(tiles + tile_nxt);
                if (HASH) hb_nxt = __ldg(tile_hash + tile_nxt);
            }
            uint32_t markers = 0;
            for (uint32_t k = 0;; ++k) {
                const TileDesc td = nxt;
                const uint32_t tile = tile_nxt;
                const uint32_t seq = seq_nxt;
                const unsigned long long hb = hb_nxt;
                if (tile != kNoTile) {
                    tile_nxt = walk.next(seq_nxt);
                    if (tile_nxt != kNoTile) {
                        nxt = load_tile_desc(tiles + tile_nxt);
                        if (HASH) hb_nxt = __ldg(tile_hash + tile_nxt);
                    }
                }
                const uint32_t sw = k % SW, se = k % SE;
                if (k >= (uint32_t)SW && !mbar_wait(&ctl->empty_w[sw], ((k / SW) & 1u) ^ 1u, abort, status)) break;
                if (k >= (uint32_t)SE && !mbar_wait(&ctl->empty_e[se], ((k / SE) & 1u) ^ 1u, abort, status)) break;
                ctl->tile_idx[k % kDescRing] = tile;
                if (tile == kNoTile) {  // end marker
                    mbar_arrive(&ctl->full_w[sw]);
                    if (HASH) mbar_arrive(&ctl->full_e[se]);
                    if (++markers == (uint32_t)kResolvers) break;
                    continue;
                }
                ctl->desc[k % kDescRing] = td;
                ctl->seq[k % kDescRing] = seq;
                const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
                const uint64_t left = td.n_unit - v0;
                {
                    const uint64_t smoff = sm_offset(td.n_unit, log2b);
                    EncodeTileInfo ti;
                    ti.sm_dst = msgs + td.msg_off + smoff + sm_bytes_of_values<DT>(v0);
                    ti.pay_dst = msgs + td.msg_off + smoff + pad16(sm_section_bytes(td.n_unit, DT));
                    ti.c_ptr = HASH ? cache + hb * 16ull : cache + td.c_off;
                    ti.w_src = weights + td.w_off;
                    ti.nv = (uint32_t)min((uint64_t)kTileValues, left);
                    ctl->info[k % kDescRing] = ti;
                }
                if constexpr (HASH) {
                    // the cached hashes of the tile's blocks (16 bytes each) come in for every tile
                    if (left >= (uint64_t)kTileValues) {
                        mbar_arrive_expect_tx(&ctl->full_w[sw], kWBytes);
                        bulk_load(ring_w + (size_t)sw * kWBytes, weights + td.w_off, kWBytes, &ctl->full_w[sw]);
                    } else {
                        mbar_arrive(&ctl->full_w[sw]);
                    }
                    const uint32_t nblk = (uint32_t)((min((uint64_t)kTileValues, left) + (1u << log2b) - 1u) >> log2b);
                    mbar_arrive_expect_tx(&ctl->full_e[se], nblk * 16u);
                    bulk_load(ring_h + (size_t)se * kHStage, cache + hb * 16ull, nblk * 16u, &ctl->full_e[se]);
                } else if (left >= (uint64_t)kTileValues) {
                    // both copies of the tile complete on the one barrier the consumers wait for
                    mbar_arrive_expect_tx(&ctl->full_w[sw], kWBytes + kEBytes);
                    bulk_load(ring_w + (size_t)sw * kWBytes, weights + td.w_off, kWBytes, &ctl->full_w[sw]);
                    bulk_load(ring_e + (size_t)se * kEBytes, cache + td.c_off, kEBytes, &ctl->full_w[sw]);
                } else {
                    // short tile: consumers read global memory themselves
                    mbar_arrive(&ctl->full_w[sw]);
                }
                ctl->issued = k + 1;
            }
        }
    } else if (warp == kAggregatorWarp) {
        // ---------------------------------------------------------------- aggregator
        uint64_t run_incl = 0;  // payload bytes of the current alone-worked unit up to the last tile
        uint32_t byte_acc = 0;  // its bitmap byte in the making (tiles of fewer than 8 blocks)
        uint32_t markers = 0;
        for (uint32_t k = 0;; ++k) {
            const uint32_t se = k % SE;
            if (!mbar_wait(&ctl->voted[se], (k / SE) & 1u, abort, status)) break;
            const uint32_t tile = ctl->tile_idx[k % kDescRing];
            if (tile == kNoTile) {  // pass the end marker on to the resolver in charge of slot k
                if (lane == 0) mbar_arrive(&ctl->summed[se]);
                if (++markers == (uint32_t)kResolvers) break;
                continue;
            }
            const TileDesc td = ctl->desc[k % kDescRing];
            const uint32_t seq_bits = ctl->seq[k % kDescRing];
            const bool seq = seq_bits != 0;
            HashTile ht{nullptr, nullptr, nullptr};
            if constexpr (HASH) {
                // the cached hashes were staged by a bulk copy that completes on full_e: observe it here too
                if (!mbar_wait(&ctl->full_e[se], (k / SE) & 1u, abort, status)) break;
                ht.hold = reinterpret_cast<const ulonglong2*>(ring_h + (size_t)se * kHStage);
                ht.part = reinterpret_cast<const ulonglong2*>(ring_h + (size_t)se * kHStage + kHoldBytes);
                ht.dst = reinterpret_cast<ulonglong2*>(ctl->info[k % kDescRing].c_ptr);
            }
            const uint64_t agg = aggregate_tile<DT, FINE, HASH>(td, tile, log2b, !seq, ctl->ballot[se], ctl->bm[se],
                                                                ctl->pre[se], msgs, tile_status, ht, lane);
            if (seq) {
                // the run is this block's: the tile's offset is the running sum; a run that does not start its
                // unit carries on from the inclusive offset that the run before it left in its last tile's
                // status word (that run went out many draws earlier; the wait is bounded all the same; reading
                // the word in the producer thread instead, tiles ahead, was slower)
                uint64_t excl = run_incl;
                if (td.tile_in_unit == 0)
                    excl = 0;
                else if (seq_bits & kSeqRunStart) {
                    excl = wait_status(tile_status + tile - 1, status) & kValueMask;
                    __syncwarp();
                    if (lane == 0) st_status(tile_status + tile - 1, 0ull);  // its one reader leaves the word empty again
                }
                run_incl = excl + agg;
                if ((seq_bits & kSeqRunEnd) && td.tile_in_unit != td.n_tiles_unit - 1u && lane == 0)
                    st_status(tile_status + tile, kFlagPrefix | run_incl);
                const uint32_t nbt = kTileValues >> log2b;
                const bool last = td.tile_in_unit == td.n_tiles_unit - 1u;
                if (nbt < 8) {
                    const uint32_t tpb = 8u / nbt, p = td.tile_in_unit & (tpb - 1u);
                    byte_acc = (p == 0 ? 0u : byte_acc) | (ctl->bm[se][0] << (p * nbt));
                    if ((p == tpb - 1u || last) && lane == 0) msgs[td.msg_off + td.tile_in_unit / tpb] = (uint8_t)byte_acc;
                }
                if (last) finish_unit<DT>(td, log2b, run_incl, msgs, wire_bytes, changed_blocks, lane);
                if (lane == 0) {
                    ctl->base[se] = excl;
                    ctl->agg[se] = agg;
                }
            } else if (lane == 0) {
                ctl->agg[se] = agg;
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&ctl->summed[se]);
                if (seq) mbar_arrive(&ctl->resolved[se]);
            }
        }
    } else if (warp >= kResolverWarp0) {
        // ---------------------------------------------------------------- resolvers (slots k = i, i + R, ...)
        for (uint32_t k = warp - kResolverWarp0;; k += kResolvers) {
            const uint32_t se = k % SE;
            if (!mbar_wait(&ctl->summed[se], (k / SE) & 1u, abort, status)) break;
            const uint32_t tile = ctl->tile_idx[k % kDescRing];
            if (tile == kNoTile) break;
            if (ctl->seq[k % kDescRing] != 0) continue;  // the aggregator has done it all
            const TileDesc td = ctl->desc[k % kDescRing];
            const uint64_t excl = resolve_tile<DT>(td, tile, log2b, ctl->agg[se], ctl->bm[se], msgs, wire_bytes,
                                                   changed_blocks, tile_status, status, lane);
            if (lane == 0) {
                ctl->base[se] = excl;
                mbar_arrive(&ctl->resolved[se]);
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers
        uint32_t k_end = kNoTile;  // slot of the first end marker, once seen
        uint32_t k = 0;
        // stage and phase of slot k in the two rings, and of slot k - kDefer in the exponent ring, kept
        // as running counters (the ring depths are no powers of two)
        uint32_t sw = 0, pw = 0, se = 0, pe = 0, je = 0, pj = 0;
        // HASH: the lanes of a warp that share a block (a power of two, at most the warp) add up their terms
        const uint32_t hash_lanes_l2 = min(5u, log2b - (uint32_t)P::kLog2Values);
        for (;; ++k) {
            // (the producer starts the loads of slot k only once both of its stages are free, and the cached
            // exponents land on the same barrier as the weights; with HashCache the cached hashes, which only
            // the aggregator reads, land on full_e)
            if (!mbar_wait(&ctl->full_w[sw], pw, abort, status)) break;
            if (tid == 0) ctl->seen = k + 1;
            const bool marker = ctl->tile_idx[k % kDescRing] == kNoTile;
            if (marker) {
                if (k_end == kNoTile) k_end = k;
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&ctl->voted[se]);  // pass the end marker on to the aggregator
                    mbar_arrive(&ctl->empty_w[sw]);  // and hand the marker's (unused) stages back
                    mbar_arrive(&ctl->empty_e[se]);
                }
            } else {
                const EncodeTileInfo ti = ctl->info[k % kDescRing];
                const uint32_t nv = ti.nv;
                const uint8_t* const s_w = ring_w + (size_t)sw * kWBytes;
                uint8_t* const s_e = ring_e + (size_t)se * kEBytes;
                uint64_t hash_a[P::kPerThread], hash_b[P::kPerThread];  // HASH: the pieces' sums of terms
                // The pieces of this thread.  Most instances compile the loop twice: for full tiles (staged
                // in shared memory, every piece complete, no tests on the way) and for a unit's last, short
                // tile; that measured 2-12 % faster (fp16 most).  Two instances keep one loop that tests as it
                // goes, which measured faster for them: bf16 with coarse blocks and the exponent cache (1 %),
                // fp32 with HashCache (5 %).
                constexpr bool kOneBody = (DT == CIERA_BF16 && !FINE && HASH == 0) || (DT == CIERA_FP32 && HASH != 0);
                if constexpr (kOneBody) {
                    // a plain loop that tests as it goes
#define CIERA_PIECES_FULL false
#define CIERA_PIECES_STAGED (nv == (uint32_t)kTileValues)
#include "ciera_encode_pieces.inc"
#undef CIERA_PIECES_FULL
#undef CIERA_PIECES_STAGED
                } else {
                    auto pieces = [&](auto full_tag) {
                        constexpr bool kFull = decltype(full_tag)::value;
#define CIERA_PIECES_FULL kFull
#define CIERA_PIECES_STAGED kFull
#include "ciera_encode_pieces.inc"
#undef CIERA_PIECES_FULL
#undef CIERA_PIECES_STAGED
                    };
                    if (nv == (uint32_t)kTileValues)
                        pieces(std::true_type{});
                    else
                        pieces(std::false_type{});
                }
                if constexpr (HASH) {
                    uint64_t* const part = reinterpret_cast<uint64_t*>(ring_h + (size_t)se * kHStage + kHoldBytes);
                    if constexpr (HASH == 3) {
                        // the tile's cached hashes have to be there now (they land on full_e)
                        if (!mbar_wait(&ctl->full_e[se], pe, abort, status)) break;
                        finish_hash_groups<DT, P::kPerThread>(hash_a, hash_b, hash_lanes_l2, log2b, nv, tid,
                                                              reinterpret_cast<const uint64_t*>(ring_h + (size_t)se * kHStage),
                                                              reinterpret_cast<uint64_t*>(ti.c_ptr),
                                                              reinterpret_cast<uint8_t*>(part), lane);
                    } else {
                        reduce_hash_terms<P::kPerThread>(hash_a, hash_b, hash_lanes_l2, (P::start(tid, 0) >> P::kLog2Values) >> hash_lanes_l2,
                                                         (P::start(tid, P::kPerThread - 1) >> P::kLog2Values) >> hash_lanes_l2, part, lane);
                    }
                }
                __syncwarp();  // the warp's shared-memory accesses above are ordered before lane 0's arrives
                if (lane == 0) {
                    mbar_arrive(&ctl->empty_w[sw]);
                    mbar_arrive(&ctl->voted[se]);
                }
            }

            // the changed exponents of the tile handled kDefer slots ago: its offset is known by now
            if (k >= (uint32_t)kDefer) {
                if (k - kDefer < k_end) {
                    if (!mbar_wait(&ctl->resolved[je], pj, abort, status)) break;
                    send_changed<DT, FINE, HASH>(ctl->info[(k - kDefer) % kDescRing], log2b, ctl->bm[je], ctl->pre[je],
                                                 ctl->base[je], (uint32_t)ctl->agg[je], ring_e + (size_t)je * kEBytes,
                                                 s_gather, tid);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->empty_e[je]);
                }
                if (++je == (uint32_t)SE) {
                    je = 0;
                    pj ^= 1u;
                }
            }
            if (marker && k + 1u == k_end + (uint32_t)kResolvers) break;  // that was the last end marker
            if (++sw == (uint32_t)SW) {
                sw = 0;
                pw ^= 1u;
            }
            if (++se == (uint32_t)SE) {
                se = 0;
                pe ^= 1u;
            }
        }
        // tiles whose changed exponents are still to be sent (when kDefer > kResolvers)
        if (!*abort && k_end != kNoTile) {
            for (uint32_t j = k + 1u >= (uint32_t)kDefer ? k + 1u - kDefer : 0u; j < k_end; ++j) {
                const uint32_t je = j % SE;
                if (!mbar_wait(&ctl->resolved[je], (j / SE) & 1u, abort, status)) break;
                send_changed<DT, FINE, HASH>(ctl->info[j % kDescRing], log2b, ctl->bm[je], ctl->pre[je], ctl->base[je],
                                             (uint32_t)ctl->agg[je], ring_e + (size_t)je * kEBytes, s_gather, tid);
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->empty_e[je]);
            }
        }
    }

    // leave together; after an aborted run wait (bounded) for bulk copies that are still in flight
    __syncthreads();
    if (tid == 0 && ctl->abort) {
        for (uint32_t k = ctl->seen; k < ctl->issued; ++k) {
            for (uint32_t i = 0; i < kMaxBarrierPolls; ++i)
                if (mbar_try_wait(&ctl->full_w[k % SW], (k / SW) & 1u)) break;
            if (HASH) {
                for (uint32_t i = 0; i < kMaxBarrierPolls; ++i)
                    if (mbar_try_wait(&ctl->full_e[k % SE], (k / SE) & 1u)) break;
            }
        }
    }
    // The scratch is handed back the way it was found, all zero: the hand-off words of the runs were emptied by
    // their readers, the run counter by its last draw; the status words of the spread tiles (read by any number
    // of later tiles) and the counter of finished blocks are emptied here by the block that finishes last.
    __shared__ unsigned int s_last;
    if (tid == 0) {
        __threadfence();
        s_last = atomicAdd(blocks_done, 1u) + 1u == gridDim.x ? 1u : 0u;
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        for (uint32_t t = spread_first + tid; t < n_tiles; t += kEncodeThreads) st_status(tile_status + t, 0ull);
        if (tid == 0) atomicExch(blocks_done, 0u);
    }
}

// (with HashCache the size depends on the block size: see hash_hold_bytes, hash_part_bytes)
template <int DT, bool FINE, int HASH>
static size_t encode_smem_bytes(uint32_t log2b) {
    using Cfg = typename EncodeCfgOf<DT, FINE, HASH>::type;
    constexpr int SW = Cfg::kWStages, SE = Cfg::kEStages;
    const size_t hash_stage = HASH ? (size_t)hash_hold_bytes<DT>(log2b) + hash_part_bytes<DT>(log2b) : 0;
    return (size_t)SW * kTileValues * Traits<DT>::kValueBytes + (size_t)SE * kTileValues +
           sizeof(EncodeCtl<SW, SE, Cfg::kBmWords>) + (size_t)SE * hash_stage + (FINE ? (size_t)kWarps * kWarpGatherBytes : 0);
}

// Largest grid whose blocks are all resident at once, per device and block size (0 = not yet known).
template <int DT, bool FINE, int HASH>
static int encode_grid_limit(uint32_t log2b, int* out) {
    static std::atomic<int> cached[64][16];  // (zero-initialised; any host thread may be the first to fill an entry)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64 || log2b >= 16) return CIERA_ERR_UNSUPPORTED;
    if (cached[dev][log2b].load(std::memory_order_acquire) == 0) {
        const size_t smem = encode_smem_bytes<DT, FINE, HASH>(log2b);
        // (the limit set here is the largest any block size asks for: the smallest block of the class)
        e = cudaFuncSetAttribute(encode_kernel<DT, FINE, HASH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)encode_smem_bytes<DT, FINE, HASH>(FINE ? 0u : HASH == 1 ? kHashShortRingsLog2 + 1u : kFineLog2));
        if (e != cudaSuccess) return record_cuda_error(e);
        int per_sm = 0, sms = 0, coop = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, encode_kernel<DT, FINE, HASH>, kEncodeThreads, smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (per_sm < 1 || sms < 1 || !coop) return CIERA_ERR_UNSUPPORTED;
        cached[dev][log2b].store(per_sm * sms, std::memory_order_release);
    }
    *out = cached[dev][log2b].load(std::memory_order_acquire);
    return CIERA_OK;
}

// `scratch`: one status word per tile, then the run counter and the counter of finished blocks; all zero when
// the kernel starts, and all zero again when it has finished without a device-side error.
template <int DT, bool FINE, int HASH = 0>
static int launch_encode(const ciera_plan* p, const void* weights_dev, void* sender_cache_dev, void* messages_dev,
                         uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* scratch, int32_t* status_dev,
                         cudaStream_t s) {
    int limit = 0;
    const int rc = encode_grid_limit<DT, FINE, HASH>(p->log2b, &limit);
    if (rc) return rc;
    const TileDesc* tiles = p->tiles_dev;
    uint32_t nt = (uint32_t)p->tiles.size();
    const uint32_t grid = nt < (uint32_t)limit ? nt : (uint32_t)limit;
    const uint2* seq_runs = p->seq_runs_dev;
    uint32_t n_runs = (uint32_t)p->seq_runs.size();
    uint32_t spread_first = p->seq_first.back();
    uint32_t log2b = p->log2b;
    const uint8_t* w = (const uint8_t*)weights_dev;
    uint8_t* c = (uint8_t*)sender_cache_dev;
    uint8_t* m = (uint8_t*)messages_dev;
    unsigned long long* wb = (unsigned long long*)wire_bytes_dev;
    unsigned long long* ts = (unsigned long long*)scratch;
    unsigned int* ticket = (unsigned int*)((uint8_t*)scratch + workspace_sender_counters_offset(nt));
    unsigned int* done = ticket + 1;
    const unsigned long long* tile_hash = HASH ? p->tile_hash_dev : nullptr;
    const size_t smem = encode_smem_bytes<DT, FINE, HASH>(log2b);
    const bool has_spread = p->seq_first.back() < nt;  // tiles of longer units: look-back between blocks
    cudaError_t e;
    if (has_spread) {
        // cooperative launch: the runtime starts the grid only when all of its blocks fit on the
        // GPU together, which is what the look-back between blocks relies on
        void* args[] = {&tiles, &nt, &seq_runs, &n_runs, &spread_first, &log2b, &w, &c, &m, &wb, &changed_blocks_dev, &ts,
                        &ticket, &done, &status_dev, &tile_hash};
        e = cudaLaunchCooperativeKernel((const void*)encode_kernel<DT, FINE, HASH>, dim3(grid), dim3(kEncodeThreads), args,
                                        smem, s);
    } else {
        encode_kernel<DT, FINE, HASH><<<grid, kEncodeThreads, smem, s>>>(
            tiles, nt, seq_runs, n_runs, spread_first, log2b, w, c, m, wb, changed_blocks_dev, ts, ticket, done, status_dev,
            tile_hash);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return record_cuda_error(e);
    count_launch();
    return CIERA_OK;
}

// picks the kernel for the plan's precision and block class
static int launch_encode_any(const ciera_plan* p, const void* weights_dev, void* sender_cache_dev, void* messages_dev,
                             uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* scratch, int32_t* status_dev,
                             cudaStream_t s) {
    const bool fine = is_fine(p->log2b);
    if (p->dtype == CIERA_FP16)
        return fine ? launch_encode<CIERA_FP16, true>(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev,
                                                      changed_blocks_dev, scratch, status_dev, s)
                    : launch_encode<CIERA_FP16, false>(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev,
                                                       changed_blocks_dev, scratch, status_dev, s);
    if (p->dtype == CIERA_BF16)
        return fine ? launch_encode<CIERA_BF16, true>(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev,
                                                      changed_blocks_dev, scratch, status_dev, s)
                    : launch_encode<CIERA_BF16, false>(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev,
                                                       changed_blocks_dev, scratch, status_dev, s);
    return fine ? launch_encode<CIERA_FP32, true>(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev,
                                                  changed_blocks_dev, scratch, status_dev, s)
                : launch_encode<CIERA_FP32, false>(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev,
                                                   changed_blocks_dev, scratch, status_dev, s);
}

// the sender with HashCache: blocks of 16 values and more (checked by the caller)
int launch_encode_hashed(const ciera_plan* p, const void* weights_dev, void* hash_cache_dev, void* messages_dev,
                         uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* scratch, int32_t* status_dev,
                         cudaStream_t s) {
    const bool short_rings = p->log2b <= kHashShortRingsLog2;
    if (p->dtype == CIERA_BF16 && hash_finished_by_consumers<CIERA_BF16>(p->log2b))
        return launch_encode<CIERA_BF16, false, 3>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                   changed_blocks_dev, scratch, status_dev, s);
    if (p->dtype == CIERA_FP16 && hash_finished_by_consumers<CIERA_FP16>(p->log2b))
        return launch_encode<CIERA_FP16, false, 3>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                   changed_blocks_dev, scratch, status_dev, s);
    if (p->dtype == CIERA_FP16)
        return short_rings ? launch_encode<CIERA_FP16, false, 2>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                                 changed_blocks_dev, scratch, status_dev, s)
                           : launch_encode<CIERA_FP16, false, 1>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                                 changed_blocks_dev, scratch, status_dev, s);
    if (p->dtype == CIERA_FP32 && hash_finished_by_consumers<CIERA_FP32>(p->log2b))
        return launch_encode<CIERA_FP32, false, 3>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                   changed_blocks_dev, scratch, status_dev, s);
    if (p->dtype == CIERA_BF16)
        return short_rings ? launch_encode<CIERA_BF16, false, 2>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                                 changed_blocks_dev, scratch, status_dev, s)
                           : launch_encode<CIERA_BF16, false, 1>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                                 changed_blocks_dev, scratch, status_dev, s);
    return short_rings ? launch_encode<CIERA_FP32, false, 2>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                             changed_blocks_dev, scratch, status_dev, s)
                       : launch_encode<CIERA_FP32, false, 1>(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev,
                                                             changed_blocks_dev, scratch, status_dev, s);
}

}  // namespace ciera

using namespace ciera;

static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

extern "C" int ciera_encode(const ciera_plan* p, const void* weights_dev, void* sender_cache_dev, void* messages_dev,
                            uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* workspace_dev,
                            int32_t* status_dev, void* stream) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    if (p->n_units == 0) return CIERA_OK;
    if (!wire_bytes_dev || !changed_blocks_dev) return CIERA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t nt = (uint32_t)p->tiles.size();
    cudaError_t e;
    if (p->has_empty_units) {  // units without tiles: their outputs are written here
        e = cudaMemsetAsync(wire_bytes_dev, 0, sizeof(uint64_t) * p->n_units, s);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaMemsetAsync(changed_blocks_dev, 0, sizeof(uint32_t) * p->n_units, s);
        if (e != cudaSuccess) return record_cuda_error(e);
    }
    if (nt == 0) return CIERA_OK;
    if (!weights_dev || !sender_cache_dev || !messages_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(weights_dev) || misaligned16(sender_cache_dev) || misaligned16(messages_dev) ||
        misaligned16(workspace_dev) || ((uintptr_t)wire_bytes_dev & 7u) || ((uintptr_t)changed_blocks_dev & 3u))
        return CIERA_ERR_MISALIGNED;
    // scratch = one look-back status word per tile, then two counters: all zero on entry (ciera_workspace_init,
    // or left so by the previous call), and the kernel hands it back all zero
    return launch_encode_any(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev, changed_blocks_dev,
                             workspace_dev, status_dev, s);
}

// ------------------------------------------------------------------------------------------
// Encode for callers that have no scratch buffer to give.
//
// Some callers hand this library only the buffers they already own -- parameter shards, caches,
// communication buffers -- and cannot come up with one more device allocation at the moment of the
// call: a training runtime whose memory pool has claimed the whole GPU (a fresh allocation would
// fail or fragment the pool), a gather hook that must not synchronise the device (allocating
// does), a plug-in that was given pointers but no allocator.  For them the look-back scratch of
// the encode kernel lives in the library itself: a fixed array in device memory that every GPU
// loading the library holds from load until the process exits.

static __device__ __align__(256) unsigned long long g_encode_scratch[CIERA_NOALLOC_MAX_TILES + 2];

// Device address of g_encode_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, not an address a kernel could use, so the address is looked up once
// per device (with that device current) and kept.
static int encode_scratch_address(unsigned long long** out) {
    static std::atomic<unsigned long long*> cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    unsigned long long* ptr = cached[dev].load(std::memory_order_acquire);
    if (ptr == nullptr) {
        void* q = nullptr;
        e = cudaGetSymbolAddress(&q, g_encode_scratch);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (q == nullptr) return CIERA_ERR_CUDA;
        ptr = static_cast<unsigned long long*>(q);
        cached[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return CIERA_OK;
}

extern "C" int ciera_encode_noalloc(const ciera_plan* p, const void* weights_dev, void* sender_cache_dev,
                                    void* messages_dev, uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev,
                                    int32_t* status_dev, void* stream) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt > CIERA_NOALLOC_MAX_TILES) return CIERA_ERR_TOO_LARGE;
    if (p->n_units == 0) return CIERA_OK;
    if (!wire_bytes_dev || !changed_blocks_dev) return CIERA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (p->has_empty_units) {  // units without tiles: their outputs are written here
        e = cudaMemsetAsync(wire_bytes_dev, 0, sizeof(uint64_t) * p->n_units, s);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaMemsetAsync(changed_blocks_dev, 0, sizeof(uint32_t) * p->n_units, s);
        if (e != cudaSuccess) return record_cuda_error(e);
    }
    if (nt == 0) return CIERA_OK;
    if (!weights_dev || !sender_cache_dev || !messages_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(weights_dev) || misaligned16(sender_cache_dev) || misaligned16(messages_dev) ||
        ((uintptr_t)wire_bytes_dev & 7u) || ((uintptr_t)changed_blocks_dev & 3u))
        return CIERA_ERR_MISALIGNED;
    unsigned long long* scratch = nullptr;
    int rc = encode_scratch_address(&scratch);
    if (rc) return rc;
    // the array keeps what the previous call left in it: the status words of this call's tiles and
    // the unit counter behind them have to start at zero
    e = cudaMemsetAsync(scratch, 0, sizeof(unsigned long long) * nt + 16, s);
    if (e != cudaSuccess) return record_cuda_error(e);
    return launch_encode_any(p, weights_dev, sender_cache_dev, messages_dev, wire_bytes_dev, changed_blocks_dev, scratch,
                             status_dev, s);
}
