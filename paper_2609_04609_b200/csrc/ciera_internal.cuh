// Internal declarations shared by the translation units of libciera (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "ciera.h"

namespace ciera {

// One tile = kTileValues consecutive values of one unit = the work of one thread block.
// Each thread owns kVPT consecutive values ("a group"): 16 values are 16 exponent bytes, i.e.
// one 128-bit access on each of the byte-wide streams (cache, sm, payload).
constexpr int kThreads = 512;
constexpr int kVPT = 16;
constexpr int kTileValues = kThreads * kVPT;  // 8192
constexpr int kWarps = kThreads / 32;
// Block sizes come in two classes.  "Coarse" blocks (16 values and more) hold whole pieces, so a
// piece has one flag and a tile at most 512 blocks; "fine" blocks (1, 2, 4 or 8 values) are
// smaller than (or as large as) a piece, a piece has several flags and a tile up to 8192 blocks.
constexpr uint32_t kFineLog2 = 4;                    // log2b < kFineLog2: fine
constexpr int kBitmapWords = kTileValues / 16 / 32;  // 16: words of block flags of a tile, coarse
constexpr int kFineBitmapWords = kTileValues / 32;   // 256: the same, fine
__host__ __device__ inline bool is_fine(uint32_t log2b) { return log2b < kFineLog2; }

// Device-side tile descriptor: everything a thread block needs, in one 48-byte record so that
// a single dependent load stands between block start and the first data load.
struct __align__(16) TileDesc {
    uint64_t w_off;         // byte offset of the tile's first value in the weights buffer
    uint64_t c_off;         // byte offset of the tile's first value in the cache
    uint64_t msg_off;       // byte offset of the unit's message slot
    uint64_t n_unit;        // N of the unit
    uint32_t unit;          // index into the per-unit outputs
    uint32_t tile_in_unit;  // 0 .. n_tiles_unit-1
    uint32_t first_tile;    // table index of the unit's first tile
    uint32_t n_tiles_unit;  // tiles of this unit
};
static_assert(sizeof(TileDesc) == 48, "TileDesc must stay three 16-byte words");

// Tile status word used by the single-pass look-back of the encode kernel.
//   bits 63:62  0 = empty, 1 = aggregate of this tile, 2 = inclusive prefix up to this tile
//   bits 61:56  the tile's own bitmap bits when a tile holds fewer than 8 blocks
//   bits 55:0   payload bytes
constexpr unsigned long long kFlagAggregate = 1ull << 62;
constexpr unsigned long long kFlagPrefix = 2ull << 62;
constexpr unsigned long long kValueMask = (1ull << 56) - 1;
constexpr int kBitsShift = 56;

// Upper bound on polls of one status word before a tile gives up and raises CIERA_ERR_TIMEOUT.
constexpr uint32_t kMaxPolls = 1u << 21;

template <int DT>
struct Traits;
template <>
struct Traits<CIERA_BF16> {
    static constexpr int kValueBytes = 2;
    static constexpr int kSmBytes = 1;
};
template <>
struct Traits<CIERA_FP32> {
    static constexpr int kValueBytes = 4;
    static constexpr int kSmBytes = 3;
};
// fp16: 11 bits of sign-plus-mantissa and 5 exponent bits per value on the wire, so the byte
// counts below hold for multiples of 8 values only (kSmBytes is not used for it)
template <>
struct Traits<CIERA_FP16> {
    static constexpr int kValueBytes = 2;
    static constexpr int kSmBytes = 0;
};
// bytes of sign-plus-mantissa of `values` values (a multiple of 8 for fp16), and payload bytes of
// `blocks` full blocks
template <int DT>
__host__ __device__ constexpr uint64_t sm_bytes_of_values(uint64_t values) {
    return DT == CIERA_FP16 ? (values >> 3) * 11 : values * Traits<DT>::kSmBytes;
}
template <int DT>
__host__ __device__ constexpr uint64_t payload_bytes_of_blocks(uint64_t blocks, uint32_t log2b) {
    // fp16: five bits per exponent, a block rounded up to whole bytes (1, 2, 3, 5, 10, 20, ... bytes)
    return DT == CIERA_FP16 ? blocks * (((5ull << log2b) + 7ull) >> 3) : blocks << log2b;
}

__host__ __device__ inline uint64_t pad16(uint64_t x) { return (x + 15ull) & ~15ull; }
__host__ __device__ inline uint64_t num_blocks(uint64_t n, uint32_t log2b) {
    return (n + (1ull << log2b) - 1) >> log2b;
}
__host__ __device__ inline uint64_t bitmap_bytes(uint64_t n, uint32_t log2b) { return (num_blocks(n, log2b) + 7) >> 3; }
__host__ __device__ inline uint64_t sm_offset(uint64_t n, uint32_t log2b) { return pad16(bitmap_bytes(n, log2b)); }
__host__ __device__ inline uint64_t payload_offset(uint64_t n, uint32_t sm_bytes_per_value, uint32_t log2b) {
    return sm_offset(n, log2b) + pad16(n * sm_bytes_per_value);
}

// The same sizes by precision, for code that also handles fp16 (5 exponent bits and 11
// sign-plus-mantissa bits per value, packed without gaps; every changed block of the payload starts
// on a byte boundary).
__host__ __device__ inline uint32_t sm_bits_of(int dtype) { return dtype == CIERA_FP32 ? 24u : dtype == CIERA_FP16 ? 11u : 8u; }
__host__ __device__ inline uint32_t exp_bits_of(int dtype) { return dtype == CIERA_FP16 ? 5u : 8u; }
__host__ __device__ inline uint64_t sm_section_bytes(uint64_t n, int dtype) { return (n * sm_bits_of(dtype) + 7) >> 3; }
__host__ __device__ inline uint64_t block_payload_bytes(uint64_t len, int dtype) { return (len * exp_bits_of(dtype) + 7) >> 3; }
__host__ __device__ inline uint64_t payload_offset_of(uint64_t n, int dtype, uint32_t log2b) {
    return sm_offset(n, log2b) + pad16(sm_section_bytes(n, dtype));
}
// the largest payload a unit of n values can have: every block changed
__host__ __device__ inline uint64_t payload_bytes_max(uint64_t n, int dtype, uint32_t log2b) {
    const uint64_t nb = num_blocks(n, log2b);
    if (nb == 0) return 0;
    return (nb - 1) * block_payload_bytes(1ull << log2b, dtype) + block_payload_bytes(n - ((nb - 1) << log2b), dtype);
}

// Units with more blocks than this get their per-tile "changed blocks before" counts from a
// prefix kernel at decode time; shorter ones read them straight from the bitmap.  With fine
// blocks every unit of more than one tile goes through the prefix kernel.
constexpr uint32_t kDecodeDirectBlocks = 4096;

// Layout of the scratch ("workspace") of a plan with nt tiles, shared by the sender, transport and receiver calls:
//   [0, 8 nt)             one 64-bit look-back status word per tile                     (sender)
//   [8 nt, + 16)          the sender's run counter and its counter of finished blocks   (sender)
//   [8 nt + 16, + 16)     the counter that transport and receiver hand their tiles out from, and their count of
//                         thread blocks (producer warps) that have drawn their last number
//   [8 nt + 32, + 4 nt)   changed blocks before each tile of the units that go through the receiver's prefix kernel
// Sender, transport and receiver each need their counters all zero when they start and leave them so (the last
// thread block to finish clears them), so that no call needs a clearing launch in front of its kernel; transport
// and receiver touch nothing of the sender's, and the per-tile counts need no initial value.
__host__ __device__ inline size_t workspace_sender_counters_offset(size_t nt) { return nt * sizeof(unsigned long long); }
__host__ __device__ inline size_t workspace_ticket_offset(size_t nt) { return workspace_sender_counters_offset(nt) + 16; }
__host__ __device__ inline size_t workspace_prefix_offset(size_t nt) { return workspace_ticket_offset(nt) + 16; }
__host__ __device__ inline size_t workspace_total_bytes(size_t nt) {
    return (workspace_prefix_offset(nt) + nt * sizeof(uint32_t) + 15) / 16 * 16;
}

// The tile table lists the tiles of "short" units (up to this many tiles) first, longest units
// first, then the tiles of the longer units.  The encode kernel lets one thread block work through
// a short unit tile after tile (the tile's place in the payload is then a running sum inside the
// block) and spreads everything else tile by tile over all blocks.
constexpr uint32_t kSeqMaxTiles = 32;
// A short unit is handed out in runs of this many tiles (all units' first runs, then all second runs, ...): the
// smaller the piece of work a thread block draws, the less the blocks differ in when they finish.  A run's first
// tile takes its payload offset from the status word that the run before it left.  A multiple of 4, so that tiles
// sharing a bitmap byte (blocks of 2048 and 4096 values) stay in one run.
constexpr uint32_t kSeqRunTiles = 4;

// Bytes of a message slot that tile j of a unit moves in the transport kernel: [j * chunk,
// (j + 1) * chunk); the unit's last tile also moves whatever lies beyond (pads and, for coarse
// blocks, the bitmap: less than 100 bytes per unit plus one bitmap byte per 8 blocks).  With fine
// blocks the bitmap is a sizeable part of the message, so the chunk grows by a tile's share of it.
__host__ __device__ inline uint64_t transport_chunk_bytes(uint32_t sm_bytes_per_value, uint32_t log2b) {
    const uint64_t bitmap_share = is_fine(log2b) ? pad16((uint64_t)kTileValues >> (log2b + 3)) : 0;
    return (uint64_t)kTileValues * (sm_bytes_per_value + 1) + bitmap_share;
}

}  // namespace ciera

// The plan object behind the opaque handle.
struct ciera_plan {
    int dtype = 0;
    uint32_t block = 0;
    uint32_t log2b = 0;
    uint32_t n_units = 0;
    uint64_t total_values = 0;
    bool has_empty_units = false;
    std::vector<ciera_unit> units;
    std::vector<ciera::TileDesc> tiles;
    std::vector<uint32_t> long_units;  // first tile of every unit whose decode needs the prefix kernel
    std::vector<uint32_t> seq_first;   // first tile of every short unit, in table order, + end marker
    struct SeqRun {
        uint32_t lo, hi;               // tiles [lo, hi) of the table
    };
    std::vector<SeqRun> seq_runs;      // the short units' runs of tiles in the order they are handed out
    std::vector<uint32_t> unit_first;  // first tile of every unit (0xffffffff: a unit without values)
    std::vector<uint64_t> hash_base;   // index of every unit's first block in a per-block hash cache
    std::vector<uint64_t> tile_hash;   // the same for every tile's first block, in tile-table order
    uint64_t total_blocks = 0;
    std::vector<uint64_t> seg_base;    // index of every unit's first 4096-byte payload segment (entropy stage)
    uint64_t total_segments = 0;
    uint64_t cache_extent = 0;         // max over units of cache_off + n_values
    // entropy stage: units of more than 64 segment slots, and their chunks of 64 slots
    // {unit, first segment of the chunk inside the unit, index among the long units, 0}
    struct EntChunk {
        uint32_t unit, first_seg, long_index, zero;
    };
    std::vector<uint32_t> ent_long_units;
    std::vector<EntChunk> ent_chunks;
    const uint32_t* ent_long_units_dev = nullptr;
    const uint4* ent_chunks_dev = nullptr;
    std::vector<uint8_t> image;        // device image: tiles, long_units, seq_first, hash_base, unit_first, seg_base, units,
                                       // ent_long_units, ent_chunks, tile_hash, seq_runs
    const ciera::TileDesc* tiles_dev = nullptr;
    const uint32_t* long_units_dev = nullptr;
    const uint32_t* seq_first_dev = nullptr;
    const uint2* seq_runs_dev = nullptr;
    const unsigned long long* hash_base_dev = nullptr;
    const unsigned long long* tile_hash_dev = nullptr;
    const uint32_t* unit_first_dev = nullptr;
    const unsigned long long* seg_base_dev = nullptr;
    const ciera_unit* units_dev = nullptr;
};

namespace ciera {
int record_cuda_error(cudaError_t e);          // stores e for ciera_last_cuda_error, returns CIERA_ERR_CUDA
void count_launch();                           // launch accounting
int check_launch();                            // cudaGetLastError -> status
// the persistent sender kernel with HashCache in place of the exponent cache (ciera_encode.cu)
int launch_encode_hashed(const ciera_plan* p, const void* weights_dev, void* hash_cache_dev, void* messages_dev,
                         uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* scratch, int32_t* status_dev,
                         cudaStream_t s);
}  // namespace ciera
