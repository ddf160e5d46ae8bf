// Single-pass decoupled look-back over per-tile status words: how a tile learns where its changed
// exponents start in its unit's payload (the sum of the payload bytes of the unit's earlier tiles)
// without a second pass.  Shared by the two sender kernels.
//
// Every wait is bounded: after kMaxPolls reads of a status word the waiting warp gives up, raises
// CIERA_ERR_TIMEOUT and carries on with offset 0 (output unspecified) instead of hanging.
#pragma once

#include "ciera_internal.cuh"

namespace ciera {

__device__ __forceinline__ unsigned long long ld_status(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_status(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Polls a tile status word until its flag is set.  Bounded: after max_polls reads (kMaxPolls in the
// kernels; the self-test passes a few dozen) it gives up, raises CIERA_ERR_TIMEOUT and returns
// "prefix 0" so that the caller finishes (with unspecified output) instead of hanging.
__device__ __forceinline__ unsigned long long wait_status(const unsigned long long* p, int32_t* status,
                                                          uint32_t max_polls = kMaxPolls) {
    unsigned long long st = ld_status(p);
    uint32_t polls = 0;
    while ((st >> 62) == 0) {
        if (++polls > max_polls) {
            if (status) atomicCAS(status, 0, (int32_t)CIERA_ERR_TIMEOUT);
            return kFlagPrefix;
        }
        if (polls > 16) __nanosleep(polls > 1024 ? 400 : 40);
        st = ld_status(p);
    }
    return st;
}

__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// The unit's last tile reports the totals and zeroes the two pads (one warp).
template <int DT>
__device__ __forceinline__ void finish_unit(const TileDesc& td, uint32_t log2b, uint64_t total, uint8_t* msgs,
                                            unsigned long long* wire_bytes, uint32_t* changed_blocks, uint32_t lane) {
    const uint64_t N = td.n_unit;
    uint8_t* msg = msgs + td.msg_off;
    const uint64_t smoff = sm_offset(N, log2b);
    const uint64_t sm_bytes = sm_section_bytes(N, DT);
    const uint64_t payoff = smoff + pad16(sm_bytes);
    if (lane == 0) {
        wire_bytes[td.unit] = payoff + total;
        // every changed block carries a full block's bytes except possibly the last one, which carries fewer
        if (DT == CIERA_FP16) {
            const uint64_t bpb = payload_bytes_of_blocks<DT>(1, log2b);
            changed_blocks[td.unit] = (uint32_t)((total + bpb - 1u) / bpb);
        } else {
            changed_blocks[td.unit] = (uint32_t)((total + (1ull << log2b) - 1u) >> log2b);
        }
    }
    for (uint64_t b = bitmap_bytes(N, log2b) + lane; b < smoff; b += 32) msg[b] = 0;
    for (uint64_t b = smoff + sm_bytes + lane; b < payoff; b += 32) msg[b] = 0;
}

// Resolver warp, one spread tile: exclusive prefix of the payload bytes over the earlier tiles of
// the same unit by a single-pass look-back over the status words, then the duties that need it.
// Returns the tile's exclusive payload offset inside its unit.
template <int DT>
__device__ __forceinline__ uint64_t resolve_tile(const TileDesc& td, uint32_t tile, uint32_t log2b, uint64_t agg,
                                                 const uint32_t* bm, uint8_t* msgs, unsigned long long* wire_bytes,
                                                 uint32_t* changed_blocks, unsigned long long* tile_status,
                                                 int32_t* status, uint32_t lane) {
    const uint32_t nbt = kTileValues >> log2b;
    uint8_t* msg = msgs + td.msg_off;
    const uint32_t mybits = nbt < 8 ? bm[0] : 0u;

    uint64_t excl = 0;
    if (td.tile_in_unit != 0) {
        int64_t hi = (int64_t)tile - 1;
        while (true) {
            const int64_t idx = hi - (int64_t)lane;
            unsigned long long st = kFlagPrefix;  // "prefix 0" stands before the unit's first tile
            if (idx >= (int64_t)td.first_tile) st = wait_status(tile_status + idx, status);
            __syncwarp();
            const uint32_t pmask = __ballot_sync(0xffffffffu, (st >> 62) == 2ull);
            const uint32_t first = pmask ? (uint32_t)__ffs(pmask) - 1u : 31u;
            excl += warp_sum_u64(lane <= first ? (st & kValueMask) : 0ull);
            if (pmask) break;
            hi -= 32;
        }
        if (lane == 0)
            st_status(tile_status + tile, kFlagPrefix | ((unsigned long long)mybits << kBitsShift) | (excl + agg));
    }

    // tiles of fewer than 8 blocks share a bitmap byte: the last tile of each byte collects the
    // bits its predecessors published in their status words
    if (nbt < 8) {
        const uint32_t tpb = 8u / nbt;
        const uint32_t p = td.tile_in_unit & (tpb - 1u);
        if (p == tpb - 1u || td.tile_in_unit == td.n_tiles_unit - 1u) {
            uint32_t part = 0;
            if (lane < p) {
                unsigned long long st = wait_status(tile_status + (tile - p + lane), status);
                part = (uint32_t)((st >> kBitsShift) & 0x3Full) << (lane * nbt);
            }
            __syncwarp();
            part = __reduce_or_sync(0xffffffffu, part);
            if (lane == 0) msg[td.tile_in_unit / tpb] = (uint8_t)(part | (mybits << (p * nbt)));
        }
    }
    if (td.tile_in_unit == td.n_tiles_unit - 1u)
        finish_unit<DT>(td, log2b, excl + agg, msgs, wire_bytes, changed_blocks, lane);
    return excl;
}

}  // namespace ciera
