// Pieces shared by the senders that work in several plain launches (the hashed sender, the fp16
// sender): a scan pass leaves a record per tile in the scratch (block flags and their count), a
// pass per unit turns the counts into payload offsets and writes what belongs to the unit as a
// whole, a payload pass sends the exponents of the flagged blocks.  Nothing waits inside a kernel.
#pragma once

#include "ciera_bits.cuh"

namespace ciera {

// Scratch record of a tile: 16 words of block flags, the number of set flags, and the number of
// set flags in the unit's earlier tiles.
constexpr uint32_t kFlagWords = kBitmapWords;
constexpr uint32_t kRecCount = kFlagWords, kRecPrefix = kFlagWords + 1, kRecWords = kFlagWords + 2;

__device__ __forceinline__ uint32_t block_flag(const uint32_t* ws, uint32_t first_tile, uint32_t log2b, uint64_t k) {
    const uint32_t nbt = kTileValues >> log2b;
    const uint64_t t = k / nbt;
    const uint32_t r = (uint32_t)(k % nbt);
    return (ws[(size_t)(first_tile + t) * kRecWords + (r >> 5)] >> (r & 31u)) & 1u;
}

// One thread block per unit: payload offset of every tile, bitmap bytes, pads, reported totals.
static __global__ void __launch_bounds__(256)
multipass_unit_kernel(const TileDesc* __restrict__ tiles, const uint32_t* __restrict__ unit_first, uint32_t log2b,
                      int dtype, uint8_t* msgs, uint32_t* ws, unsigned long long* __restrict__ wire_bytes,
                      uint32_t* __restrict__ changed_blocks) {
    __shared__ uint32_t s_warp[8];
    __shared__ uint32_t s_carry;
    const uint32_t unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t first = unit_first[unit];
    if (first == 0xffffffffu) {  // a unit without values
        if (tid == 0) {
            wire_bytes[unit] = 0;
            changed_blocks[unit] = 0;
        }
        return;
    }
    const TileDesc td0 = load_tile_desc(tiles + first);
    const uint64_t N = td0.n_unit;
    const uint32_t B = 1u << log2b;
    const uint32_t nbt = kTileValues >> log2b;
    const uint64_t nb = num_blocks(N, log2b);
    uint8_t* msg = msgs + td0.msg_off;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (uint32_t j0 = 0; j0 < td0.n_tiles_unit; j0 += 256u) {
        const uint32_t j = j0 + tid;
        const uint32_t cnt = j < td0.n_tiles_unit ? ws[(size_t)(first + j) * kRecWords + kRecCount] : 0u;
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
        if (j < td0.n_tiles_unit) ws[(size_t)(first + j) * kRecWords + kRecPrefix] = carry + wbase + incl - cnt;
        __syncthreads();
        if (tid == 255) s_carry = carry + wbase + incl;
        __syncthreads();
    }
    const uint64_t smoff = sm_offset(N, log2b);
    const uint64_t sm_bytes = sm_section_bytes(N, dtype);
    const uint64_t payoff = smoff + pad16(sm_bytes);
    if (tid == 0) {
        const uint32_t total = s_carry;  // changed blocks of the unit
        uint64_t bytes = (uint64_t)total * block_payload_bytes(B, dtype);
        const uint32_t rem = (uint32_t)(N & (B - 1u));
        if (rem && block_flag(ws, first, log2b, nb - 1))  // a changed short last block
            bytes -= block_payload_bytes(B, dtype) - block_payload_bytes(rem, dtype);
        wire_bytes[unit] = payoff + bytes;
        changed_blocks[unit] = total;
    }
    // bitmap bytes (bit k of the unit = block k, LSB first), then the two pads
    const uint64_t bm_bytes = bitmap_bytes(N, log2b);
    for (uint64_t i = tid; i < bm_bytes; i += 256u) {
        uint32_t byte = 0;
        if (nbt >= 32) {  // the byte's eight flags lie in one word of one tile
            const uint64_t k = 8 * i;
            const uint32_t r = (uint32_t)(k % nbt);
            byte = (ws[(size_t)(first + k / nbt) * kRecWords + (r >> 5)] >> (r & 31u)) & 0xFFu;
        } else {
            for (uint32_t r = 0; r < 8; ++r)
                if (8 * i + r < nb) byte |= block_flag(ws, first, log2b, 8 * i + r) << r;
        }
        msg[i] = (uint8_t)byte;
    }
    for (uint64_t b = bm_bytes + tid; b < smoff; b += 256u) msg[b] = 0;
    for (uint64_t b = smoff + sm_bytes + tid; b < payoff; b += 256u) msg[b] = 0;
}

}  // namespace ciera
