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
//   receiver  the persistent decode kernel of the other precisions, instantiated for fp16
//             (ciera_decode.cu; the bit work is Piece<CIERA_FP16> in ciera_bits.cuh).
// Blocks of 32 values and more (four pieces), so that the four lanes that share 44 bytes of packed
// sign-plus-mantissa always lie in one block.
#include "ciera_bits.cuh"
#include "ciera_multipass.cuh"

namespace ciera {

using H = Piece<CIERA_FP16>;

__device__ __forceinline__ int h_valid(uint32_t t0, uint32_t nv) { return t0 >= nv ? 0 : (int)min(8u, nv - t0); }

// ------------------------------------------------------------------------------------------
// cache := exponents(weights) (or zero)

__global__ void __launch_bounds__(kThreads)
fp16_cache_fill_kernel(const TileDesc* __restrict__ tiles, const uint8_t* __restrict__ weights, uint8_t* __restrict__ cache) {
    const TileDesc td = load_tile_desc(tiles + blockIdx.x);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const uint32_t t0 = H::start(threadIdx.x, p);
        const int nvalid = h_valid(t0, nv);
        if (nvalid == 0) continue;
        H x;
        x.e[0] = x.e[1] = 0;
        if (weights != nullptr) {
            if (nvalid == 8)
                x.split_full<Global>(weights + td.w_off + (uint64_t)t0 * 2);
            else
                x.split_partial(weights + td.w_off + (uint64_t)t0 * 2, nvalid);
        }
        if (nvalid == 8)
            x.store_exp_full<Global>(cache + td.c_off + t0);
        else
            x.store_exp_partial(cache + td.c_off + t0, nvalid);
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
        const uint32_t t0 = H::start(tid, p);
        const int nvalid = h_valid(t0, nv);
        H x, c;
        x.e[0] = x.e[1] = x.s[0] = x.s[1] = x.s[2] = 0;
        bool diff = false;
        if (nvalid == 8) {
            x.split_full<Global>(weights + td.w_off + (uint64_t)t0 * 2);
            c.load_exp_full<Global>(cache + td.c_off + t0);
            diff = x.differs(c);
            // cache refreshed where it differs (the other pieces of a changed block hold the same bytes already)
            if (diff) x.store_exp_full<Global>(cache + td.c_off + t0);
        } else if (nvalid > 0) {
            x.split_partial(weights + td.w_off + (uint64_t)t0 * 2, nvalid);
            c.load_exp_partial(cache + td.c_off + t0, nvalid);
            diff = x.differs(c);
            if (diff) x.store_exp_partial(cache + td.c_off + t0, nvalid);
        }
        // packed sign-plus-mantissa: whole groups of four lanes in a full tile, else byte by byte
        if (full_tile)
            x.store_sm_group(section, t0 >> 3, lane);
        else if (nvalid > 0)
            x.store_sm_bytes(section + (size_t)11 * (t0 >> 3), nvalid);
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
        const uint32_t kb = H::start(tid, p) >> log2b;
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
        const uint32_t kb = H::start(tid, p) >> log2b;
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
        const uint32_t t0 = H::start(tid, p);
        const int nvalid = h_valid(t0, nv);
        if (!flagged[p] || nvalid == 0) continue;
        uint32_t lo, hi;
        H x;
        if (nvalid == 8)
            x.split_full<Global>(weights + td.w_off + (uint64_t)t0 * 2);
        else
            x.split_partial(weights + td.w_off + (uint64_t)t0 * 2, nvalid);
        x.pack_exponents(lo, hi);
        uint8_t* dst = pay + (uint64_t)rank[p] * bpb + 5u * ((t0 & (B - 1u)) >> 3);
        const int nbytes = (5 * nvalid + 7) >> 3;
        for (int i = 0; i < nbytes; ++i) dst[i] = (uint8_t)(i < 4 ? lo >> (8 * i) : hi);
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

}  // namespace ciera
