// Sender side with hash-based change detection (paper Section 3.1 and Algorithm 1 as printed: the
// sender keeps HashCache[i,k], a 128-bit hash per block, instead of the previous exponents): the
// entry points, and the kernel that fills HashCache at start-up.  The sender step itself is the
// persistent kernel of ciera_encode.cu in its HashCache form; the hash is defined in ciera_hash.cuh.
//
// HBM bytes per value of that step: 2 + 1 + q for bf16 (weights in; sign-plus-mantissa and the
// exponents of changed blocks out), against 4 + 2 q with the exponent cache, plus 16 (1 + q) / B of
// HashCache traffic; the price is about 45 integer instructions per 8 values for the two hashes.
#include "ciera_bits.cuh"
#include "ciera_hash.cuh"

namespace ciera {

// Adds the terms of one 64-bit word of exponents (at value offset v of the tile) to the sums of
// its block.  `lanes` = lanes of this warp that hold words of the same block (a power of two,
// aligned); lanes whose word does not exist pass valid = false and still take part.
__device__ __forceinline__ void add_word_terms(unsigned long long (*sums)[2], uint32_t log2b, uint32_t lanes, uint32_t v,
                                               uint64_t x, bool valid, uint32_t lane) {
    const uint32_t j = (v & ((1u << log2b) - 1u)) >> 3;
    uint64_t a, b;
    hash_word_terms(j, x, a, b);
    if (!valid) a = b = 0ull;
    for (uint32_t o = 1; o < lanes; o <<= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    if ((lane & (lanes - 1u)) == 0 && valid) {  // a group's first lane holds the block's lowest word: valid if any is
        atomicAdd(&sums[v >> log2b][0], (unsigned long long)a);
        atomicAdd(&sums[v >> log2b][1], (unsigned long long)b);
    }
}

// HashCache := Hash128 of every block of one tile (weights may be null: exponents all zero).  One
// thread block per tile; thread b finishes block b (a tile has at most 512 blocks).
template <int DT>
__global__ void __launch_bounds__(kThreads)
hash_cache_init_kernel(const TileDesc* __restrict__ tiles, const unsigned long long* __restrict__ tile_hash, uint32_t log2b,
                       const uint8_t* __restrict__ weights, ulonglong2* hash_cache) {
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    __shared__ unsigned long long sums[kTileValues / 16][2];  // up to 512 blocks per tile
    const uint32_t tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31u;
    const TileDesc td = load_tile_desc(tiles + tile);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const uint32_t B = 1u << log2b;
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nblk = (nv + B - 1u) >> log2b;
    for (uint32_t b = tid; b < nbt; b += kThreads) sums[b][0] = sums[b][1] = 0ull;
    __syncthreads();

    // lanes of a warp that share a block: a lane holds P::kValues consecutive values
    const uint32_t lanes = min(32u, B >> P::kLog2Values);
#pragma unroll
    for (int p = 0; p < P::kPerThread; ++p) {
        const uint32_t t0 = P::start(tid, p);
        const int nvalid = piece_valid<DT>(t0, nv);
        P x;
#pragma unroll
        for (int i = 0; i < P::kExpWords; ++i) x.e[i] = 0;
        if (nvalid > 0 && weights != nullptr) {
            if (nvalid == P::kValues)
                x.template split_full<Global>(weights + td.w_off + (uint64_t)t0 * VB);
            else
                x.split_partial(weights + td.w_off + (uint64_t)t0 * VB, nvalid);
        }
#pragma unroll
        for (int w = 0; w < P::kExpWords / 2; ++w) {
            const uint64_t word = (uint64_t)x.e[2 * w] | ((uint64_t)x.e[2 * w + 1] << 32);
            add_word_terms(sums, log2b, lanes, t0 + 8u * w, word, nvalid > 8 * w, lane);
        }
    }
    __syncthreads();
    if (tid < nblk)
        hash_cache[tile_hash[tile] + tid] = hash_finish(sums[tid][0], sums[tid][1], min(B, nv - (tid << log2b)));
}

}  // namespace ciera

using namespace ciera;

static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

static int check_hashed_plan(const ciera_plan* p) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    if (is_fine(p->log2b)) return CIERA_ERR_UNSUPPORTED;  // blocks of fewer than 16 values: exact comparison only
    return CIERA_OK;
}

extern "C" int ciera_hash_cache_init(const ciera_plan* p, void* hash_cache_dev, const void* weights_dev, void* stream) {
    int rc = check_hashed_plan(p);
    if (rc) return rc;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    if (!hash_cache_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(hash_cache_dev) || misaligned16(weights_dev)) return CIERA_ERR_MISALIGNED;
    cudaStream_t s = (cudaStream_t)stream;
    if (p->dtype == CIERA_FP16)
        hash_cache_init_kernel<CIERA_FP16><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->tile_hash_dev, p->log2b,
                                                                   (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev);
    else if (p->dtype == CIERA_BF16)
        hash_cache_init_kernel<CIERA_BF16><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->tile_hash_dev, p->log2b,
                                                                   (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev);
    else
        hash_cache_init_kernel<CIERA_FP32><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->tile_hash_dev, p->log2b,
                                                                   (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev);
    count_launch();
    return check_launch();
}

extern "C" int ciera_encode_hashed(const ciera_plan* p, const void* weights_dev, void* hash_cache_dev, void* messages_dev,
                                   uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* workspace_dev,
                                   int32_t* status_dev, void* stream) {
    int rc = check_hashed_plan(p);
    if (rc) return rc;
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
    if (!weights_dev || !hash_cache_dev || !messages_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(weights_dev) || misaligned16(hash_cache_dev) || misaligned16(messages_dev) ||
        misaligned16(workspace_dev) || ((uintptr_t)wire_bytes_dev & 7u) || ((uintptr_t)changed_blocks_dev & 3u))
        return CIERA_ERR_MISALIGNED;
    // scratch as for ciera_encode: all zero on entry (ciera_workspace_init, or left so by the previous call)
    return launch_encode_hashed(p, weights_dev, hash_cache_dev, messages_dev, wire_bytes_dev, changed_blocks_dev,
                                workspace_dev, status_dev, s);
}
