// Sender side with hash-based change detection (paper Section 3.1 and Algorithm 1 as printed: the
// sender keeps HashCache[i,k], a 128-bit hash per block, instead of the previous exponents).
//
// The paper fixes only that the hash has 128 bits and is built from two independent 64-bit
// SplitMix64 hashes.  The construction used here:
//   mix(z)  = the SplitMix64 output function, gamma = its increment 0x9E3779B97F4A7C15;
//   a block of L exponent bytes is read as ceil(L / 8) little-endian 64-bit words x_j (the last
//   one zero-padded);  H_s = mix(L + sum_j mix(s + (j + 1) * gamma + x_j))  (mod 2^64);
//   Hash128 = (H_s1, H_s2) with s1 = 0 and s2 = 0x6A09E667F3BCC908.
// The per-word terms are summed, so the threads holding a block's words can be combined in any
// order: a shuffle reduction inside the warp, then a shared-memory atomic per warp and block.
//
// Three plain launches per call (no waiting between thread blocks anywhere):
//   scan     one thread block per tile: split, sign-plus-mantissa out, block hashes, compare with
//            HashCache and refresh it; leaves the tile's block flags and their count in the scratch;
//   unit     one thread block per unit: per-tile payload offsets (running count over the unit's
//            tiles), the unit's bitmap bytes, pads, reported length and changed-block count;
//   payload  one thread block per tile: the exponents of the flagged blocks (their weights are read
//            a second time) go to their place in the payload.
// HBM bytes per value: 2 + 1 (scan) and 3 q (payload) for bf16, against 4 + 2 q with the exponent
// cache, plus 16 bytes per block of HashCache traffic; the price is about 40 integer instructions
// per 8 values for the two hashes.
#include "ciera_bits.cuh"
#include "ciera_multipass.cuh"

namespace ciera {

constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kSeed1 = 0x0000000000000000ull;
constexpr uint64_t kSeed2 = 0x6A09E667F3BCC908ull;
__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

// Adds the terms of one 64-bit word of exponents (at value offset v of the tile) to the sums of
// its block.  `lanes` = lanes of this warp that hold words of the same block (a power of two,
// aligned); lanes whose word does not exist pass valid = false and still take part.
__device__ __forceinline__ void add_word_terms(unsigned long long (*sums)[2], uint32_t log2b, uint32_t lanes, uint32_t v,
                                               uint64_t x, bool valid, uint32_t lane) {
    const uint32_t j = (v & ((1u << log2b) - 1u)) >> 3;
    uint64_t a = valid ? mix64(kSeed1 + (uint64_t)(j + 1u) * kGamma + x) : 0ull;
    uint64_t b = valid ? mix64(kSeed2 + (uint64_t)(j + 1u) * kGamma + x) : 0ull;
    for (uint32_t o = 1; o < lanes; o <<= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    if ((lane & (lanes - 1u)) == 0 && valid) {  // a group's first lane holds the block's lowest word: valid if any is
        atomicAdd(&sums[v >> log2b][0], (unsigned long long)a);
        atomicAdd(&sums[v >> log2b][1], (unsigned long long)b);
    }
}

// Hashes of the blocks of one tile.  INIT: HashCache := hashes (weights may be null: exponents
// all zero).  Otherwise the scan pass described at the head of this file.
template <int DT, bool INIT>
__global__ void __launch_bounds__(kThreads)
hashed_scan_kernel(const TileDesc* __restrict__ tiles, const unsigned long long* __restrict__ hash_base, uint32_t log2b,
                   const uint8_t* __restrict__ weights, ulonglong2* hash_cache, uint8_t* msgs, uint32_t* ws) {
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;
    __shared__ unsigned long long sums[kTileValues / 16][2];  // up to 512 blocks per tile
    __shared__ uint32_t s_count;
    const uint32_t tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31u;
    const TileDesc td = load_tile_desc(tiles + tile);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const uint32_t B = 1u << log2b;
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nblk = (nv + B - 1u) >> log2b;

    // the cached hash of "my" block (thread b takes block b, nbt <= 512) is fetched first, so that
    // its latency passes while the tile is hashed
    const unsigned long long kglob = hash_base[td.unit] + (unsigned long long)td.tile_in_unit * nbt;
    ulonglong2 old = make_ulonglong2(0ull, 0ull);
    if (!INIT && tid < nblk) old = hash_cache[kglob + tid];
    for (uint32_t b = tid; b < nbt; b += kThreads) sums[b][0] = sums[b][1] = 0ull;
    if (tid == 0) s_count = 0;
    __syncthreads();

    uint8_t* sm_dst = INIT ? nullptr : msgs + td.msg_off + sm_offset(td.n_unit, log2b) + v0 * SMB;
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
            if (!INIT) {
                if (nvalid == P::kValues)
                    x.template store_sm_full<Global>(sm_dst + (size_t)t0 * SMB);
                else
                    x.store_sm_partial(sm_dst + (size_t)t0 * SMB, nvalid);
            }
        }
#pragma unroll
        for (int w = 0; w < P::kExpWords / 2; ++w) {
            const uint64_t word = (uint64_t)x.e[2 * w] | ((uint64_t)x.e[2 * w + 1] << 32);
            add_word_terms(sums, log2b, lanes, t0 + 8u * w, word, nvalid > 8 * w, lane);
        }
    }
    __syncthreads();

    // one thread per block: finish the two hashes and compare with HashCache
    bool changed = false;
    if (tid < nblk) {
        const uint32_t L = min(B, nv - (tid << log2b));
        ulonglong2 h;
        h.x = mix64(sums[tid][0] + L);
        h.y = mix64(sums[tid][1] + L);
        changed = old.x != h.x || old.y != h.y;
        if (INIT || changed) hash_cache[kglob + tid] = h;  // HashCache[i,k] <- h
    }
    if (INIT) return;
    const uint32_t flags = __ballot_sync(0xffffffffu, changed);
    if (lane == 0) {  // 16 warps write the tile's 16 flag words
        ws[(size_t)tile * kRecWords + (tid >> 5)] = flags;
        if (flags) atomicAdd(&s_count, (uint32_t)__popc(flags));
    }
    __syncthreads();
    if (tid == 0) ws[(size_t)tile * kRecWords + kRecCount] = s_count;
}

// One thread block per tile, every warp on its own (no barrier): exponents of the flagged blocks to
// the payload.  A warp first looks at the flags of its own pieces and leaves if none is set;
// otherwise it works out the ranks from the tile's scratch record with shuffles and fetches the
// weights of its flagged pieces a second time.
template <int DT>
__global__ void __launch_bounds__(kThreads)
hashed_payload_kernel(const TileDesc* __restrict__ tiles, uint32_t log2b, const uint8_t* __restrict__ weights,
                      uint8_t* msgs, const uint32_t* __restrict__ ws) {
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;
    const uint32_t tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31u;
    const uint32_t* rec = ws + (size_t)tile * kRecWords;
    // which of this lane's pieces are flagged; most warps leave here
    uint32_t word[P::kPerThread];
    bool flagged[P::kPerThread];
    bool any = false;
#pragma unroll
    for (int p = 0; p < P::kPerThread; ++p) {
        const uint32_t kb = P::start(tid, p) >> log2b;
        word[p] = __ldg(rec + (kb >> 5));
        flagged[p] = (word[p] >> (kb & 31u)) & 1u;
        any |= flagged[p];
    }
    if (!__any_sync(0xffffffffu, any)) return;
    // ranks: set flags before each word of the record (every lane of the warp takes part)
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
    uint32_t rank[P::kPerThread];
#pragma unroll
    for (int p = 0; p < P::kPerThread; ++p) {
        const uint32_t kb = P::start(tid, p) >> log2b;
        rank[p] = __shfl_sync(0xffffffffu, pre_l, kb >> 5) + __popc(word[p] & ((1u << (kb & 31u)) - 1u));
    }
    if (!any) return;
    const TileDesc td = load_tile_desc(tiles + tile);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    uint8_t* pay = msgs + td.msg_off + payload_offset(td.n_unit, SMB, log2b) + ((uint64_t)prefix << log2b);
#pragma unroll
    for (int p = 0; p < P::kPerThread; ++p) {
        const uint32_t t0 = P::start(tid, p);
        const int nvalid = piece_valid<DT>(t0, nv);
        if (!flagged[p] || nvalid == 0) continue;
        uint8_t* dst = pay + ((uint64_t)rank[p] << log2b) + (t0 & ((1u << log2b) - 1u));
        P x;
        if (nvalid == P::kValues) {
            x.template split_full<Global>(weights + td.w_off + (uint64_t)t0 * VB);
            x.template store_exp_full<Global>(dst);
        } else {
            x.split_partial(weights + td.w_off + (uint64_t)t0 * VB, nvalid);
            x.store_exp_partial(dst, nvalid);
        }
    }
}

}  // namespace ciera

using namespace ciera;

static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

static int check_hashed_plan(const ciera_plan* p) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    if (is_fine(p->log2b)) return CIERA_ERR_UNSUPPORTED;  // blocks of fewer than 16 values: exact comparison only
    if (p->dtype == CIERA_FP16) return CIERA_ERR_UNSUPPORTED;
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
    if (p->dtype == CIERA_BF16)
        hashed_scan_kernel<CIERA_BF16, true><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->hash_base_dev, p->log2b,
                                                                     (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev,
                                                                     nullptr, nullptr);
    else
        hashed_scan_kernel<CIERA_FP32, true><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->hash_base_dev, p->log2b,
                                                                     (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev,
                                                                     nullptr, nullptr);
    count_launch();
    return check_launch();
}

extern "C" int ciera_encode_hashed(const ciera_plan* p, const void* weights_dev, void* hash_cache_dev, void* messages_dev,
                                   uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* workspace_dev,
                                   void* stream) {
    int rc = check_hashed_plan(p);
    if (rc) return rc;
    if (p->n_units == 0) return CIERA_OK;
    if (!wire_bytes_dev || !changed_blocks_dev) return CIERA_ERR_INVALID_ARG;
    const uint32_t nt = (uint32_t)p->tiles.size();
    cudaStream_t s = (cudaStream_t)stream;
    if (nt != 0) {
        if (!weights_dev || !hash_cache_dev || !messages_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
        if (misaligned16(weights_dev) || misaligned16(hash_cache_dev) || misaligned16(messages_dev) ||
            misaligned16(workspace_dev))
            return CIERA_ERR_MISALIGNED;
    }
    if (((uintptr_t)wire_bytes_dev & 7u) || ((uintptr_t)changed_blocks_dev & 3u)) return CIERA_ERR_MISALIGNED;
    // scratch: one record of 18 words per tile; the scan pass writes every record's flags and count,
    // the unit pass its payload offset
    uint32_t* ws = (uint32_t*)workspace_dev;
    if (nt != 0) {
        if (p->dtype == CIERA_BF16)
            hashed_scan_kernel<CIERA_BF16, false><<<nt, kThreads, 0, s>>>(
                p->tiles_dev, p->hash_base_dev, p->log2b, (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev,
                (uint8_t*)messages_dev, ws);
        else
            hashed_scan_kernel<CIERA_FP32, false><<<nt, kThreads, 0, s>>>(
                p->tiles_dev, p->hash_base_dev, p->log2b, (const uint8_t*)weights_dev, (ulonglong2*)hash_cache_dev,
                (uint8_t*)messages_dev, ws);
        count_launch();
        rc = check_launch();
        if (rc) return rc;
    }
    multipass_unit_kernel<<<p->n_units, 256, 0, s>>>(p->tiles_dev, p->unit_first_dev, p->log2b, p->dtype,
                                                     (uint8_t*)messages_dev, ws, (unsigned long long*)wire_bytes_dev,
                                                     changed_blocks_dev);
    count_launch();
    rc = check_launch();
    if (rc) return rc;
    if (nt != 0) {
        if (p->dtype == CIERA_BF16)
            hashed_payload_kernel<CIERA_BF16><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)weights_dev,
                                                                      (uint8_t*)messages_dev, ws);
        else
            hashed_payload_kernel<CIERA_FP32><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)weights_dev,
                                                                      (uint8_t*)messages_dev, ws);
        count_launch();
        rc = check_launch();
    }
    return rc;
}
