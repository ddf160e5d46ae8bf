// Entropy stage (paper Section 3.1; Algorithm 1: payload <- ANSEncode(...), newExp <- ANSDecode(...)):
// the exponents of changed blocks are coded with rANS between the sender step and the transport, and
// decoded between the transport and the receiver step.  The paper uses a vendor library whose
// stream format is not public; the coder and the layout here are this library's own.
//
// Model: one static table per unit, 256 symbols, probabilities in 1/4096 (f[s] = max(1,
// floor(h[s] * 4096 / P)) for the symbols that occur; a shortfall goes to the most frequent symbol,
// an excess is taken from the largest entries).
// Coder: 32-bit state x in [2^16, 2^32), 16-bit words.
//   encode s:  if x >= f[s] * 2^20: emit x mod 2^16, x >>= 16;   x <- (x / f) * 4096 + x mod f + c[s]
//   decode:    slot = x mod 4096, s = symbol of slot;  x <- f[s] * (x / 4096) + slot - c[s];
//              if x < 2^16: x <- x * 2^16 + next word
// The raw payload is cut into segments of 4096 bytes; one warp codes a segment with its 32 lanes as
// 32 interleaved coders (lane l owns bytes 32 t + l).  The encoder walks the steps t backwards and
// appends the words its lanes emit (ballot, rank = lanes below); the decoder walks forwards and
// takes the words from the end of the list backwards, so neither side needs per-lane streams.
// Coded section: [256 x u16 f] [n_seg x u32 word counts] [segments: 32 x u32 final states, words,
// 2 zero bytes if the count is odd].  It replaces the raw payload only if strictly shorter; the
// receiver knows the raw length from the bitmap and so tells the two forms apart by the length.
//
// One thread block works on one unit: nothing waits for another block anywhere.
#include "ciera_bits.cuh"

namespace ciera {

constexpr uint32_t kProbBits = 12, kProbScale = 1u << kProbBits;
constexpr uint32_t kRansL = 1u << 16;
constexpr uint32_t kSegment = 4096;                              // bytes of raw payload per segment
constexpr uint32_t kSegWordsMax = kSegment * kProbBits / 16;     // 3072: a symbol adds at most 12 bits
constexpr uint32_t kSegSlot = 4 * 32 + 2 * kSegWordsMax;         // 6272 bytes: states + words
constexpr int kEntThreads = 256, kEntWarps = kEntThreads / 32;

__host__ __device__ inline uint64_t segments_of(uint64_t bytes) { return (bytes + kSegment - 1) / kSegment; }
__host__ __device__ inline uint32_t segment_bytes(uint32_t nw) { return 4u * 32u + 2u * nw + ((nw & 1u) ? 2u : 0u); }

// ------------------------------------------------------------------------------------------ sender

__global__ void __launch_bounds__(kEntThreads)
entropy_encode_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                      uint32_t sm_bytes_per_value, uint32_t log2b, uint8_t* msgs, unsigned long long* wire_bytes,
                      uint8_t* scratch_slots, uint32_t* scratch_nw) {
    __shared__ __align__(16) uint8_t s_seg[kEntWarps][kSegment];  // a warp's segment of raw payload
    __shared__ uint32_t s_hist[kEntWarps][256];
    __shared__ uint16_t s_f[256], s_c[256];
    __shared__ unsigned long long s_rcp[256];  // ceil(2^64 / f): floor(x / f) = high half of x * rcp, exact for x < 2^32
    __shared__ uint32_t s_scan[kEntWarps];
    __shared__ unsigned long long s_total;
    const uint32_t unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[unit];
    if (un.n_values == 0) return;
    const uint64_t payoff = payload_offset(un.n_values, sm_bytes_per_value, log2b);
    const uint64_t P = wire_bytes[unit] - payoff;
    if (P == 0 || P >= (1ull << 32)) return;  // nothing to code (or too much for 32-bit counts: stays raw)
    uint8_t* const pay = msgs + un.msg_off + payoff;  // 16-byte aligned
    const uint32_t nseg = (uint32_t)segments_of(P);

    // 1. histogram of the raw payload (one private copy per warp)
    for (uint32_t i = lane; i < 256; i += 32) s_hist[warp][i] = 0;
    __syncwarp();
    for (uint64_t i = (uint64_t)tid * 16; i < P; i += (uint64_t)kEntThreads * 16) {
        if (i + 16 <= P) {
            const uint4 v = *reinterpret_cast<const uint4*>(pay + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 16; ++k) atomicAdd(&s_hist[warp][(w[k >> 2] >> (8 * (k & 3))) & 0xFFu], 1u);
        } else {
            for (uint64_t k = i; k < P; ++k) atomicAdd(&s_hist[warp][pay[k]], 1u);
        }
    }
    __syncthreads();
    // 2. the model: thread s owns symbol s
    {
        uint32_t h = 0;
        for (int w = 0; w < kEntWarps; ++w) h += s_hist[w][tid];
        uint32_t f = 0;
        if (h) {
            f = (uint32_t)((uint64_t)h * kProbScale / P);
            if (f == 0) f = 1;
        }
        s_hist[0][tid] = h;  // every thread has read all copies of its own symbol only
        s_f[tid] = (uint16_t)f;
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t sum = 0, best = 0;
        for (uint32_t s = 0; s < 256; ++s) {
            sum += s_f[s];
            if (s_hist[0][s] > s_hist[0][best]) best = s;
        }
        if (sum < kProbScale) {
            s_f[best] = (uint16_t)(s_f[best] + (kProbScale - sum));
        } else {
            uint32_t excess = sum - kProbScale;
            while (excess) {
                uint32_t big = 0;
                for (uint32_t s = 1; s < 256; ++s)
                    if (s_f[s] > s_f[big]) big = s;
                const uint32_t take = min((uint32_t)s_f[big] - 1u, excess);
                s_f[big] = (uint16_t)(s_f[big] - take);
                excess -= take;
            }
        }
        uint32_t run = 0;
        for (uint32_t s = 0; s < 256; ++s) {
            s_c[s] = (uint16_t)run;
            run += s_f[s];
        }
        s_total = 0;
    }
    __syncthreads();
    // x / f through a multiplication: rcp = ceil(2^64 / f) exceeds 2^64 / f by less than 1, so for
    // x < 2^32 the product x * rcp / 2^64 exceeds x / f by less than 2^-32 -- too little to reach the
    // next integer, because the fraction of x / f is at most 1 - 1/4096.  (f = 1 is handled apart.)
    s_rcp[tid] = s_f[tid] > 1 ? (~0ull) / s_f[tid] + 1ull : 0ull;
    __syncthreads();

    // 3. segments: warp w codes segments w, w + 8, ... into the unit's slots of the scratch
    const unsigned long long slot0 = seg_base[unit];
    for (uint32_t g = warp; g < nseg; g += kEntWarps) {
        const uint32_t n = (uint32_t)min((uint64_t)kSegment, P - (uint64_t)g * kSegment);
        const uint8_t* src = pay + (uint64_t)g * kSegment;
        for (uint32_t i = lane * 16; i < n; i += 32 * 16) {
            if (i + 16 <= n) {
                *reinterpret_cast<uint4*>(&s_seg[warp][i]) = *reinterpret_cast<const uint4*>(src + i);
            } else {
                for (uint32_t k = i; k < n; ++k) s_seg[warp][k] = src[k];
            }
        }
        __syncwarp();
        uint8_t* slot = scratch_slots + (slot0 + g) * kSegSlot;
        uint16_t* words = reinterpret_cast<uint16_t*>(slot + 4 * 32);
        uint32_t x = kRansL, nw = 0;
        const uint32_t steps = (n + 31u) >> 5;
        for (uint32_t t = steps; t-- > 0;) {
            const uint32_t i = 32u * t + lane;
            const bool has = i < n;
            const uint32_t s = has ? s_seg[warp][i] : 0u;
            const uint32_t f = has ? s_f[s] : 1u, c = s_c[s];
            const bool emit = has && (x >> 20) >= f;  // x >= f * 2^20
            const uint32_t votes = __ballot_sync(0xffffffffu, emit);
            if (emit) {
                words[nw + __popc(votes & ((1u << lane) - 1u))] = (uint16_t)x;
                x >>= 16;
            }
            nw += __popc(votes);
            if (has) {
                const uint32_t q = f > 1 ? (uint32_t)__umul64hi((unsigned long long)x, s_rcp[s]) : x;
                x = q * kProbScale + (x - q * f) + c;
            }
        }
        reinterpret_cast<uint32_t*>(slot)[lane] = x;
        if (lane == 0) {
            if (nw & 1u) words[nw] = 0;
            scratch_nw[slot0 + g] = nw;
            atomicAdd(&s_total, (unsigned long long)segment_bytes(nw));
        }
        __syncwarp();
    }
    __threadfence_block();
    __syncthreads();  // every warp is done reading the raw payload and writing its slots

    // 4. keep the raw form unless the coded one is strictly shorter; else move it into the message
    const uint64_t C = 512ull + 4ull * nseg + s_total;
    if (C >= P) return;
    uint16_t* table = reinterpret_cast<uint16_t*>(pay);
    table[tid] = s_f[tid];
    uint32_t* dir = reinterpret_cast<uint32_t*>(pay + 512);
    uint8_t* data = pay + 512 + 4ull * nseg;
    uint64_t carry = 0;  // bytes of the segments before this chunk (same in every thread)
    for (uint32_t g0 = 0; g0 < nseg; g0 += kEntThreads) {
        const uint32_t g = g0 + tid;
        const uint32_t nw = g < nseg ? scratch_nw[slot0 + g] : 0u;
        const uint32_t size = g < nseg ? segment_bytes(nw) : 0u;
        if (g < nseg) dir[g] = nw;
        // exclusive scan of the sizes over the chunk
        uint32_t incl = size;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += v;
        }
        if (lane == 31) s_scan[warp] = incl;
        __syncthreads();
        uint32_t wbase = 0, chunk_total = 0;
        for (int w = 0; w < kEntWarps; ++w) {
            if (w < (int)warp) wbase += s_scan[w];
            chunk_total += s_scan[w];
        }
        // park (offset, size) of the chunk's segments where the warps can read them
        uint32_t* s_off = &s_hist[1][0];
        uint32_t* s_size = &s_hist[2][0];
        s_off[tid] = wbase + incl - size;
        s_size[tid] = size;
        __syncthreads();
        const uint32_t in_chunk = min((uint32_t)kEntThreads, nseg - g0);
        for (uint32_t k = warp; k < in_chunk; k += kEntWarps) {
            const uint32_t* from = reinterpret_cast<const uint32_t*>(scratch_slots + (slot0 + g0 + k) * kSegSlot);
            uint32_t* to = reinterpret_cast<uint32_t*>(data + carry + s_off[k]);
            for (uint32_t i = lane; i < (s_size[k] >> 2); i += 32) to[i] = from[i];
        }
        carry += chunk_total;
        __syncthreads();
    }
    if (tid == 0) wire_bytes[unit] = payoff + C;
}

// ---------------------------------------------------------------------------------------- receiver

struct DecodeShared {
    uint8_t sym[kProbScale];       // slot -> symbol
    uint16_t f[256], c[256];
    uint32_t off[kEntThreads];     // per segment of a chunk: byte offset in the data part
    uint32_t nw[kEntThreads];      //                         word count
    uint32_t scan[kEntWarps];
    unsigned long long changed;    // set bits of the unit's bitmap
    uint32_t bad;
    __align__(16) uint8_t seg[kEntWarps][kSegSlot];  // a warp's coded segment
};

__global__ void __launch_bounds__(kEntThreads)
entropy_decode_kernel(const ciera_unit* __restrict__ units, uint32_t sm_bytes_per_value, uint32_t log2b, uint8_t* msgs,
                      unsigned long long* wire_bytes, uint8_t* scratch_raw, int32_t* status) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    DecodeShared& sh = *reinterpret_cast<DecodeShared*>(smem_raw);
    const uint32_t unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[unit];
    const uint64_t N = un.n_values;
    if (N == 0) return;
    uint8_t* const msg = msgs + un.msg_off;
    const uint64_t payoff = payload_offset(N, sm_bytes_per_value, log2b);
    const uint32_t B = 1u << log2b;
    if (tid == 0) {
        sh.changed = 0;
        sh.bad = 0;
    }
    __syncthreads();
    // raw payload length from the bitmap (its bits past the last block and the pad behind it are zero)
    {
        const uint64_t words = (bitmap_bytes(N, log2b) + 3) >> 2;  // inside the 16-byte padded bitmap
        const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msg);
        uint32_t cnt = 0;
        for (uint64_t i = tid; i < words; i += kEntThreads) cnt += __popc(bm32[i]);
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0 && cnt) atomicAdd(&sh.changed, (unsigned long long)cnt);
    }
    __syncthreads();
    uint64_t P = sh.changed << log2b;
    const uint32_t rem = (uint32_t)(N & (B - 1u));
    if (rem) {
        const uint64_t kb = num_blocks(N, log2b) - 1;
        if ((msg[kb >> 3] >> (kb & 7u)) & 1u) P -= (B - rem);
    }
    const uint64_t wire = wire_bytes[unit];
    if (P == 0 || wire == payoff + P) return;  // nothing travelled, or the raw form did
    const uint64_t C = wire - payoff;
    const uint32_t nseg = (uint32_t)segments_of(P);
    const uint8_t* const pay = msg + payoff;
    if (wire < payoff || C >= P || C < 512ull + 4ull * nseg) {
        if (tid == 0 && status) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
        return;
    }
    // the model
    sh.f[tid] = reinterpret_cast<const uint16_t*>(pay)[tid];
    __syncthreads();
    if (tid == 0) {
        uint32_t run = 0;
        for (uint32_t s = 0; s < 256; ++s) {
            sh.c[s] = (uint16_t)run;  // up to 4096 behind the last symbol that occurs
            run += sh.f[s];
        }
        if (run != kProbScale) sh.bad = 1;
    }
    __syncthreads();
    if (sh.bad) {
        if (tid == 0 && status) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
        return;
    }
    // slot -> symbol: every thread looks up 16 consecutive slots.  The owner of a slot is the last
    // symbol that starts at or below it (symbols that do not occur share their start with the next
    // one, or start at 4096 behind the last occurring one): bisection over the 256 starts.
    for (uint32_t slot = tid * 16; slot < tid * 16 + 16; ++slot) {
        uint32_t lo = 0, hi = 255;
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1) >> 1;
            if (sh.c[mid] <= slot)
                lo = mid;
            else
                hi = mid - 1;
        }
        sh.sym[slot] = (uint8_t)lo;
    }
    __syncthreads();

    const uint32_t* dir = reinterpret_cast<const uint32_t*>(pay + 512);
    const uint8_t* data = pay + 512 + 4ull * nseg;
    const uint64_t data_bytes = C - 512ull - 4ull * nseg;
    uint8_t* raw = scratch_raw + un.cache_off;  // the unit's stretch of the scratch (16-byte aligned)
    uint64_t carry = 0;
    for (uint32_t g0 = 0; g0 < nseg; g0 += kEntThreads) {
        const uint32_t g = g0 + tid;
        const uint32_t nw = g < nseg ? dir[g] : 0u;
        const uint32_t size = g < nseg ? segment_bytes(min(nw, kSegWordsMax)) : 0u;
        if (g < nseg && nw > kSegWordsMax) sh.bad = 1;
        uint32_t incl = size;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)lane >= o) incl += v;
        }
        if (lane == 31) sh.scan[warp] = incl;
        __syncthreads();
        uint32_t wbase = 0, chunk_total = 0;
        for (int w = 0; w < kEntWarps; ++w) {
            if (w < (int)warp) wbase += sh.scan[w];
            chunk_total += sh.scan[w];
        }
        sh.off[tid] = wbase + incl - size;
        sh.nw[tid] = min(nw, kSegWordsMax);
        if (tid == 0 && carry + chunk_total > data_bytes) sh.bad = 1;  // sizes must stay inside the section
        __syncthreads();
        if (sh.bad) break;
        const uint32_t in_chunk = min((uint32_t)kEntThreads, nseg - g0);
        for (uint32_t k = warp; k < in_chunk; k += kEntWarps) {
            const uint32_t gg = g0 + k;
            const uint32_t n = (uint32_t)min((uint64_t)kSegment, P - (uint64_t)gg * kSegment);
            const uint32_t snw = sh.nw[k];
            // the coded segment into shared memory (4-byte aligned in the section)
            const uint32_t* from = reinterpret_cast<const uint32_t*>(data + carry + sh.off[k]);
            uint32_t* stage = reinterpret_cast<uint32_t*>(sh.seg[warp]);
            for (uint32_t i = lane; i < (segment_bytes(snw) >> 2); i += 32) stage[i] = from[i];
            __syncwarp();
            const uint16_t* words = reinterpret_cast<const uint16_t*>(sh.seg[warp] + 4 * 32);
            uint32_t x = stage[lane], ptr = snw;
            uint8_t* out = raw + (uint64_t)gg * kSegment;
            const uint32_t steps = (n + 31u) >> 5;
            bool broken = false;
            for (uint32_t t = 0; t < steps; ++t) {
                const uint32_t i = 32u * t + lane;
                const bool has = i < n;
                bool need = false;
                if (has) {
                    const uint32_t slot = x & (kProbScale - 1u);
                    const uint32_t s = sh.sym[slot];
                    out[i] = (uint8_t)s;
                    x = (uint32_t)sh.f[s] * (x >> kProbBits) + slot - sh.c[s];
                    need = x < kRansL;
                }
                const uint32_t votes = __ballot_sync(0xffffffffu, need);
                const uint32_t k_need = __popc(votes);
                if (k_need > ptr) {
                    broken = true;
                    break;
                }
                if (need) x = (x << 16) | words[ptr - k_need + __popc(votes & ((1u << lane) - 1u))];
                ptr -= k_need;
            }
            // all words used and every lane back at the start state, or the section is damaged
            if (broken || ptr != 0 || __any_sync(0xffffffffu, x != kRansL)) sh.bad = 1;
            __syncwarp();
        }
        carry += chunk_total;
        __syncthreads();
        if (sh.bad) break;
    }
    __syncthreads();
    if (sh.bad || carry != data_bytes) {
        if (tid == 0 && status) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
        return;
    }
    // the raw payload goes back into the message, which then is what the sender step had written
    __threadfence_block();
    uint8_t* dst = msg + payoff;
    for (uint64_t i = (uint64_t)tid * 16; i < P; i += (uint64_t)kEntThreads * 16) {
        if (i + 16 <= P) {
            *reinterpret_cast<uint4*>(dst + i) = *reinterpret_cast<const uint4*>(raw + i);
        } else {
            for (uint64_t k = i; k < P; ++k) dst[k] = raw[k];
        }
    }
    if (tid == 0) wire_bytes[unit] = payoff + P;
}

}  // namespace ciera

using namespace ciera;

static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

// scratch of the sender stage: per segment slot a word count and kSegSlot bytes
static size_t encode_scratch_bytes(const ciera_plan* p) {
    return ((size_t)p->total_segments * sizeof(uint32_t) + 15) / 16 * 16 + (size_t)p->total_segments * kSegSlot;
}

extern "C" size_t ciera_plan_entropy_scratch_bytes(const ciera_plan* p) {
    if (!p) return 0;
    const size_t enc = encode_scratch_bytes(p), dec = (size_t)p->cache_extent;
    return (enc > dec ? enc : dec) + 16;
}

extern "C" int ciera_entropy_encode(const ciera_plan* p, void* messages_dev, uint64_t* wire_bytes_dev, void* scratch_dev,
                                    void* stream) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    if (p->tiles.empty()) return CIERA_OK;
    if (!messages_dev || !wire_bytes_dev || !scratch_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(scratch_dev) || ((uintptr_t)wire_bytes_dev & 7u))
        return CIERA_ERR_MISALIGNED;
    uint32_t* nw = (uint32_t*)scratch_dev;
    uint8_t* slots = (uint8_t*)scratch_dev + ((size_t)p->total_segments * sizeof(uint32_t) + 15) / 16 * 16;
    entropy_encode_kernel<<<p->n_units, kEntThreads, 0, (cudaStream_t)stream>>>(
        p->units_dev, p->seg_base_dev, p->dtype == CIERA_BF16 ? 1u : 3u, p->log2b, (uint8_t*)messages_dev,
        (unsigned long long*)wire_bytes_dev, slots, nw);
    count_launch();
    return check_launch();
}

extern "C" int ciera_entropy_decode(const ciera_plan* p, void* messages_dev, uint64_t* wire_bytes_dev, void* scratch_dev,
                                    int32_t* status_dev, void* stream) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    if (p->tiles.empty()) return CIERA_OK;
    if (!messages_dev || !wire_bytes_dev || !scratch_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(scratch_dev) || ((uintptr_t)wire_bytes_dev & 7u))
        return CIERA_ERR_MISALIGNED;
    static std::atomic<int> configured[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    if (!configured[dev].load(std::memory_order_acquire)) {
        e = cudaFuncSetAttribute(entropy_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(DecodeShared));
        if (e != cudaSuccess) return record_cuda_error(e);
        configured[dev].store(1, std::memory_order_release);
    }
    entropy_decode_kernel<<<p->n_units, kEntThreads, sizeof(DecodeShared), (cudaStream_t)stream>>>(
        p->units_dev, p->dtype == CIERA_BF16 ? 1u : 3u, p->log2b, (uint8_t*)messages_dev,
        (unsigned long long*)wire_bytes_dev, (uint8_t*)scratch_dev, status_dev);
    count_launch();
    return check_launch();
}
