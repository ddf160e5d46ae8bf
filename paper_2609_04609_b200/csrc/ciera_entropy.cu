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
// Coded section: [A x u16 f] [n_seg x u32 word counts] [segments: 32 x u32 final states, words,
// 2 zero bytes if the count is odd].  It replaces the raw payload only if strictly shorter; the
// receiver knows the raw length from the bitmap and so tells the two forms apart by the length.
// The symbols are the exponents of the changed blocks (Algorithm 1 codes {exp[k] | bitmap[k] = 1}):
// for bf16 and fp32 the payload's bytes as they are, A = 256 table entries.  For fp16 the five-bit
// packing of the payload is undone into a scratch first (one symbol per byte, A = 32 entries travel),
// segments are cut every 4096 symbols, "raw length" above is the packed payload's, and the receiver
// packs the decoded symbols back into the message.
//
// Work split: a unit of up to 64 segments' worth of values (262 144) is done by one thread block from
// start to end (histogram, model, segments into a scratch, coded form into the message).  Longer
// units go through a chain of launches whose grids run over chunks of 64 segments, so that their
// work spreads over the GPU: sender = histogram, model, segments, layout, copy; receiver = layout,
// segments, restore.  Nothing waits for another thread block anywhere.
#include "ciera_bits.cuh"

namespace ciera {

constexpr uint32_t kProbBits = 12, kProbScale = 1u << kProbBits;
constexpr uint32_t kRansL = 1u << 16;
constexpr uint32_t kSegment = 4096;                              // bytes of raw payload per segment
constexpr uint32_t kSegWordsMax = kSegment * kProbBits / 16;     // 3072: a symbol adds at most 12 bits
constexpr uint32_t kSegSlot = 4 * 32 + 2 * kSegWordsMax;         // 6272 bytes: states + words
constexpr int kEntThreads = 256, kEntWarps = kEntThreads / 32;
constexpr uint32_t kLongSegs = 64;  // units with more segment slots than this take the chunked path

__host__ __device__ inline uint64_t segments_of(uint64_t bytes) { return (bytes + kSegment - 1) / kSegment; }
__host__ __device__ inline uint32_t segment_bytes(uint32_t nw) { return 4u * 32u + 2u * nw + ((nw & 1u) ? 2u : 0u); }
// bytes of the frequency table that travels: one u16 per symbol of the alphabet
__host__ __device__ inline uint32_t model_bytes(int dt) { return dt == CIERA_FP16 ? 64u : 512u; }

// ---------------------------------------------------------------------------------- shared pieces

// Adds the bytes pay[lo, hi) to the warp-private histograms (lo a multiple of 16, pay 16-byte aligned).
__device__ __forceinline__ void histogram_add(uint32_t (*hist)[256], const uint8_t* pay, uint64_t lo, uint64_t hi,
                                              uint32_t tid) {
    const uint32_t warp = tid >> 5;
    for (uint64_t i = lo + (uint64_t)tid * 16; i < hi; i += (uint64_t)kEntThreads * 16) {
        if (i + 16 <= hi) {
            const uint4 v = *reinterpret_cast<const uint4*>(pay + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 16; ++k) atomicAdd(&hist[warp][(w[k >> 2] >> (8 * (k & 3))) & 0xFFu], 1u);
        } else {
            for (uint64_t k = i; k < hi; ++k) atomicAdd(&hist[warp][pay[k]], 1u);
        }
    }
}

// Exclusive running sums of f[0..255] by one warp (lane l owns symbols 8 l .. 8 l + 7): returns the sum of
// the symbols before the lane's first one and leaves the sums inside its group in local[]; `total`
// gets the sum of all.
__device__ __forceinline__ uint32_t warp_prefix256(const uint16_t* f, uint32_t lane, uint32_t local[8], uint32_t& total) {
    uint32_t run = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        local[i] = run;
        run += f[8 * lane + i];
    }
    uint32_t incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)lane >= o) incl += t;
    }
    total = __shfl_sync(0xffffffffu, incl, 31);
    return incl - run;
}

// Index of the largest of v[0..255], the lowest index among equals (one warp; v(s) gives the value).
template <class V>
__device__ __forceinline__ uint32_t warp_argmax256(V v, uint32_t lane) {
    unsigned long long key = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t s = 8 * lane + i;
        const unsigned long long k = ((unsigned long long)v(s) << 8) | (255u - s);
        key = k > key ? k : key;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long k = __shfl_xor_sync(0xffffffffu, key, o);
        key = k > key ? k : key;
    }
    return 255u - (uint32_t)(key & 255u);
}

// Frequencies from counts (h[256] in shared memory, P = their sum): thread s owns symbol s, then the
// first warp settles the sum.  Ends with a barrier; f is then final.
__device__ __forceinline__ void normalise_model(const uint32_t* h, uint64_t P, uint16_t* f, uint32_t tid) {
    {
        uint32_t v = 0;
        if (h[tid]) {
            v = (uint32_t)((uint64_t)h[tid] * kProbScale / P);
            if (v == 0) v = 1;
        }
        f[tid] = (uint16_t)v;
    }
    __syncthreads();
    if (tid < 32) {
        uint32_t local[8], sum;
        warp_prefix256(f, tid, local, sum);
        if (sum < kProbScale) {  // the shortfall goes to the most frequent symbol
            const uint32_t best = warp_argmax256([&](uint32_t s) { return h[s]; }, tid);
            if (tid == 0) f[best] = (uint16_t)(f[best] + (kProbScale - sum));
        } else {  // an excess is taken from the largest entries
            uint32_t excess = sum - kProbScale;
            while (excess) {
                const uint32_t big = warp_argmax256([&](uint32_t s) { return (uint32_t)f[s]; }, tid);
                const uint32_t take = min((uint32_t)f[big] - 1u, excess);
                __syncwarp();
                if (tid == 0) f[big] = (uint16_t)(f[big] - take);
                __syncwarp();
                excess -= take;
            }
        }
    }
    __syncthreads();
}

// Starts c[] and reciprocals from final frequencies.  Ends with a barrier.
// x / f through a multiplication: rcp = ceil(2^64 / f) exceeds 2^64 / f by less than 1, so for
// x < 2^32 the product x * rcp / 2^64 exceeds x / f by less than 2^-32 -- too little to reach the next
// integer, because the fraction of x / f is at most 1 - 1/4096.  (f = 1 is handled apart.)
// The coder reads one 16-byte entry per symbol: {rcp low, rcp high, f | c << 16, 0}.
__device__ __forceinline__ void encoder_tables(const uint16_t* f, uint4* enc, uint32_t tid) {
    const unsigned long long rcp = f[tid] > 1 ? (~0ull) / f[tid] + 1ull : 0ull;
    enc[tid].x = (uint32_t)rcp;
    enc[tid].y = (uint32_t)(rcp >> 32);
    enc[tid].w = 0u;
    if (tid < 32) {
        uint32_t local[8], total;
        const uint32_t base = warp_prefix256(f, tid, local, total);
#pragma unroll
        for (int i = 0; i < 8; ++i) enc[8 * tid + i].z = (uint32_t)f[8 * tid + i] | ((base + local[i]) << 16);
    }
    __syncthreads();
}

// One warp codes one segment: src[0, n) -> slot (32 states, then the words).  Returns the word count.
__device__ __forceinline__ uint32_t encode_segment(const uint8_t* src, uint32_t n, uint8_t* stage, const uint4* enc,
                                                   uint8_t* slot, uint32_t lane) {
    for (uint32_t i = lane * 16; i < n; i += 32 * 16) {
        if (i + 16 <= n) {
            *reinterpret_cast<uint4*>(stage + i) = *reinterpret_cast<const uint4*>(src + i);
        } else {
            for (uint32_t k = i; k < n; ++k) stage[k] = src[k];
        }
    }
    __syncwarp();
    uint16_t* words = reinterpret_cast<uint16_t*>(slot + 4 * 32);
    uint32_t x = kRansL, nw = 0;
    const uint32_t below = (1u << lane) - 1u;
    const uint32_t enc_a = (uint32_t)__cvta_generic_to_shared(enc);
    const uint32_t stage_a = (uint32_t)__cvta_generic_to_shared(stage) + lane;
    // one coder step of this lane for the symbol at byte 32 t + lane of the segment
    auto step = [&](uint32_t t, bool has) {
        uint32_t s = 0;
        if (has) asm volatile("ld.shared.u8 %0, [%1];" : "=r"(s) : "r"(stage_a + 32u * t) : "memory");
        uint4 en;
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(en.x), "=r"(en.y), "=r"(en.z), "=r"(en.w)
                     : "r"(enc_a + (s << 4))
                     : "memory");
        const uint32_t fs = en.z & 0xFFFFu, cs = en.z >> 16;
        const bool emit = has && (x >> 20) >= fs;  // x >= f * 2^20
        const uint32_t votes = __ballot_sync(0xffffffffu, emit);
        if (emit) {
            words[nw + __popc(votes & below)] = (uint16_t)x;
            x >>= 16;
        }
        nw += __popc(votes);
        if (has) {
            const unsigned long long rcp = (unsigned long long)en.x | ((unsigned long long)en.y << 32);
            const uint32_t q = fs > 1 ? (uint32_t)__umul64hi((unsigned long long)x, rcp) : x;
            x = q * kProbScale + (x - q * fs) + cs;
        }
    };
    uint32_t t = (n + 31u) >> 5;
    if (n & 31u) {  // the last, incomplete step comes first (the coder walks backwards)
        --t;
        step(t, lane < (n & 31u));
    }
    while (t-- > 0) step(t, true);
    reinterpret_cast<uint32_t*>(slot)[lane] = x;
    if (lane == 0 && (nw & 1u)) words[nw] = 0;
    __syncwarp();
    return nw;
}

// Receiver tables from the transmitted frequencies (f[] already in shared memory and synced):
// starts c[], then one word per slot: symbol | (f - 1) << 8 | (slot - c) << 20.  Returns false (in every
// thread) if the table does not sum to 4096.  The owner of a slot is the last symbol that starts at or
// below it (symbols that do not occur share their start with the next one, or start at 4096 behind the
// last occurring one).
__device__ __forceinline__ bool decoder_tables(const uint16_t* f, uint16_t* c, uint32_t* tab, uint32_t* flag, uint32_t tid) {
    if (tid < 32) {
        uint32_t local[8], total;
        const uint32_t base = warp_prefix256(f, tid, local, total);
#pragma unroll
        for (int i = 0; i < 8; ++i) c[8 * tid + i] = (uint16_t)min(base + local[i], kProbScale);
        if (tid == 0) *flag = total == kProbScale ? 1u : 0u;
    }
    __syncthreads();
    if (*flag == 0) return false;
    // thread t fills slots 16 t .. 16 t + 15: a binary search for the owner of the first, then a walk
    {
        uint32_t slot = tid * 16;
        uint32_t lo = 0, hi = 255;
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1) >> 1;
            if (c[mid] <= slot)
                lo = mid;
            else
                hi = mid - 1;
        }
        uint32_t cs = c[lo], fm1 = (uint32_t)f[lo] - 1u;
        for (uint32_t k = 0; k < 16; ++k, ++slot) {
            if (slot - cs > fm1) {  // past the owner's last slot: on to the next symbol that occurs
                do ++lo; while (lo < 255u && c[lo + 1] <= slot);
                cs = c[lo];
                fm1 = (uint32_t)f[lo] - 1u;
            }
            // the owner occurs (f >= 1, its slots are [c, c + f)): the sum is 4096 and every slot has one
            tab[slot] = lo | (fm1 & 0xFFFu) << 8 | ((slot - cs) & 0xFFFu) << 20;
        }
    }
    __syncthreads();
    return true;
}

// One warp decodes one segment: coded (32 states + snw words, 4-byte aligned, in global memory) ->
// out[0, n).  The words are read where they lie (a step takes a handful of neighbouring words from the
// end of what is left, so the reads of a warp fall into one or two cache lines that stay in L1 for the
// next steps); without a staged copy the kernel's shared memory is the slot table, and many warps per
// SM hide the latency of a line's first touch.
// Returns false (in every lane) if the words run out, are left over, or a lane does not end in the
// start state.
__device__ __forceinline__ bool decode_segment(const uint8_t* coded, uint32_t snw, uint32_t n, const uint32_t* tab,
                                               uint8_t* out, uint32_t lane) {
    const uint16_t* words = reinterpret_cast<const uint16_t*>(coded + 4 * 32);
    for (uint32_t i = lane * 64u; i < snw; i += 32u * 64u)  // bring the word list towards the SM, a line per lane
        asm volatile("prefetch.global.L2 [%0];" ::"l"(words + i));
    const uint32_t tab_a = (uint32_t)__cvta_generic_to_shared(tab);
    uint32_t x = reinterpret_cast<const uint32_t*>(coded)[lane], ptr = snw;
    const uint32_t below = (1u << lane) - 1u;
    const uint32_t full = n >> 5;  // steps in which every lane has a symbol
    uint8_t* o = out + lane;
    bool ok = true;
    // one step: `has` = this lane decodes a symbol in it
    auto step = [&](bool has) -> bool {
        bool need = false;
        if (has) {
            uint32_t en;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(en) : "r"(tab_a + ((x & (kProbScale - 1u)) << 2)) : "memory");
            *o = (uint8_t)en;
            x = (((en >> 8) & 0xFFFu) + 1u) * (x >> kProbBits) + (en >> 20);
            need = x < kRansL;
        }
        o += 32;
        const uint32_t votes = __ballot_sync(0xffffffffu, need);
        const uint32_t k_need = __popc(votes);
        if (k_need > ptr) return false;  // the words run out (the same in every lane)
        ptr -= k_need;
        if (need) x = (x << 16) | words[ptr + __popc(votes & below)];
        return true;
    };
    for (uint32_t t = 0; t < full && ok; ++t) ok = step(true);
    if (ok && (n & 31u)) ok = step(lane < (n & 31u));
    ok = ok && ptr == 0 && !__any_sync(0xffffffffu, x != kRansL);
    __syncwarp();
    return ok;
}

// Raw payload length Q in bytes and symbol count S of a unit from its bitmap (block-wide; `acc` in shared
// memory, zeroed and synced by the caller).  The bitmap's bits past the last block and the pad behind it
// are zero.
__device__ __forceinline__ uint64_t raw_payload_bytes(const uint8_t* msg, uint64_t N, int dt, uint32_t log2b,
                                                      unsigned long long* acc, uint32_t tid, uint64_t& S) {
    const uint64_t words = (bitmap_bytes(N, log2b) + 3) >> 2;  // inside the 16-byte padded bitmap
    const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msg);
    uint32_t cnt = 0;
    for (uint64_t i = tid; i < words; i += kEntThreads) cnt += __popc(bm32[i]);
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if ((tid & 31u) == 0 && cnt) atomicAdd(acc, (unsigned long long)cnt);
    __syncthreads();
    // every changed block carries a full block's bytes (one per exponent; fp16: five bits per exponent, rounded up
    // to whole bytes per block), a changed short last block fewer
    const uint32_t B = 1u << log2b;
    uint64_t Q = *acc * block_payload_bytes(B, dt);
    S = *acc << log2b;
    const uint32_t rem = (uint32_t)(N & (B - 1u));
    if (rem) {
        const uint64_t kb = num_blocks(N, log2b) - 1;
        if ((msg[kb >> 3] >> (kb & 7u)) & 1u) {
            Q -= block_payload_bytes(B, dt) - block_payload_bytes(rem, dt);
            S -= B - rem;
        }
    }
    return Q;
}

// Symbol count of a sender's payload of Q bytes.  bf16, fp32: a byte each.  fp16: the changed blocks lie one
// after the other, a full one taking block_payload_bytes(B) bytes, so Q and the last block's bit (a short last
// block is the only one of another size) give the count.  0 if Q is not such a sum.
__device__ __forceinline__ uint64_t symbols_of_payload(const uint8_t* msg, uint64_t N, int dt, uint32_t log2b, uint64_t Q) {
    if (dt != CIERA_FP16) return Q;
    const uint32_t B = 1u << log2b, full = (uint32_t)block_payload_bytes(B, dt);
    const uint32_t rem = (uint32_t)(N & (B - 1u));
    uint64_t tail_bytes = 0, tail_symbols = 0;
    if (rem) {
        const uint64_t kb = num_blocks(N, log2b) - 1;
        if ((msg[kb >> 3] >> (kb & 7u)) & 1u) {
            tail_bytes = block_payload_bytes(rem, dt);
            tail_symbols = rem;
        }
    }
    if (Q < tail_bytes || (Q - tail_bytes) % full != 0) return 0;
    return ((Q - tail_bytes) / full << log2b) + tail_symbols;
}

// fp16: the symbols [lo, hi) of a payload between their packed form (five bits each, a block starting on a byte
// boundary at block index x block_payload_bytes(B); all blocks before a short last one are full) and one byte
// each.  lo is a multiple of 8 and of the block size where that is smaller; hi <= symbol count.  A group of 8
// symbols is 5 bytes: one thread moves a group.  `sym` is 8-byte aligned.
__device__ __forceinline__ uint64_t packed_group_offset(uint64_t s0, uint32_t log2b) {
    const uint32_t B = 1u << log2b;
    return (s0 >> log2b) * block_payload_bytes(B, CIERA_FP16) + (uint64_t)(((uint32_t)s0 & (B - 1u)) >> 3) * 5u;
}
__device__ __forceinline__ void unpack_symbols(const uint8_t* pay, uint8_t* sym, uint32_t log2b, uint64_t lo, uint64_t hi,
                                               uint32_t tid, uint32_t threads) {
    const uint32_t group = min(1u << log2b, 8u);
    for (uint64_t s0 = lo + (uint64_t)tid * group; s0 < hi; s0 += (uint64_t)threads * group) {
        const uint32_t ns = (uint32_t)min((uint64_t)group, hi - s0), nbytes = (5u * ns + 7u) >> 3;
        const uint8_t* src = pay + packed_group_offset(s0, log2b);
        unsigned long long v = 0;
        for (uint32_t k = 0; k < nbytes; ++k) v |= (unsigned long long)src[k] << (8u * k);
        if (ns == 8u) {
            unsigned long long out = 0;
#pragma unroll
            for (uint32_t k = 0; k < 8u; ++k) out |= ((v >> (5u * k)) & 31ull) << (8u * k);
            *reinterpret_cast<unsigned long long*>(sym + s0) = out;
        } else {
            for (uint32_t k = 0; k < ns; ++k) sym[s0 + k] = (uint8_t)((v >> (5u * k)) & 31u);
        }
    }
}
__device__ __forceinline__ void pack_symbols(const uint8_t* sym, uint8_t* pay, uint32_t log2b, uint64_t lo, uint64_t hi,
                                             uint32_t tid, uint32_t threads) {
    const uint32_t group = min(1u << log2b, 8u);
    for (uint64_t s0 = lo + (uint64_t)tid * group; s0 < hi; s0 += (uint64_t)threads * group) {
        const uint32_t ns = (uint32_t)min((uint64_t)group, hi - s0), nbytes = (5u * ns + 7u) >> 3;
        unsigned long long v = 0;
        for (uint32_t k = 0; k < ns; ++k) v |= (unsigned long long)(sym[s0 + k] & 31u) << (5u * k);
        uint8_t* dst = pay + packed_group_offset(s0, log2b);
        for (uint32_t k = 0; k < nbytes; ++k) dst[k] = (uint8_t)(v >> (8u * k));
    }
}

// Exclusive scan of one value per thread over the block; `scan` holds kEntWarps words.  Returns
// the thread's offset; `total` gets the block's sum.  Contains barriers.
__device__ __forceinline__ uint32_t block_scan(uint32_t v, uint32_t* scan, uint32_t tid, uint32_t& total) {
    const uint32_t lane = tid & 31u, warp = tid >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)lane >= o) incl += t;
    }
    __syncthreads();  // the previous use of scan[] is over
    if (lane == 31) scan[warp] = incl;
    __syncthreads();
    uint32_t wbase = 0;
    total = 0;
    for (int w = 0; w < kEntWarps; ++w) {
        if (w < (int)warp) wbase += scan[w];
        total += scan[w];
    }
    return wbase + incl - v;
}

// ------------------------------------------------------------------------------------------ sender
// units of up to kLongSegs segment slots: one thread block per unit, start to end

template <bool HALF>  // HALF: fp16, five-bit symbols (see the head of this file)
__global__ void __launch_bounds__(kEntThreads, 5)
entropy_encode_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                      int dt, uint32_t log2b, uint8_t* msgs, unsigned long long* wire_bytes,
                      uint8_t* scratch_slots, uint32_t* scratch_nw, uint8_t* scratch_sym) {
    __shared__ __align__(16) uint8_t s_seg[kEntWarps][kSegment];  // a warp's segment of symbols
    // the warps' private histograms are needed before the segments are staged, the two small lists of
    // step 4 after: all of them lie in the first part of s_seg
    uint32_t (*const s_hist)[256] = reinterpret_cast<uint32_t (*)[256]>(&s_seg[0][0]);
    static_assert(sizeof(uint32_t) * 256 * kEntWarps <= sizeof(uint8_t) * kSegment * kEntWarps, "histograms overlay the stages");
    __shared__ uint16_t s_f[256];
    __shared__ uint4 s_enc[256];
    __shared__ uint32_t s_scan[kEntWarps];
    __shared__ unsigned long long s_total;
    const uint32_t unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[unit];
    if (un.n_values == 0 || segments_of(un.n_values) > kLongSegs) return;
    const uint64_t payoff = payload_offset_of(un.n_values, dt, log2b);
    const uint64_t Q = wire_bytes[unit] - payoff;
    // nothing to code; or a length that no sender step reports (shorter than the fixed sections, more
    // than the payload of a unit whose every block changed, not a sum of block sizes): everything below is indexed by the
    // symbol count P, so such a unit is left alone
    if (Q == 0 || Q > payload_bytes_max(un.n_values, dt, log2b)) return;
    const uint64_t P = symbols_of_payload(msgs + un.msg_off, un.n_values, dt, log2b, Q);
    if (P == 0 || P > un.n_values) return;
    uint8_t* const pay = msgs + un.msg_off + payoff;  // 16-byte aligned
    const uint32_t nseg = (uint32_t)segments_of(P);
    constexpr uint32_t hdr = HALF ? 64u : 512u;  // = model_bytes(dt)
    const uint8_t* src = pay;  // the symbols, one per byte
    if (HALF) {
        uint8_t* sym = scratch_sym + un.cache_off;
        unpack_symbols(pay, sym, log2b, 0, P, tid, kEntThreads);
        src = sym;
        __syncthreads();
    }

    // 1. histogram of the symbols (one private copy per warp), 2. the model
    for (uint32_t i = lane; i < 256; i += 32) s_hist[warp][i] = 0;
    if (tid == 0) s_total = 0;
    __syncwarp();
    histogram_add(s_hist, src, 0, P, tid);
    __syncthreads();
    {
        uint32_t h = 0;
        for (int w = 0; w < kEntWarps; ++w) h += s_hist[w][tid];
        __syncthreads();
        s_hist[0][tid] = h;
    }
    __syncthreads();
    normalise_model(s_hist[0], P, s_f, tid);
    encoder_tables(s_f, s_enc, tid);

    // 3. segments: warp w codes segments w, w + 8, ... into the unit's slots of the scratch
    const unsigned long long slot0 = seg_base[unit];
    for (uint32_t g = warp; g < nseg; g += kEntWarps) {
        const uint32_t n = (uint32_t)min((uint64_t)kSegment, P - (uint64_t)g * kSegment);
        const uint32_t nw = encode_segment(src + (uint64_t)g * kSegment, n, s_seg[warp], s_enc,
                                           scratch_slots + (slot0 + g) * kSegSlot, lane);
        if (lane == 0) {
            scratch_nw[slot0 + g] = nw;
            atomicAdd(&s_total, (unsigned long long)segment_bytes(nw));
        }
    }
    __syncthreads();  // every warp is done reading the raw payload and writing its slots

    // 4. keep the raw form unless the coded one is strictly shorter; else move it into the message
    const uint64_t C = (uint64_t)hdr + 4ull * nseg + s_total;
    if (C >= Q) return;
    if (tid < hdr / 2u) reinterpret_cast<uint16_t*>(pay)[tid] = s_f[tid];
    uint32_t* dir = reinterpret_cast<uint32_t*>(pay + hdr);
    uint8_t* data = pay + hdr + 4ull * nseg;
    // nseg <= kLongSegs <= kEntThreads: one round
    const uint32_t nw = tid < nseg ? scratch_nw[slot0 + tid] : 0u;
    const uint32_t size = tid < nseg ? segment_bytes(nw) : 0u;
    if (tid < nseg) dir[tid] = nw;
    uint32_t total;
    uint32_t* s_off = &s_hist[1][0];
    uint32_t* s_size = &s_hist[2][0];
    s_off[tid] = block_scan(size, s_scan, tid, total);
    s_size[tid] = size;
    __syncthreads();
    for (uint32_t k = warp; k < nseg; k += kEntWarps) {
        const uint32_t* from = reinterpret_cast<const uint32_t*>(scratch_slots + (slot0 + k) * kSegSlot);
        uint32_t* to = reinterpret_cast<uint32_t*>(data + s_off[k]);
        for (uint32_t i = lane; i < (s_size[k] >> 2); i += 32) to[i] = from[i];
    }
    if (tid == 0) wire_bytes[unit] = payoff + C;
}

// longer units: grids over chunks of kLongSegs segments.  A chunk record = {unit, first segment of
// the chunk inside the unit, index of the unit among the long ones, 0}.  Per long unit the scratch
// holds a record of 2048 bytes: 256 x u32 counts, 256 x u16 frequencies, then the words below.
constexpr uint32_t kLongRec = 2048;
struct LongState {            // at byte 1536 of a long unit's record
    unsigned long long total;   // sender: bytes of all coded segments
    unsigned long long P;       // receiver: symbols of the raw payload
    uint32_t coded;             // 1: the coded form is (sender) / was (receiver) chosen
    uint32_t bad;               // receiver: a segment did not decode
    uint32_t nseg;              // segments of the symbols
    uint32_t pad;
    unsigned long long Q;       // receiver: raw payload length in bytes (P = its symbols)
};
__device__ __forceinline__ uint32_t* long_hist(uint8_t* recs, uint32_t li) { return reinterpret_cast<uint32_t*>(recs + (size_t)li * kLongRec); }
__device__ __forceinline__ uint16_t* long_model(uint8_t* recs, uint32_t li) { return reinterpret_cast<uint16_t*>(recs + (size_t)li * kLongRec + 1024); }
__device__ __forceinline__ LongState* long_state(uint8_t* recs, uint32_t li) { return reinterpret_cast<LongState*>(recs + (size_t)li * kLongRec + 1536); }

// Symbol count of a unit's payload on the sender (0: nothing to code); Q gets the payload's length in bytes.
// A reported length that no sender step can have produced -- shorter than the fixed sections, a payload
// longer than that of a unit whose every block changed, not a sum of block sizes, e.g. the stale word of a unit that an aborted
// encode never finished -- also gives 0: the histogram, the segments and the scratch slots are all indexed
// by the symbol count, so it must stay inside the unit's slot (a value has one exponent, and plans are
// limited to units whose block counts fit 32 bits).
__device__ __forceinline__ uint64_t sender_payload(const ciera_unit& un, int dt, uint32_t log2b, const uint8_t* msgs,
                                                   const unsigned long long* wire_bytes, uint32_t unit, uint64_t& payoff,
                                                   uint64_t& Q) {
    payoff = payload_offset_of(un.n_values, dt, log2b);
    Q = wire_bytes[unit] - payoff;
    if (Q == 0 || Q > payload_bytes_max(un.n_values, dt, log2b) || Q >= (1ull << 32)) return 0;
    const uint64_t P = symbols_of_payload(msgs + un.msg_off, un.n_values, dt, log2b, Q);
    return (P <= un.n_values && P < (1ull << 32)) ? P : 0;
}
// where a unit's symbols lie, one per byte: in the message, or (fp16) unpacked in the scratch
__device__ __forceinline__ const uint8_t* sender_symbols(const ciera_unit& un, int dt, const uint8_t* msgs, uint64_t payoff,
                                                         const uint8_t* scratch_sym) {
    return dt == CIERA_FP16 ? scratch_sym + un.cache_off : msgs + un.msg_off + payoff;
}

// fp16 only: the long units' payloads unpacked into the scratch, a chunk per thread block
__global__ void __launch_bounds__(kEntThreads)
entropy_long_unpack_kernel(const ciera_unit* __restrict__ units, const uint4* __restrict__ chunks, int dt, uint32_t log2b,
                           const uint8_t* msgs, const unsigned long long* wire_bytes, uint8_t* scratch_sym) {
    const uint4 ch = chunks[blockIdx.x];
    const ciera_unit un = units[ch.x];
    uint64_t payoff, Q;
    const uint64_t P = sender_payload(un, dt, log2b, msgs, wire_bytes, ch.x, payoff, Q);
    const uint64_t lo = (uint64_t)ch.y * kSegment;
    if (lo >= P) return;
    const uint64_t hi = min(P, lo + (uint64_t)kLongSegs * kSegment);
    unpack_symbols(msgs + un.msg_off + payoff, scratch_sym + un.cache_off, log2b, lo, hi, threadIdx.x, kEntThreads);
}

__global__ void __launch_bounds__(kEntThreads)
entropy_long_hist_kernel(const ciera_unit* __restrict__ units, const uint4* __restrict__ chunks, int dt, uint32_t log2b,
                         const uint8_t* msgs, const unsigned long long* wire_bytes, uint8_t* recs,
                         const uint8_t* scratch_sym) {
    __shared__ uint32_t s_hist[kEntWarps][256];
    const uint4 ch = chunks[blockIdx.x];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[ch.x];
    uint64_t payoff, Q;
    const uint64_t P = sender_payload(un, dt, log2b, msgs, wire_bytes, ch.x, payoff, Q);
    const uint64_t lo = (uint64_t)ch.y * kSegment;
    if (lo >= P) return;
    const uint64_t hi = min(P, lo + (uint64_t)kLongSegs * kSegment);
    for (uint32_t i = lane; i < 256; i += 32) s_hist[warp][i] = 0;
    __syncwarp();
    histogram_add(s_hist, sender_symbols(un, dt, msgs, payoff, scratch_sym), lo, hi, tid);
    __syncthreads();
    uint32_t h = 0;
    for (int w = 0; w < kEntWarps; ++w) h += s_hist[w][tid];
    if (h) atomicAdd(long_hist(recs, ch.z) + tid, h);
}

__global__ void __launch_bounds__(kEntThreads)
entropy_long_model_kernel(const ciera_unit* __restrict__ units, const uint32_t* __restrict__ long_units, int dt,
                          uint32_t log2b, const uint8_t* msgs, const unsigned long long* wire_bytes, uint8_t* recs) {
    __shared__ uint32_t s_h[256];
    __shared__ uint16_t s_f[256];
    const uint32_t li = blockIdx.x, tid = threadIdx.x, unit = long_units[li];
    uint64_t payoff, Q;
    const uint64_t P = sender_payload(units[unit], dt, log2b, msgs, wire_bytes, unit, payoff, Q);
    if (tid == 0) {
        LongState* st = long_state(recs, li);
        st->total = 0;
        st->coded = 0;
        st->bad = 0;
    }
    if (P == 0) return;
    s_h[tid] = long_hist(recs, li)[tid];
    __syncthreads();
    normalise_model(s_h, P, s_f, tid);
    long_model(recs, li)[tid] = s_f[tid];
}

template <bool HALF>  // HALF: fp16, five-bit symbols (see the head of this file)
__global__ void __launch_bounds__(kEntThreads)
entropy_long_encode_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                           const uint4* __restrict__ chunks, int dt, uint32_t log2b, const uint8_t* msgs,
                           const unsigned long long* wire_bytes, uint8_t* recs, uint8_t* scratch_slots,
                           uint32_t* scratch_nw, const uint8_t* scratch_sym) {
    __shared__ __align__(16) uint8_t s_seg[kEntWarps][kSegment];
    __shared__ uint16_t s_f[256];
    __shared__ uint4 s_enc[256];
    __shared__ unsigned long long s_total;
    const uint4 ch = chunks[blockIdx.x];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[ch.x];
    uint64_t payoff, Q;
    const uint64_t P = sender_payload(un, dt, log2b, msgs, wire_bytes, ch.x, payoff, Q);
    if ((uint64_t)ch.y * kSegment >= P) return;
    const uint32_t nseg = (uint32_t)segments_of(P);
    const uint32_t g_end = min(nseg, ch.y + kLongSegs);
    s_f[tid] = long_model(recs, ch.z)[tid];
    if (tid == 0) s_total = 0;
    __syncthreads();
    encoder_tables(s_f, s_enc, tid);
    const uint8_t* pay = HALF ? scratch_sym + un.cache_off : msgs + un.msg_off + payoff;  // the symbols
    const unsigned long long slot0 = seg_base[ch.x];
    for (uint32_t g = ch.y + warp; g < g_end; g += kEntWarps) {
        const uint32_t n = (uint32_t)min((uint64_t)kSegment, P - (uint64_t)g * kSegment);
        const uint32_t nw = encode_segment(pay + (uint64_t)g * kSegment, n, s_seg[warp], s_enc,
                                           scratch_slots + (slot0 + g) * kSegSlot, lane);
        if (lane == 0) {
            scratch_nw[slot0 + g] = nw;
            atomicAdd(&s_total, (unsigned long long)segment_bytes(nw));
        }
    }
    __syncthreads();
    if (tid == 0) atomicAdd(&long_state(recs, ch.z)->total, s_total);
}

// decides raw or coded for a long unit; coded: table and word counts into the message, the byte
// offset of every segment into the scratch
__global__ void __launch_bounds__(kEntThreads)
entropy_long_layout_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                           const uint32_t* __restrict__ long_units, int dt, uint32_t log2b, uint8_t* msgs,
                           unsigned long long* wire_bytes, uint8_t* recs, const uint32_t* scratch_nw,
                           uint32_t* scratch_off) {
    __shared__ uint32_t s_scan[kEntWarps];
    const uint32_t li = blockIdx.x, tid = threadIdx.x, unit = long_units[li];
    const ciera_unit un = units[unit];
    uint64_t payoff, Q;
    const uint64_t P = sender_payload(un, dt, log2b, msgs, wire_bytes, unit, payoff, Q);
    if (P == 0) return;
    const uint32_t nseg = (uint32_t)segments_of(P);
    const uint32_t hdr = model_bytes(dt);
    LongState* st = long_state(recs, li);
    const uint64_t C = (uint64_t)hdr + 4ull * nseg + st->total;
    if (C >= Q) return;
    uint8_t* pay = msgs + un.msg_off + payoff;
    if (tid < hdr / 2u) reinterpret_cast<uint16_t*>(pay)[tid] = long_model(recs, li)[tid];
    uint32_t* dir = reinterpret_cast<uint32_t*>(pay + hdr);
    const unsigned long long slot0 = seg_base[unit];
    uint32_t carry = 0;  // C < Q < 2^32: offsets fit
    for (uint32_t g0 = 0; g0 < nseg; g0 += kEntThreads) {
        const uint32_t g = g0 + tid;
        const uint32_t nw = g < nseg ? scratch_nw[slot0 + g] : 0u;
        if (g < nseg) dir[g] = nw;
        uint32_t total;
        const uint32_t off = block_scan(g < nseg ? segment_bytes(nw) : 0u, s_scan, tid, total);
        if (g < nseg) scratch_off[slot0 + g] = carry + off;
        carry += total;
    }
    if (tid == 0) {
        st->coded = 1;
        st->nseg = nseg;
        wire_bytes[unit] = payoff + C;
    }
}

__global__ void __launch_bounds__(kEntThreads)
entropy_long_copy_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                         const uint4* __restrict__ chunks, int dt, uint32_t log2b, uint8_t* msgs, uint8_t* recs,
                         const uint8_t* scratch_slots, const uint32_t* scratch_nw, const uint32_t* scratch_off) {
    const uint4 ch = chunks[blockIdx.x];
    const LongState* st = long_state(recs, ch.z);
    if (st->coded == 0) return;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const ciera_unit un = units[ch.x];
    const uint32_t nseg = st->nseg;
    uint8_t* data = msgs + un.msg_off + payload_offset_of(un.n_values, dt, log2b) + model_bytes(dt) + 4ull * nseg;
    const unsigned long long slot0 = seg_base[ch.x];
    const uint32_t g_end = min(nseg, ch.y + kLongSegs);
    for (uint32_t g = ch.y + warp; g < g_end; g += kEntWarps) {
        const uint32_t* from = reinterpret_cast<const uint32_t*>(scratch_slots + (slot0 + g) * kSegSlot);
        uint32_t* to = reinterpret_cast<uint32_t*>(data + scratch_off[slot0 + g]);
        const uint32_t words4 = segment_bytes(scratch_nw[slot0 + g]) >> 2;
        for (uint32_t i = lane; i < words4; i += 32) to[i] = from[i];
    }
}

// ---------------------------------------------------------------------------------------- receiver
// units of up to kLongSegs segment slots: one thread block per unit, start to end

struct DecodeShared {
    uint32_t tab[kProbScale];      // slot -> symbol | (f - 1) << 8 | (slot - c) << 20
    uint16_t f[256], c[256];
    uint32_t off[kEntThreads];     // per segment: byte offset in the data part
    uint32_t nw[kEntThreads];      //              word count
    uint32_t scan[kEntWarps];
    unsigned long long changed;    // set bits of the unit's bitmap
    uint32_t flag, bad;
};

__device__ __forceinline__ void raise_corrupt(int32_t* status) {
    if (status) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
}

template <bool HALF>  // HALF: fp16, five-bit symbols (see the head of this file)
__global__ void __launch_bounds__(kEntThreads)
entropy_decode_kernel(const ciera_unit* __restrict__ units, int dt, uint32_t log2b, uint8_t* msgs,
                      unsigned long long* wire_bytes, uint8_t* scratch_raw, int32_t* status) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    DecodeShared& sh = *reinterpret_cast<DecodeShared*>(smem_raw);
    const uint32_t unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[unit];
    const uint64_t N = un.n_values;
    if (N == 0 || segments_of(N) > kLongSegs) return;
    uint8_t* const msg = msgs + un.msg_off;
    const uint64_t payoff = payload_offset_of(N, dt, log2b);
    if (tid == 0) {
        sh.changed = 0;
        sh.bad = 0;
    }
    __syncthreads();
    uint64_t P;  // symbols; Q = bytes of the raw payload
    const uint64_t Q = raw_payload_bytes(msg, N, dt, log2b, &sh.changed, tid, P);
    const uint64_t wire = wire_bytes[unit];
    if (Q == 0 || wire == payoff + Q) return;  // nothing travelled, or the raw form did
    const uint64_t C = wire - payoff;
    const uint32_t nseg = (uint32_t)segments_of(P);
    constexpr uint32_t hdr = HALF ? 64u : 512u;  // = model_bytes(dt)
    uint8_t* const pay = msg + payoff;
    if (wire < payoff || C >= Q || C < (uint64_t)hdr + 4ull * nseg) {
        if (tid == 0) raise_corrupt(status);
        return;
    }
    sh.f[tid] = tid < hdr / 2u ? reinterpret_cast<const uint16_t*>(pay)[tid] : (uint16_t)0;
    __syncthreads();
    if (!decoder_tables(sh.f, sh.c, sh.tab, &sh.flag, tid)) {
        if (tid == 0) raise_corrupt(status);
        return;
    }
    // where the segments lie (nseg <= kLongSegs <= kEntThreads: one round)
    const uint32_t* dir = reinterpret_cast<const uint32_t*>(pay + hdr);
    const uint8_t* data = pay + hdr + 4ull * nseg;
    const uint64_t data_bytes = C - hdr - 4ull * nseg;
    const uint32_t nw = tid < nseg ? dir[tid] : 0u;
    if (nw > kSegWordsMax) sh.bad = 1;
    uint32_t total;
    sh.off[tid] = block_scan(tid < nseg ? segment_bytes(min(nw, kSegWordsMax)) : 0u, sh.scan, tid, total);
    sh.nw[tid] = min(nw, kSegWordsMax);
    __syncthreads();
    if (sh.bad || total != data_bytes) {
        if (tid == 0) raise_corrupt(status);
        return;
    }
    uint8_t* raw = scratch_raw + un.cache_off;  // the unit's stretch of the scratch (16-byte aligned)
    for (uint32_t g = warp; g < nseg; g += kEntWarps) {
        const uint32_t n = (uint32_t)min((uint64_t)kSegment, P - (uint64_t)g * kSegment);
        if (!decode_segment(data + sh.off[g], sh.nw[g], n, sh.tab, raw + (uint64_t)g * kSegment, lane))
            sh.bad = 1;
    }
    __syncthreads();
    if (sh.bad) {
        if (tid == 0) raise_corrupt(status);
        return;
    }
    // the raw payload goes back into the message, which then is what the sender step had written
    if (HALF) {
        pack_symbols(raw, pay, log2b, 0, P, tid, kEntThreads);
    } else {
        for (uint64_t i = (uint64_t)tid * 16; i < P; i += (uint64_t)kEntThreads * 16) {
            if (i + 16 <= P) {
                *reinterpret_cast<uint4*>(pay + i) = *reinterpret_cast<const uint4*>(raw + i);
            } else {
                for (uint64_t k = i; k < P; ++k) pay[k] = raw[k];
            }
        }
    }
    if (tid == 0) wire_bytes[unit] = payoff + Q;
}

// longer units: layout (one block per unit), segments and restore (grids over chunks)
__global__ void __launch_bounds__(kEntThreads)
entropy_long_parse_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                          const uint32_t* __restrict__ long_units, int dt, uint32_t log2b, const uint8_t* msgs,
                          const unsigned long long* wire_bytes, uint8_t* recs, uint32_t* scratch_off, uint32_t* scratch_nw,
                          int32_t* status) {
    __shared__ uint32_t s_scan[kEntWarps];
    __shared__ unsigned long long s_changed;
    __shared__ uint32_t s_bad;
    const uint32_t li = blockIdx.x, tid = threadIdx.x, unit = long_units[li];
    const ciera_unit un = units[unit];
    const uint64_t N = un.n_values;
    LongState* st = long_state(recs, li);
    if (tid == 0) {
        st->coded = 0;
        st->bad = 0;
        s_changed = 0;
        s_bad = 0;
    }
    __syncthreads();
    const uint8_t* msg = msgs + un.msg_off;
    const uint64_t payoff = payload_offset_of(N, dt, log2b);
    uint64_t P;  // symbols; Q = bytes of the raw payload
    const uint64_t Q = raw_payload_bytes(msg, N, dt, log2b, &s_changed, tid, P);
    const uint64_t wire = wire_bytes[unit];
    if (Q == 0 || wire == payoff + Q) return;
    const uint64_t C = wire - payoff;
    const uint64_t nseg64 = segments_of(P);
    const uint32_t hdr = model_bytes(dt);
    if (wire < payoff || C >= Q || P >= (1ull << 32) || C < (uint64_t)hdr + 4ull * nseg64) {
        if (tid == 0) raise_corrupt(status);
        return;
    }
    const uint32_t nseg = (uint32_t)nseg64;
    const uint8_t* pay = msg + payoff;
    const uint32_t* dir = reinterpret_cast<const uint32_t*>(pay + hdr);
    const uint64_t data_bytes = C - hdr - 4ull * nseg;
    const unsigned long long slot0 = seg_base[unit];
    uint64_t carry = 0;
    for (uint32_t g0 = 0; g0 < nseg; g0 += kEntThreads) {
        const uint32_t g = g0 + tid;
        const uint32_t nw = g < nseg ? dir[g] : 0u;
        if (nw > kSegWordsMax) s_bad = 1;
        uint32_t total;
        const uint32_t off = block_scan(g < nseg ? segment_bytes(min(nw, kSegWordsMax)) : 0u, s_scan, tid, total);
        if (g < nseg) {
            scratch_off[slot0 + g] = (uint32_t)(carry + off);
            scratch_nw[slot0 + g] = min(nw, kSegWordsMax);
        }
        carry += total;
    }
    __syncthreads();
    if (s_bad || carry != data_bytes) {
        if (tid == 0) raise_corrupt(status);
        return;
    }
    if (tid == 0) {
        st->P = P;
        st->Q = Q;
        st->nseg = nseg;
        st->coded = 1;
    }
}

template <bool HALF>  // HALF: fp16, five-bit symbols (see the head of this file)
__global__ void __launch_bounds__(kEntThreads)
entropy_long_decode_kernel(const ciera_unit* __restrict__ units, const unsigned long long* __restrict__ seg_base,
                           const uint4* __restrict__ chunks, int dt, uint32_t log2b, const uint8_t* msgs,
                           uint8_t* recs, const uint32_t* scratch_off, const uint32_t* scratch_nw, uint8_t* scratch_raw,
                           int32_t* status) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    DecodeShared& sh = *reinterpret_cast<DecodeShared*>(smem_raw);
    const uint4 ch = chunks[blockIdx.x];
    LongState* st = long_state(recs, ch.z);
    if (st->coded == 0 || ch.y >= st->nseg) return;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const ciera_unit un = units[ch.x];
    const uint64_t P = st->P;
    const uint32_t nseg = st->nseg;
    const uint8_t* pay = msgs + un.msg_off + payload_offset_of(un.n_values, dt, log2b);
    constexpr uint32_t hdr = HALF ? 64u : 512u;  // = model_bytes(dt)
    sh.f[tid] = tid < hdr / 2u ? reinterpret_cast<const uint16_t*>(pay)[tid] : (uint16_t)0;
    if (tid == 0) sh.bad = 0;
    __syncthreads();
    if (!decoder_tables(sh.f, sh.c, sh.tab, &sh.flag, tid)) {
        if (tid == 0) {
            st->bad = 1;
            raise_corrupt(status);
        }
        return;
    }
    const uint8_t* data = pay + hdr + 4ull * nseg;
    uint8_t* raw = scratch_raw + un.cache_off;
    const unsigned long long slot0 = seg_base[ch.x];
    const uint32_t g_end = min(nseg, ch.y + kLongSegs);
    for (uint32_t g = ch.y + warp; g < g_end; g += kEntWarps) {
        const uint32_t n = (uint32_t)min((uint64_t)kSegment, P - (uint64_t)g * kSegment);
        if (!decode_segment(data + scratch_off[slot0 + g], scratch_nw[slot0 + g], n, sh.tab,
                            raw + (uint64_t)g * kSegment, lane))
            sh.bad = 1;
    }
    __syncthreads();
    if (tid == 0 && sh.bad) {
        st->bad = 1;
        raise_corrupt(status);
    }
}

__global__ void __launch_bounds__(kEntThreads)
entropy_long_restore_kernel(const ciera_unit* __restrict__ units, const uint4* __restrict__ chunks, int dt,
                            uint32_t log2b, uint8_t* msgs, unsigned long long* wire_bytes, const uint8_t* recs_c,
                            const uint8_t* scratch_raw) {
    const uint4 ch = chunks[blockIdx.x];
    const LongState* st = long_state(const_cast<uint8_t*>(recs_c), ch.z);
    if (st->coded == 0 || st->bad != 0) return;  // raw as received, or damaged: left as it is
    const uint32_t tid = threadIdx.x;
    const ciera_unit un = units[ch.x];
    const uint64_t P = st->P;
    const uint64_t lo = (uint64_t)ch.y * kSegment;
    if (lo >= P) return;
    const uint64_t hi = min(P, lo + (uint64_t)kLongSegs * kSegment);
    const uint64_t payoff = payload_offset_of(un.n_values, dt, log2b);
    uint8_t* pay = msgs + un.msg_off + payoff;
    const uint8_t* raw = scratch_raw + un.cache_off;
    if (dt == CIERA_FP16) {
        pack_symbols(raw, pay, log2b, lo, hi, tid, kEntThreads);
    } else {
        for (uint64_t i = lo + (uint64_t)tid * 16; i < hi; i += (uint64_t)kEntThreads * 16) {
            if (i + 16 <= hi) {
                *reinterpret_cast<uint4*>(pay + i) = *reinterpret_cast<const uint4*>(raw + i);
            } else {
                for (uint64_t k = i; k < hi; ++k) pay[k] = raw[k];
            }
        }
    }
    if (ch.y == 0 && tid == 0) wire_bytes[ch.x] = payoff + st->Q;
}

}  // namespace ciera

using namespace ciera;

static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }
static size_t up16(size_t x) { return (x + 15) / 16 * 16; }

// Scratch: [word count per segment slot][byte offset per segment slot][a record per long unit]
// [body: the segment slots (sender) or the decoded symbols at the units' cache offsets (receiver)]
// [fp16 sender: the unpacked symbols at the units' cache offsets]
struct ScratchLayout {
    size_t nw, off, recs, body, sym, total;
};
static ScratchLayout scratch_layout(const ciera_plan* p) {
    ScratchLayout L;
    L.nw = 0;
    L.off = L.nw + up16((size_t)p->total_segments * sizeof(uint32_t));
    L.recs = L.off + up16((size_t)p->total_segments * sizeof(uint32_t));
    L.body = L.recs + (size_t)p->ent_long_units.size() * kLongRec;
    const size_t enc = (size_t)p->total_segments * kSegSlot, dec = (size_t)p->cache_extent;
    L.sym = L.body + up16(enc > dec ? enc : dec);
    L.total = L.sym + (p->dtype == CIERA_FP16 ? dec : 0) + 16;
    return L;
}

extern "C" size_t ciera_plan_entropy_scratch_bytes(const ciera_plan* p) { return p ? scratch_layout(p).total : 0; }

static int check_entropy_args(const ciera_plan* p, const void* messages_dev, const void* wire_bytes_dev,
                              const void* scratch_dev) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    if (p->tiles.empty()) return CIERA_OK;
    if (!messages_dev || !wire_bytes_dev || !scratch_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(scratch_dev) || ((uintptr_t)wire_bytes_dev & 7u))
        return CIERA_ERR_MISALIGNED;
    return CIERA_OK;
}

extern "C" int ciera_entropy_encode(const ciera_plan* p, void* messages_dev, uint64_t* wire_bytes_dev, void* scratch_dev,
                                    void* stream) {
    int rc = check_entropy_args(p, messages_dev, wire_bytes_dev, scratch_dev);
    if (rc || p->tiles.empty()) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    const ScratchLayout L = scratch_layout(p);
    uint8_t* base = (uint8_t*)scratch_dev;
    uint32_t* nw = (uint32_t*)(base + L.nw);
    uint32_t* off = (uint32_t*)(base + L.off);
    uint8_t* recs = base + L.recs;
    uint8_t* slots = base + L.body;
    uint8_t* sym = base + L.sym;
    const int dt = p->dtype;
    uint8_t* msgs = (uint8_t*)messages_dev;
    unsigned long long* wire = (unsigned long long*)wire_bytes_dev;
    const uint32_t n_long = (uint32_t)p->ent_long_units.size(), n_chunks = (uint32_t)p->ent_chunks.size();
    if (n_long < p->n_units) {
        auto* k = dt == CIERA_FP16 ? entropy_encode_kernel<true> : entropy_encode_kernel<false>;
        k<<<p->n_units, kEntThreads, 0, s>>>(p->units_dev, p->seg_base_dev, dt, p->log2b, msgs, wire, slots, nw, sym);
        count_launch();
        if ((rc = check_launch())) return rc;
    }
    if (n_long) {
        cudaError_t e = cudaMemsetAsync(recs, 0, (size_t)n_long * kLongRec, s);  // the counts start at zero
        if (e != cudaSuccess) return record_cuda_error(e);
        if (dt == CIERA_FP16) {
            entropy_long_unpack_kernel<<<n_chunks, kEntThreads, 0, s>>>(p->units_dev, p->ent_chunks_dev, dt, p->log2b, msgs,
                                                                        wire, sym);
            count_launch();
        }
        entropy_long_hist_kernel<<<n_chunks, kEntThreads, 0, s>>>(p->units_dev, p->ent_chunks_dev, dt, p->log2b, msgs, wire,
                                                                  recs, sym);
        entropy_long_model_kernel<<<n_long, kEntThreads, 0, s>>>(p->units_dev, p->ent_long_units_dev, dt, p->log2b, msgs,
                                                                 wire, recs);
        auto* k = dt == CIERA_FP16 ? entropy_long_encode_kernel<true> : entropy_long_encode_kernel<false>;
        k<<<n_chunks, kEntThreads, 0, s>>>(p->units_dev, p->seg_base_dev, p->ent_chunks_dev, dt, p->log2b, msgs, wire, recs,
                                           slots, nw, sym);
        entropy_long_layout_kernel<<<n_long, kEntThreads, 0, s>>>(p->units_dev, p->seg_base_dev, p->ent_long_units_dev, dt,
                                                                  p->log2b, msgs, wire, recs, nw, off);
        entropy_long_copy_kernel<<<n_chunks, kEntThreads, 0, s>>>(p->units_dev, p->seg_base_dev, p->ent_chunks_dev, dt,
                                                                  p->log2b, msgs, recs, slots, nw, off);
        for (int i = 0; i < 5; ++i) count_launch();
        if ((rc = check_launch())) return rc;
    }
    return CIERA_OK;
}

extern "C" int ciera_entropy_decode(const ciera_plan* p, void* messages_dev, uint64_t* wire_bytes_dev, void* scratch_dev,
                                    int32_t* status_dev, void* stream) {
    int rc = check_entropy_args(p, messages_dev, wire_bytes_dev, scratch_dev);
    if (rc || p->tiles.empty()) return rc;
    static std::atomic<int> configured[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    if (!configured[dev].load(std::memory_order_acquire)) {
        for (auto* k : {entropy_decode_kernel<false>, entropy_decode_kernel<true>}) {
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecodeShared));
            if (e != cudaSuccess) return record_cuda_error(e);
        }
        for (auto* k : {entropy_long_decode_kernel<false>, entropy_long_decode_kernel<true>}) {
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecodeShared));
            if (e != cudaSuccess) return record_cuda_error(e);
        }
        configured[dev].store(1, std::memory_order_release);
    }
    cudaStream_t s = (cudaStream_t)stream;
    const ScratchLayout L = scratch_layout(p);
    uint8_t* base = (uint8_t*)scratch_dev;
    uint32_t* nw = (uint32_t*)(base + L.nw);
    uint32_t* off = (uint32_t*)(base + L.off);
    uint8_t* recs = base + L.recs;
    uint8_t* raw = base + L.body;
    const int dt = p->dtype;
    uint8_t* msgs = (uint8_t*)messages_dev;
    unsigned long long* wire = (unsigned long long*)wire_bytes_dev;
    const uint32_t n_long = (uint32_t)p->ent_long_units.size(), n_chunks = (uint32_t)p->ent_chunks.size();
    if (n_long < p->n_units) {
        auto* k = dt == CIERA_FP16 ? entropy_decode_kernel<true> : entropy_decode_kernel<false>;
        k<<<p->n_units, kEntThreads, sizeof(DecodeShared), s>>>(p->units_dev, dt, p->log2b, msgs, wire, raw, status_dev);
        count_launch();
        if ((rc = check_launch())) return rc;
    }
    if (n_long) {
        entropy_long_parse_kernel<<<n_long, kEntThreads, 0, s>>>(p->units_dev, p->seg_base_dev, p->ent_long_units_dev, dt,
                                                                 p->log2b, msgs, wire, recs, off, nw, status_dev);
        auto* k = dt == CIERA_FP16 ? entropy_long_decode_kernel<true> : entropy_long_decode_kernel<false>;
        k<<<n_chunks, kEntThreads, sizeof(DecodeShared), s>>>(p->units_dev, p->seg_base_dev, p->ent_chunks_dev, dt, p->log2b,
                                                              msgs, recs, off, nw, raw, status_dev);
        entropy_long_restore_kernel<<<n_chunks, kEntThreads, 0, s>>>(p->units_dev, p->ent_chunks_dev, dt, p->log2b, msgs,
                                                                     wire, recs, raw);
        for (int i = 0; i < 3; ++i) count_launch();
        if ((rc = check_launch())) return rc;
    }
    return CIERA_OK;
}
