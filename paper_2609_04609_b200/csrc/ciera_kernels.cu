// sm_100a kernels of libciera and their launchers.
//
// All kernels share one decomposition: grid = number of tiles of the plan, one thread block of
// 512 threads per tile of 8192 values, every thread owns 16 consecutive values, so that each of
// the byte-wide streams (exponent cache, sign-plus-mantissa, payload) is touched with one
// 128-bit access per thread and the 2- or 4-byte weight stream with two or four.
#include "ciera_bits.cuh"

namespace ciera {

// ------------------------------------------------------------------------------------------
// decode: Algorithm 1, receiver part

template <int DT>
__global__ void __launch_bounds__(kThreads)
decode_kernel(const TileDesc* __restrict__ tiles, uint32_t log2b, const uint8_t* msgs, uint8_t* cache,
              uint8_t* __restrict__ weights, const unsigned long long* __restrict__ wire_bytes, int32_t* status) {
    constexpr int VB = Traits<DT>::kValueBytes;
    constexpr int SMB = Traits<DT>::kSmBytes;
    __shared__ uint32_t s_bm[kBitmapWords];
    __shared__ uint32_t s_pre[kBitmapWords];
    __shared__ uint32_t s_tot;          // changed blocks of this tile
    __shared__ unsigned long long s_before;  // changed blocks of the unit before this tile

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const TileDesc td = load_tile_desc(tiles + blockIdx.x);
    const uint64_t N = td.n_unit;
    const uint32_t B = 1u << log2b;
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, N - v0);
    const uint32_t t0 = tid * kVPT;
    const int nvalid = t0 >= nv ? 0 : (int)min(16u, nv - t0);
    const uint64_t smoff = sm_offset(N, log2b);
    const uint64_t payoff = smoff + pad16(N * SMB);
    const uint8_t* msg = msgs + td.msg_off;

    // received sign-plus-mantissa: needs nothing else, so it is in flight while the bitmap is read
    Group<DT> g;
    if (nvalid == 16)
        g.load_sm_full(msg + smoff + (v0 + t0) * SMB);
    else
        g.load_sm_partial(msg + smoff + (v0 + t0) * SMB, nvalid);

    if (tid == 0) s_before = 0;
    __syncthreads();

    // positions of changed blocks from the bitmap: set bits before this tile, then the tile's own
    const uint32_t* bm32 = reinterpret_cast<const uint32_t*>(msg);
    const uint64_t kb0 = v0 >> log2b;
    const uint32_t nbt = kTileValues >> log2b;
    const uint32_t nblk = (nv + B - 1u) >> log2b;
    {
        const uint64_t nfull = kb0 >> 5;
        uint32_t cnt = 0;
        for (uint64_t w = tid; w < nfull; w += kThreads) cnt += __popc(__ldg(bm32 + w));
        if (tid == 0 && (kb0 & 31u)) cnt += __popc(__ldg(bm32 + nfull) & ((1u << (kb0 & 31u)) - 1u));
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0 && cnt) atomicAdd(&s_before, (unsigned long long)cnt);
    }
    if (warp == 0) {
        uint32_t word = 0;
        if (nbt >= 32) {
            if (lane < (nbt >> 5) && lane * 32u < nblk) {
                word = __ldg(bm32 + (kb0 >> 5) + lane);
                const uint32_t left = nblk - lane * 32u;
                if (left < 32u) word &= (1u << left) - 1u;
            }
        } else if (lane == 0) {
            word = (__ldg(bm32 + (kb0 >> 5)) >> (kb0 & 31u)) & ((1u << nblk) - 1u);
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
            s_bm[lane] = word;
            s_pre[lane] = incl - pc;
        }
        if (lane == 31) s_tot = incl;
    }
    __syncthreads();

    if (nvalid > 0) {
        const uint32_t kb = t0 >> log2b;
        const uint32_t word = s_bm[kb >> 5];
        const bool chg = (word >> (kb & 31u)) & 1u;
        uint8_t* cptr = cache + td.c_off + t0;
        const uint8_t* src = cptr;  // unchanged block: the cached exponents
        if (chg) {                  // changed block: its exponents are in the payload
            const uint64_t rank = s_before + s_pre[kb >> 5] + __popc(word & ((1u << (kb & 31u)) - 1u));
            src = msg + payoff + (rank << log2b) + (t0 & (B - 1u));
        }
        if (nvalid == 16) {
            const uint4 ev = ld_stream16(src);
            g.e[0] = ev.x; g.e[1] = ev.y; g.e[2] = ev.z; g.e[3] = ev.w;
            if (chg) st_stream16(cptr, ev);  // ExpCache[i,k] <- newExp[j]
            g.merge_store_full(weights + td.w_off + (uint64_t)t0 * VB);
        } else {
            load_exp_partial(g.e, src, nvalid);
            if (chg) store_exp_partial(cptr, g.e, nvalid);
            g.merge_store_partial(weights + td.w_off + (uint64_t)t0 * VB, nvalid);
        }
    }

    // optional integrity check by the unit's last tile: the bitmap fixes the message length
    if (wire_bytes != nullptr && status != nullptr && tid == 0 && td.tile_in_unit == td.n_tiles_unit - 1u) {
        uint64_t total = (s_before + s_tot) << log2b;
        const uint32_t rem = nv & (B - 1u);
        if (rem) {
            const uint32_t kb = nv >> log2b;
            if ((s_bm[kb >> 5] >> (kb & 31u)) & 1u) total -= (B - rem);
        }
        if (wire_bytes[td.unit] != payoff + total) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
    }
}

// ------------------------------------------------------------------------------------------
// cache := exponents(weights)  (or zero)

template <int DT>
__global__ void __launch_bounds__(kThreads)
cache_fill_kernel(const TileDesc* __restrict__ tiles, const uint8_t* __restrict__ weights, uint8_t* __restrict__ cache) {
    constexpr int VB = Traits<DT>::kValueBytes;
    const TileDesc td = load_tile_desc(tiles + blockIdx.x);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
    const uint32_t t0 = threadIdx.x * kVPT;
    const int nvalid = t0 >= nv ? 0 : (int)min(16u, nv - t0);
    if (nvalid == 0) return;
    Group<DT> g;
    g.e[0] = g.e[1] = g.e[2] = g.e[3] = 0;
    if (weights != nullptr) {
        if (nvalid == 16)
            g.split_full(weights + td.w_off + (uint64_t)t0 * VB);
        else
            g.split_partial(weights + td.w_off + (uint64_t)t0 * VB, nvalid);
    }
    if (nvalid == 16)
        st_stream16(cache + td.c_off + t0, make_uint4(g.e[0], g.e[1], g.e[2], g.e[3]));
    else
        store_exp_partial(cache + td.c_off + t0, g.e, nvalid);
}

// ------------------------------------------------------------------------------------------
// transport stand-in: copy the used bytes of every slot

__global__ void __launch_bounds__(kThreads)
transport_kernel(const TileDesc* __restrict__ tiles, uint32_t sm_bytes_per_value, const uint8_t* __restrict__ src,
                 uint8_t* __restrict__ dst, const unsigned long long* __restrict__ wire_bytes) {
    const TileDesc td = load_tile_desc(tiles + blockIdx.x);
    const uint64_t used = wire_bytes[td.unit];
    const uint64_t chunk = transport_chunk_bytes(sm_bytes_per_value);
    const uint64_t lo = (uint64_t)td.tile_in_unit * chunk;
    if (lo >= used) return;
    const uint64_t hi = min(lo + chunk, used);
    const uint8_t* s = src + td.msg_off + lo;
    uint8_t* d = dst + td.msg_off + lo;
    const uint32_t nvec = (uint32_t)((hi - lo) >> 4);
    for (uint32_t i = threadIdx.x; i < nvec; i += kThreads) st_stream16(d + 16ull * i, ld_stream16(s + 16ull * i));
    const uint32_t tail = (uint32_t)((hi - lo) & 15ull);
    if (threadIdx.x < tail) d[16ull * nvec + threadIdx.x] = s[16ull * nvec + threadIdx.x];
}

}  // namespace ciera

// ------------------------------------------------------------------------------------------
// launchers

using namespace ciera;

static int check_plan(const ciera_plan* p) {
    if (!p) return CIERA_ERR_INVALID_ARG;
    if (!p->tiles.empty() && !p->tiles_dev) return CIERA_ERR_NOT_BOUND;
    return CIERA_OK;
}
static bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

static int cache_fill(const ciera_plan* p, void* cache_dev, const void* weights_dev, void* stream) {
    int rc = check_plan(p);
    if (rc) return rc;
    if (!cache_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(cache_dev) || misaligned16(weights_dev)) return CIERA_ERR_MISALIGNED;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    cudaStream_t s = (cudaStream_t)stream;
    if (p->dtype == CIERA_BF16)
        cache_fill_kernel<CIERA_BF16><<<nt, kThreads, 0, s>>>(p->tiles_dev, (const uint8_t*)weights_dev, (uint8_t*)cache_dev);
    else
        cache_fill_kernel<CIERA_FP32><<<nt, kThreads, 0, s>>>(p->tiles_dev, (const uint8_t*)weights_dev, (uint8_t*)cache_dev);
    count_launch();
    return check_launch();
}

extern "C" int ciera_cache_init(const ciera_plan* plan, void* cache_dev, const void* weights_dev, void* stream) {
    return cache_fill(plan, cache_dev, weights_dev, stream);
}

extern "C" int ciera_cache_update(const ciera_plan* plan, void* cache_dev, const void* weights_dev, void* stream) {
    if (!weights_dev) return CIERA_ERR_INVALID_ARG;
    return cache_fill(plan, cache_dev, weights_dev, stream);
}

extern "C" int ciera_transport(const ciera_plan* p, const void* src_messages_dev, void* dst_messages_dev,
                               const uint64_t* wire_bytes_dev, void* stream) {
    int rc = check_plan(p);
    if (rc) return rc;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    if (!src_messages_dev || !dst_messages_dev || !wire_bytes_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(src_messages_dev) || misaligned16(dst_messages_dev)) return CIERA_ERR_MISALIGNED;
    transport_kernel<<<nt, kThreads, 0, (cudaStream_t)stream>>>(
        p->tiles_dev, p->dtype == CIERA_BF16 ? 1u : 3u, (const uint8_t*)src_messages_dev, (uint8_t*)dst_messages_dev,
        (const unsigned long long*)wire_bytes_dev);
    count_launch();
    return check_launch();
}

extern "C" int ciera_decode(const ciera_plan* p, const void* messages_dev, void* receiver_cache_dev,
                            void* weights_out_dev, const uint64_t* wire_bytes_dev, int32_t* status_dev, void* stream) {
    int rc = check_plan(p);
    if (rc) return rc;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    if (!messages_dev || !receiver_cache_dev || !weights_out_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(messages_dev) || misaligned16(receiver_cache_dev) || misaligned16(weights_out_dev))
        return CIERA_ERR_MISALIGNED;
    cudaStream_t s = (cudaStream_t)stream;
    if (p->dtype == CIERA_BF16)
        decode_kernel<CIERA_BF16><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)messages_dev,
                                                         (uint8_t*)receiver_cache_dev, (uint8_t*)weights_out_dev,
                                                         (const unsigned long long*)wire_bytes_dev, status_dev);
    else
        decode_kernel<CIERA_FP32><<<nt, kThreads, 0, s>>>(p->tiles_dev, p->log2b, (const uint8_t*)messages_dev,
                                                         (uint8_t*)receiver_cache_dev, (uint8_t*)weights_out_dev,
                                                         (const unsigned long long*)wire_bytes_dev, status_dev);
    count_launch();
    return check_launch();
}

extern "C" int ciera_roundtrip_host(const ciera_plan* p, const void* weights_host, size_t weights_bytes,
                                    void* weights_out_host, uint64_t* wire_bytes_host, const ciera_device_buffers* b,
                                    void* stream) {
    int rc = check_plan(p);
    if (rc) return rc;
    if (!b || !weights_host || !weights_out_host) return CIERA_ERR_INVALID_ARG;
    if (p->tiles.empty()) return CIERA_OK;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(b->weights_dev, weights_host, weights_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return record_cuda_error(e);
    rc = ciera_encode(p, b->weights_dev, b->sender_cache_dev, b->msg_send_dev, b->wire_bytes_dev, b->changed_blocks_dev,
                      b->workspace_dev, b->status_dev, stream);
    if (rc) return rc;
    rc = ciera_transport(p, b->msg_send_dev, b->msg_recv_dev, b->wire_bytes_dev, stream);
    if (rc) return rc;
    rc = ciera_decode(p, b->msg_recv_dev, b->receiver_cache_dev, b->weights_out_dev, b->wire_bytes_dev, b->status_dev,
                      stream);
    if (rc) return rc;
    e = cudaMemcpyAsync(weights_out_host, b->weights_out_dev, weights_bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (wire_bytes_host) {
        e = cudaMemcpyAsync(wire_bytes_host, b->wire_bytes_dev, sizeof(uint64_t) * p->n_units, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return record_cuda_error(e);
    }
    return CIERA_OK;
}
