// Auxiliary sm_100a kernels of libciera: cache initialisation, the transport stand-in, and the
// host-buffer round trip.  (Encode and decode live in ciera_encode.cu / ciera_decode.cu.)
#include "ciera_bits.cuh"
#include "ciera_pipe.cuh"

namespace ciera {

// ------------------------------------------------------------------------------------------
// cache := exponents(weights)  (or zero)

template <int DT>
__global__ void __launch_bounds__(kThreads)
cache_fill_kernel(const TileDesc* __restrict__ tiles, const uint8_t* __restrict__ weights, uint8_t* __restrict__ cache) {
    using P = Piece<DT>;
    constexpr int VB = Traits<DT>::kValueBytes;
    const TileDesc td = load_tile_desc(tiles + blockIdx.x);
    const uint64_t v0 = (uint64_t)td.tile_in_unit * kTileValues;
    const uint32_t nv = (uint32_t)min((uint64_t)kTileValues, td.n_unit - v0);
#pragma unroll
    for (int p = 0; p < P::kPerThread; ++p) {
        const uint32_t t0 = P::start(threadIdx.x, p);
        const int nvalid = piece_valid<DT>(t0, nv);
        if (nvalid == 0) continue;
        P x;
#pragma unroll
        for (int i = 0; i < P::kExpWords; ++i) x.e[i] = 0;
        if (weights != nullptr) {
            if (nvalid == P::kValues)
                x.template split_full<Global>(weights + td.w_off + (uint64_t)t0 * VB);
            else
                x.split_partial(weights + td.w_off + (uint64_t)t0 * VB, nvalid);
        }
        if (nvalid == P::kValues)
            x.template store_exp_full<Global>(cache + td.c_off + t0);
        else
            x.store_exp_partial(cache + td.c_off + t0, nvalid);
    }
}

// ------------------------------------------------------------------------------------------
// transport stand-in: copy the used bytes of every slot
//
// A persistent copy kernel in which every warp works on its own: it draws tile numbers from a
// counter in the caller's scratch (so all SMs stay busy to the end whatever their pace); tile j of
// a unit moves bytes [j * chunk, (j + 1) * chunk) of the unit's slot (chunk = 16 KB for bf16, 32 KB
// for fp32, plus a tile's share of the bitmap when blocks are fine), the last tile also what lies beyond, cut off at the length the sender reported.  A warp moves 4 KB per step (eight 128-bit loads per lane in flight, then eight
// stores); tile numbers, descriptors and reported lengths are fetched three, two and one tile
// ahead, so that no step waits for them.

constexpr int kCopyThreads = 256;
constexpr int kCopyUnroll = 8;  // 128-bit loads in flight per lane

// the part of a tile descriptor the copy needs (keeps the prefetched copies small in registers)
struct CopyDesc {
    uint64_t msg_off;
    uint32_t unit, tile_in_unit, n_tiles_unit;
};
__device__ __forceinline__ CopyDesc load_copy_desc(const TileDesc* t) {
    const uint4* p = reinterpret_cast<const uint4*>(t);
    const uint4 b = __ldg(p + 1), c = __ldg(p + 2);
    CopyDesc d;
    d.msg_off = (uint64_t)b.x | ((uint64_t)b.y << 32);
    d.unit = c.x;
    d.tile_in_unit = c.y;
    d.n_tiles_unit = c.w;
    return d;
}

__global__ void __launch_bounds__(kCopyThreads)
transport_kernel(const TileDesc* __restrict__ tiles, uint32_t n_tiles, uint64_t chunk,
                 const uint8_t* __restrict__ src, uint8_t* __restrict__ dst,
                 const unsigned long long* __restrict__ wire_bytes, unsigned int* ticket) {
    const uint32_t lane = threadIdx.x & 31u;
    auto draw = [&]() {
        uint32_t t = 0;
        if (lane == 0) t = atomicAdd(ticket, 1u);
        return __shfl_sync(0xffffffffu, t, 0);
    };
    // three-deep software pipeline: tile number drawn (t_c), descriptor loaded (t_b, td_b), reported
    // length loaded (t_a, td_a, used_a)
    uint32_t t_a = draw(), t_b = draw(), t_c = draw();
    CopyDesc td_a, td_b;
    unsigned long long used_a = 0;
    if (t_a < n_tiles) {
        td_a = load_copy_desc(tiles + t_a);
        used_a = __ldg(wire_bytes + td_a.unit);
    }
    if (t_b < n_tiles) td_b = load_copy_desc(tiles + t_b);
    while (t_a < n_tiles) {
        const CopyDesc td = td_a;
        const uint64_t used = used_a;
        // advance the pipeline; none of these loads is needed before the next iteration
        const uint32_t t_d = t_c < n_tiles ? draw() : n_tiles;
        td_a = td_b;
        if (t_b < n_tiles) used_a = __ldg(wire_bytes + td_a.unit);
        if (t_c < n_tiles) td_b = load_copy_desc(tiles + t_c);
        t_a = t_b;
        t_b = t_c;
        t_c = t_d;

        const uint64_t lo = (uint64_t)td.tile_in_unit * chunk;
        if (lo >= used) continue;
        // the unit's last tile also takes what lies beyond tiles * chunk
        const bool last = td.tile_in_unit == td.n_tiles_unit - 1u;
        const uint64_t hi = (last || lo + chunk >= used) ? used : lo + chunk;
        const uint8_t* s = src + td.msg_off + lo;
        uint8_t* d = dst + td.msg_off + lo;
        const uint32_t nvec = (uint32_t)((hi - lo) >> 4);  // 16-byte pieces
        uint32_t i = lane;
        for (; i + 32u * (kCopyUnroll - 1) < nvec; i += 32u * kCopyUnroll) {
            uint4 v[kCopyUnroll];
#pragma unroll
            for (int u = 0; u < kCopyUnroll; ++u) v[u] = ld_stream16(s + 16ull * (i + 32u * u));
#pragma unroll
            for (int u = 0; u < kCopyUnroll; ++u) st_stream16(d + 16ull * (i + 32u * u), v[u]);
        }
        for (; i < nvec; i += 32u) st_stream16(d + 16ull * i, ld_stream16(s + 16ull * i));
        // a ragged end (fewer than 16 bytes; only the last tile of a message can have one)
        const uint32_t tail = (uint32_t)((hi - lo) & 15ull);
        if (lane < tail) d[16ull * nvec + lane] = s[16ull * nvec + lane];
    }
}

static int transport_grid_limit(int* out) {
    static int cached[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    if (cached[dev] == 0) {
        int per_sm = 0, sms = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, transport_kernel, kCopyThreads, 0);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (per_sm < 1 || sms < 1) return CIERA_ERR_UNSUPPORTED;
        cached[dev] = per_sm * sms;
    }
    *out = cached[dev];
    return CIERA_OK;
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
    if (p->dtype == CIERA_FP16) return fp16_cache_fill(p, cache_dev, weights_dev, s);
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
                               const uint64_t* wire_bytes_dev, void* workspace_dev, void* stream) {
    int rc = check_plan(p);
    if (rc) return rc;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    if (!src_messages_dev || !dst_messages_dev || !wire_bytes_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(src_messages_dev) || misaligned16(dst_messages_dev) || misaligned16(workspace_dev))
        return CIERA_ERR_MISALIGNED;
    // the tile counter sits past the per-tile words of the scratch and starts at zero
    unsigned int* ticket = (unsigned int*)((unsigned long long*)workspace_dev + nt);
    cudaError_t me = cudaMemsetAsync(ticket, 0, 16, (cudaStream_t)stream);
    if (me != cudaSuccess) return record_cuda_error(me);
    int limit = 0;
    rc = transport_grid_limit(&limit);
    if (rc) return rc;
    const uint32_t want = (nt + kCopyThreads / 32 - 1) / (kCopyThreads / 32);
    const uint32_t grid = want < (uint32_t)limit ? want : (uint32_t)limit;
    transport_kernel<<<grid, kCopyThreads, 0, (cudaStream_t)stream>>>(
        p->tiles_dev, nt, transport_chunk_bytes(p->dtype == CIERA_FP32 ? 3u : 1u, p->log2b), (const uint8_t*)src_messages_dev, (uint8_t*)dst_messages_dev,
        (const unsigned long long*)wire_bytes_dev, ticket);
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
    rc = ciera_transport(p, b->msg_send_dev, b->msg_recv_dev, b->wire_bytes_dev, b->workspace_dev, stream);
    if (rc) return rc;
    rc = ciera_decode(p, b->msg_recv_dev, b->receiver_cache_dev, b->weights_out_dev, b->wire_bytes_dev,
                      b->workspace_dev, b->status_dev, stream);
    if (rc) return rc;
    e = cudaMemcpyAsync(weights_out_host, b->weights_out_dev, weights_bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (wire_bytes_host) {
        e = cudaMemcpyAsync(wire_bytes_host, b->wire_bytes_dev, sizeof(uint64_t) * p->n_units, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return record_cuda_error(e);
    }
    return CIERA_OK;
}
