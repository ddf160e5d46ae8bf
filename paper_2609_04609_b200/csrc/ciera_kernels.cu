// Auxiliary sm_100a kernels of libciera: cache initialisation, the transport stand-in, and the
// host-buffer round trip.  (Encode and decode live in ciera_encode.cu / ciera_decode.cu.)
#include "ciera_bits.cuh"
#include "ciera_lookback.cuh"
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
// Tile j of a unit moves bytes [j * chunk, (j + 1) * chunk) of the unit's slot (chunk = 16 KB for
// bf16 and fp16, 32 KB for fp32, plus a tile's share of the bitmap when blocks are fine), the last
// tile also what lies beyond, cut off at the length the sender reported.  A reported length beyond
// what a message of the unit can ever take (every block changed) cannot come from a finished sender
// step -- it is a stale or damaged word, e.g. of a unit that an aborted encode left unfinished: such a
// unit moves nothing and raises CIERA_ERR_CORRUPT, so that no copy ever leaves the unit's slot.

// largest message of a unit of n values: all sections with every block changed (device twin of
// ciera_message_capacity)
__device__ __forceinline__ uint64_t slot_capacity(uint64_t n, int dtype, uint32_t log2b) {
    if (n == 0) return 0;
    const uint64_t nb = num_blocks(n, log2b);
    return payload_offset_of(n, dtype, log2b) + (nb - 1) * block_payload_bytes(1ull << log2b, dtype) +
           block_payload_bytes(n - ((nb - 1) << log2b), dtype);
}

// the part of a tile descriptor the copy needs (keeps the prefetched copies small in registers)
struct CopyDesc {
    uint64_t msg_off;
    uint64_t n_unit;
    uint32_t unit, tile_in_unit, n_tiles_unit;
};
__device__ __forceinline__ CopyDesc load_copy_desc(const TileDesc* t) {
    const uint4* p = reinterpret_cast<const uint4*>(t);
    const uint4 b = __ldg(p + 1), c = __ldg(p + 2);
    CopyDesc d;
    d.msg_off = (uint64_t)b.x | ((uint64_t)b.y << 32);
    d.n_unit = (uint64_t)b.z | ((uint64_t)b.w << 32);
    d.unit = c.x;
    d.tile_in_unit = c.y;
    d.n_tiles_unit = c.w;
    return d;
}

// A persistent kernel in which the loads are done by the copy engine.  A producer warp draws tiles from the
// counter, kPipeBatch at a time (one per lane: descriptors and reported lengths of a batch are
// fetched in parallel and two batches ahead, so tiles beyond the used part of their messages cost
// next to nothing), cuts each tile's byte range into pieces of at most kPipeStage bytes and starts
// one bulk-async copy per piece into a ring of shared-memory stages; eight consumer warps move every
// stage to its destination with 128-bit stores and hand it back.  Loads in flight then cost no
// registers and no issue slots, and the stores of one stage overlap the loads of the next ones.
constexpr uint32_t kPipeStage = 16384;
constexpr int kPipeStages = 6;
constexpr int kPipeConsumers = 8;                        // warps
constexpr int kPipeThreads = 32 * (kPipeConsumers + 1);  // + the producer warp
constexpr uint32_t kPipeBatch = 3;                       // tiles drawn at a time (measured: 3 beats 2, 4 and 8)

struct PipeSlot {
    uint8_t* dst;
    const uint8_t* tail_src;  // where the piece's last (hi - lo) % 16 bytes come from
    uint32_t bytes;           // 0xffffffff: no more work
    uint32_t pad;
};
struct PipeCtl {
    uint64_t full[kPipeStages];
    uint64_t empty[kPipeStages];
    PipeSlot slot[kPipeStages];
    int abort;
    uint32_t issued, seen;
};

__global__ void __launch_bounds__(kPipeThreads, 2)
transport_pipe_kernel(const TileDesc* __restrict__ tiles, uint32_t n_tiles, uint64_t chunk, int dtype, uint32_t log2b,
                      const uint8_t* __restrict__ src, uint8_t* __restrict__ dst,
                      const unsigned long long* __restrict__ wire_bytes, unsigned int* ticket, int32_t* status) {
    extern __shared__ __align__(128) uint8_t smem[];
    PipeCtl* ctl = reinterpret_cast<PipeCtl*>(smem + (size_t)kPipeStages * kPipeStage);
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    volatile int* abort = &ctl->abort;
    if (tid == 0) {
        for (int s = 0; s < kPipeStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kPipeConsumers);
        }
        ctl->abort = 0;
        ctl->issued = 0;
        ctl->seen = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == kPipeConsumers) {
        // ---------------------------------------------------------------- producer warp
        // every lane below kPipeBatch carries one tile through three steps: number (t_a), descriptor
        // (td_b), descriptor and reported length (td_c, used_c); a step's loads are used one batch later
        auto draw = [&]() {
            uint32_t base = 0;
            if (lane == 0) base = atomicAdd(ticket, kPipeBatch);
            base = __shfl_sync(0xffffffffu, base, 0);
            return lane < kPipeBatch ? base + lane : n_tiles;
        };
        uint32_t t_a = draw(), t_b = n_tiles, t_c = n_tiles;
        CopyDesc td_b, td_c;
        unsigned long long used_c = 0;
        auto advance = [&]() {
            td_c = td_b;
            t_c = t_b;
            if (t_c < n_tiles) {
                used_c = __ldg(wire_bytes + td_c.unit);
                if (used_c > slot_capacity(td_c.n_unit, dtype, log2b)) {  // not a length any sender step reports
                    if (status) atomicCAS(status, 0, (int32_t)CIERA_ERR_CORRUPT);
                    used_c = 0;
                }
            }
            t_b = t_a;
            if (t_b < n_tiles) td_b = load_copy_desc(tiles + t_b);
            // once a batch starts past the end there is nothing more to draw
            t_a = __any_sync(0xffffffffu, t_a < n_tiles) ? draw() : n_tiles;
        };
        advance();
        advance();
        uint32_t k = 0;  // pieces issued so far (lane 0)
        bool ok = true;
        while (ok && __any_sync(0xffffffffu, t_c < n_tiles)) {
            // this batch's byte ranges
            uint64_t lo = 0, hi = 0, off = 0;
            if (t_c < n_tiles) {
                off = td_c.msg_off;
                lo = (uint64_t)td_c.tile_in_unit * chunk;
                const bool last = td_c.tile_in_unit == td_c.n_tiles_unit - 1u;
                hi = (last || lo + chunk >= used_c) ? used_c : lo + chunk;
                if (lo >= used_c) hi = lo;  // beyond the used part: nothing to move
            }
            advance();  // the next batches' loads go out before this batch is worked on
            uint32_t todo = __ballot_sync(0xffffffffu, lo < hi);
            while (ok && todo) {
                const int l = __ffs(todo) - 1;
                todo &= todo - 1;
                uint64_t p_lo = __shfl_sync(0xffffffffu, lo, l);
                const uint64_t p_hi = __shfl_sync(0xffffffffu, hi, l);
                const uint64_t p_off = __shfl_sync(0xffffffffu, off, l);
                if (lane == 0) {
                    while (p_lo < p_hi) {
                        const uint32_t bytes = (uint32_t)min((uint64_t)kPipeStage, p_hi - p_lo);
                        const uint32_t st = k % kPipeStages;
                        if (k >= (uint32_t)kPipeStages &&
                            !mbar_wait(&ctl->empty[st], ((k / kPipeStages) & 1u) ^ 1u, abort, status)) {
                            ok = false;
                            break;
                        }
                        const uint32_t body = bytes & ~15u;
                        ctl->slot[st].dst = dst + p_off + p_lo;
                        ctl->slot[st].tail_src = src + p_off + p_lo + body;
                        ctl->slot[st].bytes = bytes;
                        if (body) {
                            mbar_arrive_expect_tx(&ctl->full[st], body);
                            bulk_load(smem + (size_t)st * kPipeStage, src + p_off + p_lo, body, &ctl->full[st]);
                        } else {
                            mbar_arrive(&ctl->full[st]);
                        }
                        ctl->issued = ++k;
                        p_lo += bytes;
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            }
        }
        // this block draws no more numbers: the last block to get here hands the counter (and the count of
        // blocks that got here, in the word behind it) back at zero, as the next call expects to find them
        if (lane == 0) {
            __threadfence();
            if (atomicAdd(ticket + 1, 1u) + 1u == gridDim.x) {
                __threadfence();
                ticket[0] = 0u;
                ticket[1] = 0u;
            }
        }
        if (lane == 0 && ok) {  // end marker
            const uint32_t st = k % kPipeStages;
            if (k < (uint32_t)kPipeStages || mbar_wait(&ctl->empty[st], ((k / kPipeStages) & 1u) ^ 1u, abort, status)) {
                ctl->slot[st].bytes = 0xffffffffu;
                mbar_arrive(&ctl->full[st]);
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers
        for (uint32_t k = 0;; ++k) {
            const uint32_t st = k % kPipeStages;
            if (!mbar_wait(&ctl->full[st], (k / kPipeStages) & 1u, abort, status)) break;
            if (tid == 0) ctl->seen = k + 1;
            const PipeSlot sl = ctl->slot[st];
            if (sl.bytes == 0xffffffffu) break;
            const uint32_t nvec = sl.bytes >> 4;
            const uint8_t* from = smem + (size_t)st * kPipeStage;
            for (uint32_t i = tid; i < nvec; i += 32u * kPipeConsumers) st_stream16(sl.dst + 16ull * i, ld_shared16(from + 16ull * i));
            const uint32_t tail = sl.bytes & 15u;  // only the last piece of a message can have one
            if (warp == 0 && lane < tail) sl.dst[16ull * nvec + lane] = sl.tail_src[lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->empty[st]);
        }
    }
    __syncthreads();
    if (tid == 0 && ctl->abort) {  // after an aborted run wait (bounded) for bulk copies still in flight
        for (uint32_t k = ctl->seen; k < ctl->issued; ++k)
            for (uint32_t i = 0; i < kMaxBarrierPolls; ++i)
                if (mbar_try_wait(&ctl->full[k % kPipeStages], (k / kPipeStages) & 1u)) break;
    }
}

static int transport_pipe_grid_limit(int* out) {
    static std::atomic<int> cached[64];  // (zero-initialised; any host thread may be the first to fill an entry)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return CIERA_ERR_UNSUPPORTED;
    if (cached[dev].load(std::memory_order_acquire) == 0) {
        const size_t smem = (size_t)kPipeStages * kPipeStage + sizeof(PipeCtl);
        e = cudaFuncSetAttribute(transport_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        int per_sm = 0, sms = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, transport_pipe_kernel, kPipeThreads, smem);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (per_sm < 1 || sms < 1) return CIERA_ERR_UNSUPPORTED;
        cached[dev].store(per_sm * sms, std::memory_order_release);
    }
    *out = cached[dev].load(std::memory_order_acquire);
    return CIERA_OK;
}

// ------------------------------------------------------------------------------------------
// Self-test of the bounded waits: both kinds of wait the persistent kernels use -- the poll of a
// look-back status word in global memory and the wait on a shared-memory barrier -- are run with a
// short limit on a word and a barrier that nobody ever completes.  Each must give up, raise
// CIERA_ERR_TIMEOUT in the status word and return; the kernel then leaves normally.  Nothing traps,
// nothing spins at the kernels' own limits, and no other kernel is involved.
//   report[0] = 1: the status-word wait gave up and returned "prefix 0"
//   report[1] = 1: the barrier wait gave up (returned false)
//   report[2] = the block's abort flag afterwards (1 expected)
//   report[3] = polls the barrier wait was given
__global__ void __launch_bounds__(64)
selftest_waits_kernel(const unsigned long long* never_written, uint32_t max_polls, int32_t* status, int32_t* report) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long st = wait_status(never_written, status, max_polls);
        report[0] = (st == kFlagPrefix) ? 1 : 0;
    } else if (threadIdx.x == 32) {
        const bool ok = mbar_wait(&bar, 0u, &abort_flag, status, max_polls);
        report[1] = ok ? 0 : 1;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        report[2] = abort_flag;
        report[3] = (int32_t)max_polls;
    }
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
    if (p->dtype == CIERA_FP16)
        cache_fill_kernel<CIERA_FP16><<<nt, kThreads, 0, s>>>(p->tiles_dev, (const uint8_t*)weights_dev, (uint8_t*)cache_dev);
    else if (p->dtype == CIERA_BF16)
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
                               const uint64_t* wire_bytes_dev, void* workspace_dev, int32_t* status_dev, void* stream) {
    int rc = check_plan(p);
    if (rc) return rc;
    const uint32_t nt = (uint32_t)p->tiles.size();
    if (nt == 0) return CIERA_OK;
    if (!src_messages_dev || !dst_messages_dev || !wire_bytes_dev || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if (misaligned16(src_messages_dev) || misaligned16(dst_messages_dev) || misaligned16(workspace_dev))
        return CIERA_ERR_MISALIGNED;
    // the tile counter (see the layout of the scratch in ciera_internal.cuh): found at zero, handed back at zero
    unsigned int* ticket = (unsigned int*)((uint8_t*)workspace_dev + workspace_ticket_offset(nt));
    int limit = 0;
    rc = transport_pipe_grid_limit(&limit);
    if (rc) return rc;
    const uint32_t want_blocks = (nt + kPipeBatch - 1) / kPipeBatch;
    const uint32_t grid = want_blocks < (uint32_t)limit ? want_blocks : (uint32_t)limit;
    transport_pipe_kernel<<<grid, kPipeThreads, (size_t)kPipeStages * kPipeStage + sizeof(PipeCtl), (cudaStream_t)stream>>>(
        p->tiles_dev, nt, transport_chunk_bytes(p->dtype == CIERA_FP32 ? 3u : 1u, p->log2b), p->dtype, p->log2b,
        (const uint8_t*)src_messages_dev, (uint8_t*)dst_messages_dev, (const unsigned long long*)wire_bytes_dev, ticket,
        status_dev);
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
    rc = ciera_transport(p, b->msg_send_dev, b->msg_recv_dev, b->wire_bytes_dev, b->workspace_dev, b->status_dev, stream);
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

extern "C" int ciera_selftest_bounded_waits(uint32_t max_polls, void* scratch_dev, int32_t* status_dev, int32_t* report_dev,
                                            void* stream) {
    if (!scratch_dev || !status_dev || !report_dev) return CIERA_ERR_INVALID_ARG;
    if (max_polls == 0 || max_polls > 4096) return CIERA_ERR_INVALID_ARG;  // a self-test, not a way to stall the GPU
    if (((uintptr_t)scratch_dev & 7u) || ((uintptr_t)status_dev & 3u) || ((uintptr_t)report_dev & 3u))
        return CIERA_ERR_MISALIGNED;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(scratch_dev, 0, 8, s);  // the word that is polled: empty, and nobody fills it
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaMemsetAsync(report_dev, 0, 16, s);
    if (e != cudaSuccess) return record_cuda_error(e);
    selftest_waits_kernel<<<1, 64, 0, s>>>((const unsigned long long*)scratch_dev, max_polls, status_dev, report_dev);
    count_launch();
    return check_launch();
}
