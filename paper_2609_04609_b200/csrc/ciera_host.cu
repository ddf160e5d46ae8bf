// Host side of libciera: size rules, the plan (tile table), the gain rule, diagnostics.
#include <string.h>

#include <algorithm>
#include <new>

#include "ciera_internal.cuh"

namespace ciera {

static thread_local int g_last_cuda_error = 0;
static std::atomic<uint64_t> g_launches{0};

int record_cuda_error(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return CIERA_ERR_CUDA;
}
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
int check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error(e);
    return CIERA_OK;
}

static bool valid_dtype(int dtype) { return dtype == CIERA_BF16 || dtype == CIERA_FP32 || dtype == CIERA_FP16; }
static uint32_t value_bytes_of(int dtype) { return dtype == CIERA_FP32 ? 4u : 2u; }

// log2 of a power of two, or -1.
static int exact_log2(uint32_t x) {
    if (x == 0 || (x & (x - 1))) return -1;
    int l = 0;
    while ((1u << l) != x) ++l;
    return l;
}

}  // namespace ciera

using namespace ciera;

// ---------------------------------------------------------------------------------- sizes

extern "C" size_t ciera_sm_offset(uint64_t n, uint32_t block) {
    if (block == 0) return 0;
    uint64_t nb = (n + block - 1) / block;
    return (size_t)pad16((nb + 7) / 8);
}

extern "C" size_t ciera_payload_offset(uint64_t n, int dtype, uint32_t block) {
    if (block == 0 || !valid_dtype(dtype)) return 0;
    return ciera_sm_offset(n, block) + (size_t)pad16(sm_section_bytes(n, dtype));
}

extern "C" size_t ciera_message_capacity(uint64_t n, int dtype, uint32_t block) {
    if (n == 0 || block == 0 || !valid_dtype(dtype)) return 0;
    // every block changed: full blocks and the (possibly short) last one
    const uint64_t nb = (n + block - 1) / block;
    return ciera_payload_offset(n, dtype, block) +
           (size_t)((nb - 1) * block_payload_bytes(block, dtype) + block_payload_bytes(n - (nb - 1) * block, dtype));
}

extern "C" size_t ciera_message_bytes(uint64_t n, int dtype, uint32_t block, uint64_t payload_bytes) {
    if (block == 0 || !valid_dtype(dtype)) return 0;
    uint64_t nb = (n + block - 1) / block;
    return (size_t)(sm_section_bytes(n, dtype) + (nb + 7) / 8 + payload_bytes);
}

// ---------------------------------------------------------------------------------- plan

namespace {
struct ImageLayout {
    size_t tiles, long_off, seq_off, hash_off, first_off, seg_off, units_off, elong_off, echunk_off, thash_off, runs_off, total;
};
size_t up16(size_t x) { return (x + 15) / 16 * 16; }
ImageLayout image_layout(const ciera_plan* p) {
    ImageLayout L;
    L.tiles = p->tiles.size() * sizeof(TileDesc);
    L.long_off = L.tiles;
    L.seq_off = L.long_off + up16(p->long_units.size() * sizeof(uint32_t));
    L.hash_off = L.seq_off + up16(p->seq_first.size() * sizeof(uint32_t));
    L.first_off = L.hash_off + up16((size_t)p->n_units * sizeof(uint64_t));
    L.seg_off = L.first_off + up16((size_t)p->n_units * sizeof(uint32_t));
    L.units_off = L.seg_off + up16((size_t)p->n_units * sizeof(uint64_t));
    L.elong_off = L.units_off + up16((size_t)p->n_units * sizeof(ciera_unit));
    L.echunk_off = L.elong_off + up16(p->ent_long_units.size() * sizeof(uint32_t));
    L.thash_off = L.echunk_off + up16(p->ent_chunks.size() * sizeof(ciera_plan::EntChunk));
    L.runs_off = L.thash_off + up16(p->tiles.size() * sizeof(uint64_t));
    L.total = L.runs_off + p->seq_runs.size() * sizeof(ciera_plan::SeqRun) + 16;
    return L;
}
}  // namespace

extern "C" int ciera_plan_create(const ciera_unit* units_host, uint32_t n_units, int dtype, uint32_t block,
                                 ciera_plan** plan_out) {
    if (!plan_out) return CIERA_ERR_INVALID_ARG;
    *plan_out = nullptr;
    if ((!units_host && n_units) || !valid_dtype(dtype)) return CIERA_ERR_INVALID_ARG;
    if (block == 0) return CIERA_ERR_INVALID_ARG;
    int l2 = exact_log2(block);
    if (l2 < 0 || block < CIERA_MIN_BLOCK || block > CIERA_MAX_BLOCK) return CIERA_ERR_UNSUPPORTED;

    uint64_t n_tiles = 0, total = 0;
    for (uint32_t u = 0; u < n_units; ++u) {
        const ciera_unit& un = units_host[u];
        if ((un.weights_off | un.cache_off | un.msg_off) & 15ull) return CIERA_ERR_MISALIGNED;
        if (un.n_values >= (1ull << 48)) return CIERA_ERR_UNSUPPORTED;
        if ((un.n_values + block - 1) / block > 0xffffffffull) return CIERA_ERR_UNSUPPORTED;  // block counts are 32-bit
        if (un.msg_capacity < ciera_message_capacity(un.n_values, dtype, block)) return CIERA_ERR_CAPACITY;
        n_tiles += (un.n_values + kTileValues - 1) / kTileValues;
        total += un.n_values;
    }
    if (n_tiles >= 0x7fffffffull) return CIERA_ERR_UNSUPPORTED;  // grid.x limit

    ciera_plan* p = new (std::nothrow) ciera_plan;
    if (!p) return CIERA_ERR_INVALID_ARG;
    p->dtype = dtype;
    p->block = block;
    p->log2b = (uint32_t)l2;
    p->n_units = n_units;
    p->total_values = total;
    for (uint32_t u = 0; u < n_units; ++u) p->has_empty_units |= units_host[u].n_values == 0;
    p->units.assign(units_host, units_host + n_units);
    p->tiles.reserve((size_t)n_tiles);
    const uint32_t vb = value_bytes_of(dtype);
    // processing order: short units by descending tile count (ties in table order), then the rest
    auto tiles_of = [&](uint32_t u) { return (uint32_t)((units_host[u].n_values + kTileValues - 1) / kTileValues); };
    std::vector<uint32_t> shorts, longs;
    for (uint32_t u = 0; u < n_units; ++u) {
        const uint32_t nt = tiles_of(u);
        if (nt == 0) continue;
        (nt <= kSeqMaxTiles ? shorts : longs).push_back(u);
    }
    std::stable_sort(shorts.begin(), shorts.end(), [&](uint32_t a, uint32_t b) { return tiles_of(a) > tiles_of(b); });
    auto emit = [&](uint32_t u) {
        const ciera_unit& un = units_host[u];
        const uint32_t nt = tiles_of(u);
        const uint32_t first = (uint32_t)p->tiles.size();
        for (uint32_t j = 0; j < nt; ++j) {
            TileDesc t;
            t.w_off = un.weights_off + (uint64_t)j * kTileValues * vb;
            t.c_off = un.cache_off + (uint64_t)j * kTileValues;
            t.msg_off = un.msg_off;
            t.n_unit = un.n_values;
            t.unit = u;
            t.tile_in_unit = j;
            t.first_tile = first;
            t.n_tiles_unit = nt;
            p->tiles.push_back(t);
        }
        const bool needs_prefix = is_fine(p->log2b) ? nt > 1 : (un.n_values + block - 1) / block > kDecodeDirectBlocks;
        if (needs_prefix) p->long_units.push_back(first);
    };
    for (uint32_t u : shorts) {
        p->seq_first.push_back((uint32_t)p->tiles.size());
        emit(u);
    }
    p->seq_first.push_back((uint32_t)p->tiles.size());
    // The short units' runs of tiles, in the order they are handed out: every unit's first run, then every unit's
    // second run.  A unit of more than kSeqRunTiles tiles is cut into a long first run and a last run of at most
    // kSeqRunTiles tiles (the first run ends on a multiple of kSeqRunTiles, so that tiles sharing a bitmap byte --
    // blocks of 2048 and 4096 values -- stay in one run).  Every start of a run costs the thread block a round
    // trip (the run's place in the table, the status word the run before it left), so runs should be few; but the
    // launch ends with the blocks working on the last runs, and the shorter those are, the closer together the
    // blocks finish.  Measured on one OLMoE-shaped layer (units of 16 tiles, 0.2848 ms with four runs of 4):
    // 8 + 4 + 4 tiles 0.2836 ms, 12 + 4 tiles 0.2823 ms (14 + 2: 0.2840, 15 + 1: 0.2857, 8 + 8: 0.2871); ending on runs of
    // 2 + 1 + 1 tiles instead 0.2932 ms.
    // (While a run's number and table entry were still waited for at its start, whole units were the faster way
    // with 16 to 128 values per block, where the aggregator warp has the least time to spare; with the look-ahead
    // runs win there too: 0.2874 against 0.2917 ms with 64 values per block, 0.2898 against 0.3005 with 128.)
    for (int pass = 0; pass < 2; ++pass) {
        for (size_t i = 0; i + 1 < p->seq_first.size(); ++i) {
            const uint32_t first = p->seq_first[i], end = p->seq_first[i + 1];
            const uint32_t n = end - first;
            const uint32_t head = n <= kSeqRunTiles ? n : (n - 1) / kSeqRunTiles * kSeqRunTiles;
            if (pass == 0)
                p->seq_runs.push_back({first, first + head});
            else if (head < n)
                p->seq_runs.push_back({first + head, end});
        }
    }
    for (uint32_t u : longs) emit(u);
    // per unit, in table order: where its tiles start and where its blocks start in a hash cache
    p->unit_first.assign(n_units, 0xffffffffu);
    for (size_t t = 0; t < p->tiles.size(); ++t)
        if (p->tiles[t].tile_in_unit == 0) p->unit_first[p->tiles[t].unit] = (uint32_t)t;
    p->hash_base.resize(n_units);
    p->seg_base.resize(n_units);
    for (uint32_t u = 0; u < n_units; ++u) {
        p->hash_base[u] = p->total_blocks;
        p->total_blocks += (units_host[u].n_values + block - 1) / block;
        // the payload of a unit has at most n_values bytes: that many 4096-byte segments
        p->seg_base[u] = p->total_segments;
        p->total_segments += (units_host[u].n_values + 4095) / 4096;
        p->cache_extent = std::max<uint64_t>(p->cache_extent, units_host[u].cache_off + units_host[u].n_values);
        const uint64_t slots = (units_host[u].n_values + 4095) / 4096;
        if (slots > 64) {  // the entropy stage spreads such a unit over several thread blocks
            const uint32_t li = (uint32_t)p->ent_long_units.size();
            p->ent_long_units.push_back(u);
            for (uint64_t g = 0; g < slots; g += 64) p->ent_chunks.push_back({u, (uint32_t)g, li, 0u});
        }
    }
    p->tile_hash.resize(p->tiles.size());
    for (size_t t = 0; t < p->tiles.size(); ++t)
        p->tile_hash[t] = p->hash_base[p->tiles[t].unit] + (uint64_t)p->tiles[t].tile_in_unit * (kTileValues >> p->log2b);
    // device image: the tile table, then (each 16-byte aligned) the index lists
    const ImageLayout L = image_layout(p);
    p->image.assign(L.total, 0);
    if (L.tiles) memcpy(p->image.data(), p->tiles.data(), L.tiles);
    if (!p->long_units.empty()) memcpy(p->image.data() + L.long_off, p->long_units.data(), p->long_units.size() * 4);
    memcpy(p->image.data() + L.seq_off, p->seq_first.data(), p->seq_first.size() * 4);
    if (!p->tile_hash.empty()) memcpy(p->image.data() + L.thash_off, p->tile_hash.data(), p->tile_hash.size() * 8);
    if (!p->seq_runs.empty())
        memcpy(p->image.data() + L.runs_off, p->seq_runs.data(), p->seq_runs.size() * sizeof(ciera_plan::SeqRun));
    if (n_units) {
        memcpy(p->image.data() + L.hash_off, p->hash_base.data(), (size_t)n_units * 8);
        memcpy(p->image.data() + L.first_off, p->unit_first.data(), (size_t)n_units * 4);
        memcpy(p->image.data() + L.seg_off, p->seg_base.data(), (size_t)n_units * 8);
        memcpy(p->image.data() + L.units_off, p->units.data(), (size_t)n_units * sizeof(ciera_unit));
        if (!p->ent_long_units.empty()) {
            memcpy(p->image.data() + L.elong_off, p->ent_long_units.data(), p->ent_long_units.size() * sizeof(uint32_t));
            memcpy(p->image.data() + L.echunk_off, p->ent_chunks.data(), p->ent_chunks.size() * sizeof(ciera_plan::EntChunk));
        }
    }
    *plan_out = p;
    return CIERA_OK;
}

extern "C" void ciera_plan_destroy(ciera_plan* plan) { delete plan; }

extern "C" uint32_t ciera_plan_n_units(const ciera_plan* p) { return p ? p->n_units : 0; }
extern "C" uint32_t ciera_plan_n_tiles(const ciera_plan* p) { return p ? (uint32_t)p->tiles.size() : 0; }
extern "C" uint32_t ciera_plan_tile_values(const ciera_plan*) { return kTileValues; }
extern "C" uint64_t ciera_plan_total_values(const ciera_plan* p) { return p ? p->total_values : 0; }

extern "C" size_t ciera_plan_device_bytes(const ciera_plan* p) { return p ? p->image.size() : 0; }
extern "C" const void* ciera_plan_host_image(const ciera_plan* p) { return p ? p->image.data() : nullptr; }

extern "C" size_t ciera_plan_workspace_bytes(const ciera_plan* p) {
    if (!p) return 0;
    return workspace_total_bytes(p->tiles.size());  // status words, counters, per-tile counts: see ciera_internal.cuh
}

extern "C" int ciera_workspace_init(const ciera_plan* p, void* workspace_dev, void* stream) {
    if (!p || !workspace_dev) return CIERA_ERR_INVALID_ARG;
    if ((uintptr_t)workspace_dev & 15u) return CIERA_ERR_MISALIGNED;
    cudaError_t e = cudaMemsetAsync(workspace_dev, 0, workspace_total_bytes(p->tiles.size()), (cudaStream_t)stream);
    if (e != cudaSuccess) return record_cuda_error(e);
    return CIERA_OK;
}

extern "C" size_t ciera_plan_hash_cache_bytes(const ciera_plan* p) { return p ? (size_t)p->total_blocks * 16 : 0; }
extern "C" size_t ciera_plan_unit_hash_offset(const ciera_plan* p, uint32_t unit) {
    return (p && unit < p->n_units) ? (size_t)p->hash_base[unit] * 16 : 0;
}
extern "C" size_t ciera_plan_hashed_workspace_bytes(const ciera_plan* p) {
    return ciera_plan_workspace_bytes(p);  // the same kernel, the same scratch
}

extern "C" int ciera_plan_bind(ciera_plan* p, void* plan_dev, size_t plan_dev_bytes, void* stream) {
    if (!p || !plan_dev) return CIERA_ERR_INVALID_ARG;
    if ((uintptr_t)plan_dev & 15u) return CIERA_ERR_MISALIGNED;
    const size_t need = p->image.size();
    if (plan_dev_bytes < need) return CIERA_ERR_CAPACITY;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(plan_dev, p->image.data(), need, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return record_cuda_error(e);
    p->tiles_dev = (const TileDesc*)plan_dev;
    const ImageLayout L = image_layout(p);
    const uint8_t* base = (const uint8_t*)plan_dev;
    p->long_units_dev = (const uint32_t*)(base + L.long_off);
    p->seq_first_dev = (const uint32_t*)(base + L.seq_off);
    p->hash_base_dev = (const unsigned long long*)(base + L.hash_off);
    p->unit_first_dev = (const uint32_t*)(base + L.first_off);
    p->seg_base_dev = (const unsigned long long*)(base + L.seg_off);
    p->units_dev = (const ciera_unit*)(base + L.units_off);
    p->ent_long_units_dev = (const uint32_t*)(base + L.elong_off);
    p->ent_chunks_dev = (const uint4*)(base + L.echunk_off);
    p->tile_hash_dev = (const unsigned long long*)(base + L.thash_off);
    p->seq_runs_dev = (const uint2*)(base + L.runs_off);
    return CIERA_OK;
}

// ---------------------------------------------------------------------------------- gain rule

static double comm_seconds(const ciera_gain_in* in, double bytes) {
    if (in->n_points < 2 || !in->table_bytes || !in->table_secs)
        return in->alpha + (double)(in->world_size - 1) * bytes / in->beta;
    int i = 0;
    while (i < in->n_points - 2 && bytes > in->table_bytes[i + 1]) ++i;
    double x0 = in->table_bytes[i], x1 = in->table_bytes[i + 1];
    double y0 = in->table_secs[i], y1 = in->table_secs[i + 1];
    return y0 + (bytes - x0) * (y1 - y0) / (x1 - x0);
}

static int gain_of(const ciera_gain_in* in, double* g_out);

extern "C" int ciera_should_compress(const ciera_gain_in* in, double* gain_seconds_out, int* decision_out) {
    double g = 0.0;
    const int rc = gain_of(in, &g);
    if (rc) return rc;
    if (gain_seconds_out) *gain_seconds_out = g;
    if (decision_out) *decision_out = g > 0.0 ? 1 : 0;
    return CIERA_OK;
}

static int gain_of(const ciera_gain_in* in, double* g_out) {
    if (!in || !valid_dtype(in->dtype) || in->block == 0) return CIERA_ERR_INVALID_ARG;
    if (!(in->q >= 0.0 && in->q <= 1.0)) return CIERA_ERR_INVALID_ARG;
    if (in->n_points >= 2 && in->table_bytes && in->table_secs) {
        for (int i = 0; i + 1 < in->n_points; ++i)
            if (!(in->table_bytes[i + 1] > in->table_bytes[i])) return CIERA_ERR_INVALID_ARG;
    } else if (!(in->beta > 0.0) || in->world_size < 1) {
        return CIERA_ERR_INVALID_ARG;
    }
    const double n = (double)in->n_values;
    const double s_full = n * value_bytes_of(in->dtype);
    const double s_exp = n * exp_bits_of(in->dtype) / 8.0;  // exponent bits per value / 8
    const double s_sm = s_full - s_exp;
    const uint64_t blocks = (in->n_values + in->block - 1) / in->block;
    const double s_bm = (double)((blocks + 7) / 8);
    const double sent = s_sm + s_bm + in->q * s_exp;
    const double sender = in->overlapped ? 0.0 : in->t_hash + in->t_cmp;
    *g_out = comm_seconds(in, s_full) - (comm_seconds(in, sent) + sender + in->t_decmp);
    return CIERA_OK;
}

// ---------------------------------------------------------------------------------- selection

extern "C" int ciera_select_shards(const ciera_gain_in* shards, uint32_t n_shards, uint64_t cache_budget_bytes,
                                   int with_sender_cache, uint32_t* ranking_out, uint8_t* selected_out,
                                   double* gains_out, uint64_t* footprints_out, uint64_t* used_bytes_out) {
    if ((!shards && n_shards) || (!selected_out && n_shards)) return CIERA_ERR_INVALID_ARG;
    std::vector<double> g(n_shards);
    std::vector<uint64_t> m(n_shards);
    for (uint32_t i = 0; i < n_shards; ++i) {
        const int rc = gain_of(&shards[i], &g[i]);
        if (rc) return rc;
        if (shards[i].world_size < 1) return CIERA_ERR_INVALID_ARG;
        // M_i = (W - 1) S_e^i per GPU, S_e^i = one exponent byte per value (+ S_e^i for this
        // library's sender-side exponent cache when asked for)
        m[i] = (uint64_t)(shards[i].world_size - 1 + (with_sender_cache ? 1 : 0)) * shards[i].n_values;
    }
    // positive gains in descending order of g_i / M_i (ties: original order), then the rest
    std::vector<uint32_t> cand, rest;
    for (uint32_t i = 0; i < n_shards; ++i) ((g[i] > 0.0 && m[i] > 0) ? cand : rest).push_back(i);
    std::stable_sort(cand.begin(), cand.end(),
                     [&](uint32_t a, uint32_t b) { return g[a] / (double)m[a] > g[b] / (double)m[b]; });
    for (uint32_t i = 0; i < n_shards; ++i) selected_out[i] = 0;
    uint64_t used = 0;
    for (uint32_t i : cand) {  // until the budget is exhausted: stop at the first shard that does not fit
        if (m[i] > cache_budget_bytes - used) break;
        selected_out[i] = 1;
        used += m[i];
    }
    if (ranking_out) {
        uint32_t k = 0;
        for (uint32_t i : cand) ranking_out[k++] = i;
        for (uint32_t i : rest) ranking_out[k++] = i;
    }
    for (uint32_t i = 0; i < n_shards; ++i) {
        if (gains_out) gains_out[i] = g[i];
        if (footprints_out) footprints_out[i] = m[i];
    }
    if (used_bytes_out) *used_bytes_out = used;
    return CIERA_OK;
}

// ---------------------------------------------------------------------------------- diagnostics

extern "C" int ciera_last_cuda_error(void) { return g_last_cuda_error; }
extern "C" uint64_t ciera_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" const char* ciera_status_string(int s) {
    switch (s) {
        case CIERA_OK: return "ok";
        case CIERA_ERR_INVALID_ARG: return "invalid argument";
        case CIERA_ERR_UNSUPPORTED: return "unsupported block size or unit size";
        case CIERA_ERR_MISALIGNED: return "offset or pointer not 16-byte aligned";
        case CIERA_ERR_CAPACITY: return "buffer or message slot too small";
        case CIERA_ERR_CUDA: return "CUDA runtime error";
        case CIERA_ERR_TIMEOUT: return "device wait ran out";
        case CIERA_ERR_CORRUPT: return "message length contradicts its bitmap";
        case CIERA_ERR_NOT_BOUND: return "plan not bound to device memory";
        case CIERA_ERR_TOO_LARGE: return "plan has more tiles than the built-in scratch of ciera_encode_noalloc holds";
        default: return "unknown status";
    }
}
