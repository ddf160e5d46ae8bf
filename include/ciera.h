/*
 * ciera.h -- C ABI of the B200 (sm_100a) exponent-reuse codec.
 *
 * The library implements the data-parallel hot path of CIERA's "Exponent Reuse based
 * Compression" (paper Section 3.1, Algorithm 1) and the gain rule of "Benefit-driven
 * Selective Compression" (Section 3.2):
 *
 *   sender    split every weight into exponent and sign-plus-mantissa, compare the exponents
 *             with a cached copy block by block, emit (bitmap, sign-plus-mantissa of all
 *             values, exponents of changed blocks), refresh the cache for changed blocks;
 *   receiver  patch its exponent cache with the changed blocks, merge cache and
 *             sign-plus-mantissa back into bit-identical weights.
 *
 * Conventions
 *   - Every function returns a ciera_status (0 = CIERA_OK, negative = error).  Nothing throws,
 *     nothing is printed, and no codec state lives in the library: caches, messages and scratch
 *     are the caller's buffers.  What the library does keep per process: the launch counter, the
 *     thread's last CUDA error, and per device the grid sizes it has worked out for its kernels.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host pointers.
 *     The library never allocates device memory: the caller owns every device buffer and
 *     passes scratch space explicitly.  The only host allocation is the plan object.  (One
 *     exception, stated where it is declared: ciera_encode_noalloc works in a fixed device array
 *     that is part of the library image, for callers that cannot supply scratch.)
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Device work is
 *     enqueued on it and the call returns without waiting, unless stated otherwise.
 *     The sender, transport, receiver and entropy calls read every size they need on the device
 *     and leave their scratch as they found it, so a step may be captured in a CUDA graph and
 *     replayed; call each entry point once outside a capture first (its first call on a device
 *     queries occupancy and sets kernel attributes).  The host-side launch counter does not see
 *     replays.
 *   - Errors found on the device (a wait that ran out, a message whose length contradicts its
 *     bitmap) are written to the caller's `status_dev` word: 0 = none, otherwise the first
 *     ciera_status that was raised.  The word is only ever written on error; clear it yourself.
 *   - A *unit* is one shard of one tensor: N consecutive values.  Units are independent; one call
 *     processes a whole table of them ("batched launch over simulated shards").
 *
 * Wire format of one unit's message (b bits per value, m = b - 8 sign-plus-mantissa bits,
 * block size B, nb = ceil(N/B) blocks; Section 3.2 for the sizes, Algorithm 1 for the order
 * bitmap, mant, payload):
 *
 *   [ bitmap : ceil(nb/8) bytes, block k -> byte k>>3 bit k&7, unused high bits 0 ]
 *   [ zero pad to a multiple of 16 ]
 *   [ sm     : N*m/8 bytes; bf16: byte j = sign<<7 | mantissa(7);
 *              fp32: bytes 3j..3j+2 = (sign<<23 | mantissa(23)) little-endian ]
 *   [ zero pad to a multiple of 16 ]
 *   [ payload: for every changed block in ascending k, its exponent bytes (B of them, fewer
 *              for a short last block) ]
 *
 * No header travels: the payload length follows from the bitmap.  The paper's byte count
 * S_{s+m} + S_bm + (changed exponent bytes) is ciera_message_bytes(); the length that has to
 * be moved (it includes the two pads, at most 30 bytes) is what ciera_encode reports.
 * Bytes of a slot past the reported length are unspecified.
 */
#ifndef CIERA_H
#define CIERA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CIERA_API __attribute__((visibility("default")))
#else
#define CIERA_API
#endif

typedef enum ciera_status {
    CIERA_OK = 0,
    CIERA_ERR_INVALID_ARG = -1, /* null pointer, zero block, bad enum, inconsistent sizes      */
    CIERA_ERR_UNSUPPORTED = -2, /* block size outside the supported set                         */
    CIERA_ERR_MISALIGNED = -3,  /* an offset or base pointer is not a multiple of 16 bytes      */
    CIERA_ERR_CAPACITY = -4,    /* a message slot, plan image or scratch buffer is too small    */
    CIERA_ERR_CUDA = -5,        /* a CUDA runtime call failed (see ciera_last_cuda_error)       */
    CIERA_ERR_TIMEOUT = -6,     /* device: a bounded wait on another tile ran out               */
    CIERA_ERR_CORRUPT = -7,     /* device: message length disagrees with its bitmap             */
    CIERA_ERR_NOT_BOUND = -8,   /* the plan has no device image yet (ciera_plan_bind)           */
    CIERA_ERR_TOO_LARGE = -9    /* more tiles than the built-in scratch of ciera_encode_noalloc */
} ciera_status;

typedef enum ciera_dtype {
    CIERA_BF16 = 0, /* b = 16: 1 sign, 8 exponent, 7 mantissa bits  -> m = 8  */
    CIERA_FP32 = 1, /* b = 32: 1 sign, 8 exponent, 23 mantissa bits -> m = 24 */
    CIERA_FP16 = 2  /* b = 16: 1 sign, 5 exponent, 10 mantissa bits -> m = 11 (IEEE binary16).  On the
                       wire its exponents take 5 bits and its sign-plus-mantissa 11 bits each, packed
                       without gaps (value j of a section at bits [j*w, (j+1)*w), bit i of a section =
                       byte i >> 3, bit i & 7); every changed block of the payload starts on a byte
                       boundary (a block of 1, 2, 4, 8, 16 ... values takes 1, 2, 3, 5, 10 ... bytes);
                       the caches still hold one byte per value.  Every block size; the hashed
                       sender takes it too (blocks of 16 values and more, as for the other
                       precisions), and so does the entropy stage, which codes the 5-bit exponents
                       as symbols of their own (it undoes the packing first; 32 table entries
                       travel instead of 256). */
} ciera_dtype;

/* One unit = one shard of one tensor.  All offsets are in BYTES from the base pointer of the
 * respective buffer and must be multiples of 16. */
typedef struct ciera_unit {
    uint64_t n_values;     /* N; may be 0, may be smaller than the block size                   */
    uint64_t weights_off;  /* into the weights buffer (encode: input, decode: output)           */
    uint64_t cache_off;    /* into the exponent cache (1 byte per value)                        */
    uint64_t msg_off;      /* into the message buffer: start of this unit's slot                */
    uint64_t msg_capacity; /* size of the slot, >= ciera_message_capacity(N, dtype, block)      */
} ciera_unit;

/* ---- sizes (host, pure functions; Section 3.2) ------------------------------------------- */

/* Smallest and largest supported block size B (a power of two in this range).  B = 1 is change
 * detection per value: the bitmap has one bit per value and the payload holds exactly the exponents
 * that changed (Section 2.3: a block stays reusable with probability (1-c)^B, so finer blocks are
 * reused more often, at the price of a longer bitmap). */
#define CIERA_MIN_BLOCK 1u
#define CIERA_MAX_BLOCK 4096u

/* Slot size that always suffices: every block changed (payload = N exponent bytes). */
CIERA_API size_t ciera_message_capacity(uint64_t n_values, int dtype, uint32_t block);
/* Offset of the sign-plus-mantissa section / of the payload section inside a slot. */
CIERA_API size_t ciera_sm_offset(uint64_t n_values, uint32_t block);
CIERA_API size_t ciera_payload_offset(uint64_t n_values, int dtype, uint32_t block);
/* The paper's transmitted bytes S_{s+m} + S_bm + payload_bytes (no pads). */
CIERA_API size_t ciera_message_bytes(uint64_t n_values, int dtype, uint32_t block, uint64_t payload_bytes);

/* ---- plan: the tile table of a unit table -------------------------------------------------- */

/* A plan splits every unit into tiles of ciera_plan_tile_values() consecutive values (one tile
 * is the work of one thread block) and holds the device-side table that the kernels read.  It
 * is immutable after ciera_plan_bind and may be shared by any number of calls and streams. */
typedef struct ciera_plan ciera_plan;

/* Host only.  Validates the units (alignment, capacity, block size) and builds the table.
 * `units_host` is copied.  Destroy with ciera_plan_destroy. */
CIERA_API int ciera_plan_create(const ciera_unit* units_host, uint32_t n_units, int dtype, uint32_t block,
                      ciera_plan** plan_out);
CIERA_API void ciera_plan_destroy(ciera_plan* plan);

CIERA_API uint32_t ciera_plan_n_units(const ciera_plan* plan);
CIERA_API uint32_t ciera_plan_n_tiles(const ciera_plan* plan);
CIERA_API uint32_t ciera_plan_tile_values(const ciera_plan* plan);
CIERA_API uint64_t ciera_plan_total_values(const ciera_plan* plan);
/* Bytes of device memory the table needs (>= 16), and the host image that has to be there. */
CIERA_API size_t ciera_plan_device_bytes(const ciera_plan* plan);
CIERA_API const void* ciera_plan_host_image(const ciera_plan* plan);
/* Bytes of scratch ("workspace") that ciera_encode, ciera_transport and ciera_decode work in: 12 bytes per
 * tile (a look-back status word for the sender, a count for the receiver) and a few counters. */
CIERA_API size_t ciera_plan_workspace_bytes(const ciera_plan* plan);
/* Zero-fills a workspace of ciera_plan_workspace_bytes(plan) bytes (16-byte aligned) on `stream`.  Every
 * call that takes a workspace (ciera_encode, ciera_encode_hashed, ciera_transport, ciera_decode,
 * ciera_roundtrip_host) expects its counters in it all zero when it starts and leaves them all zero when it
 * has finished, so that no launch is spent on clearing them before every call: initialise a workspace once
 * after allocating it, and again after a call whose device status word came back with an error (a kernel
 * that gave up leaves the workspace in an unspecified state).  A plain cudaMemset of the whole workspace
 * does the same. */
CIERA_API int ciera_workspace_init(const ciera_plan* plan, void* workspace_dev, void* stream);

/* Copies the table into caller-owned device memory `plan_dev` (>= ciera_plan_device_bytes,
 * 16-byte aligned) on `stream`, waits for the copy, and remembers the pointer.  The memory must
 * stay valid and unmodified for as long as the plan is used. */
CIERA_API int ciera_plan_bind(ciera_plan* plan, void* plan_dev, size_t plan_dev_bytes, void* stream);

/* ---- caches (Algorithm 1: persistent sender / receiver state) ------------------------------ */

/* cache := exponents of `weights_dev`, or all zero if weights_dev == NULL.  The paper switches
 * its method on once warm-up is over and does not say what the caches hold at that moment;
 * initialising both sides from the same weights (as if they had been sent uncompressed), or
 * both to zero, keeps them in agreement. */
CIERA_API int ciera_cache_init(const ciera_plan* plan, void* cache_dev, const void* weights_dev, void* stream);
/* cache := exponents of `weights_dev`, unconditionally (e.g. after a checkpoint restore). */
CIERA_API int ciera_cache_update(const ciera_plan* plan, void* cache_dev, const void* weights_dev, void* stream);

/* ---- sender: Algorithm 1, sender part; Section 3.1 ----------------------------------------- */

/*
 * For every unit: split, block-wise change detection against `sender_cache_dev`, write the
 * message into the unit's slot of `messages_dev`, refresh the cache for changed blocks.
 *   weights_dev         in   values of the plan's dtype at units[].weights_off
 *   sender_cache_dev    i/o  1 byte per value at units[].cache_off
 *   messages_dev        out  slots at units[].msg_off
 *   wire_bytes_dev      out  [n_units] bytes that have to travel (payload offset + payload bytes;
 *                            0 for an empty unit)
 *   changed_blocks_dev  out  [n_units] number of set bitmap bits
 *   workspace_dev       i/o  scratch of ciera_plan_workspace_bytes(), 16-byte aligned (look-back status
 *                            words, the counter that runs of tiles are handed out from); all zero on
 *                            entry -- see ciera_workspace_init -- and handed back all zero; must not
 *                            be shared by calls that can overlap on the GPU
 *   status_dev          i/o  device error word (may be NULL)
 * One kernel launch for the whole table, nothing else (a table that holds empty units: two small
 * clearing operations in front of it, which write those units' zero lengths and counts).
 */
CIERA_API int ciera_encode(const ciera_plan* plan, const void* weights_dev, void* sender_cache_dev, void* messages_dev,
                 uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev, void* workspace_dev,
                 int32_t* status_dev, void* stream);

/* ---- sender, for callers that cannot supply scratch ---------------------------------------- */

/* Largest plan ciera_encode_noalloc accepts: 65 536 tiles (ciera_plan_n_tiles), i.e. at most
 * 536 870 912 values per call.  The library keeps 8 bytes per tile (+ 16) = 512 KiB of device memory
 * for it on every GPU that loads the library, from load until the process exits. */
#define CIERA_NOALLOC_MAX_TILES 65536u

/*
 * (This entry point has no counterpart in the paper; it is a convenience of this library.)
 *
 * Same work and same outputs as ciera_encode, but without the `workspace_dev` argument: the
 * look-back scratch is a fixed array inside the library.  It is meant for callers that can pass the
 * buffers they already own but cannot obtain a fresh device allocation when they call -- a training
 * runtime whose memory pool already holds the whole GPU, a parameter-gather hook that must not
 * stall the device (allocating does), a plug-in that was handed pointers but no allocator.  The
 * call itself allocates nothing, on the host or on the device.
 *
 *   - Plans with more than CIERA_NOALLOC_MAX_TILES tiles are refused with CIERA_ERR_TOO_LARGE before
 *     any device work is enqueued; split the unit table, or use ciera_encode with your own scratch.
 *   - The first call on each device looks up the array's device address (a CUDA runtime query made
 *     with that device current).  Make that first call outside of any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the last call left in it; every
 *     call therefore clears the part it uses, on `stream`, before its kernel.  Two calls that can
 *     run on the GPU at the same time (different streams, no ordering between them) race on the
 *     array and produce garbage: order them, or give all but one of them ciera_encode with scratch
 *     of its own.
 */
CIERA_API int ciera_encode_noalloc(const ciera_plan* plan, const void* weights_dev, void* sender_cache_dev,
                         void* messages_dev, uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev,
                         int32_t* status_dev, void* stream);

/* ---- sender with hash-based change detection (Section 3.1; Algorithm 1, sender, as printed) ---
 *
 * Instead of the previous exponents the sender keeps HashCache: one 128-bit hash per block, built
 * from two independent 64-bit SplitMix64 hashes of the block's exponents.  A block travels iff its
 * hash differs from the cached one; the cached hash is then replaced.  The message is the same as
 * ciera_encode's (a collision -- both 64-bit halves at once, which behave like independent random
 * functions of the block but are not a cryptographic hash -- would leave a changed block unsent).
 * The construction (the paper prints none): with mix() the SplitMix64 output function, a block of L
 * exponent bytes read as little-endian 64-bit words x_j (the last one zero-padded),
 * H_i = mix(L + sum_j mix(s_i + (j + 1) * g_i + x_j)) mod 2^64, Hash128 = (H_1, H_2) with
 * s_1 = 0, g_1 = 0x9E3779B97F4A7C15 (the generator's increment), s_2 = 0x6A09E667F3BCC908,
 * g_2 = 0xD1342543DE82EF95; stored as two little-endian 64-bit words per block.
 * Blocks of 16 values and more only (CIERA_ERR_UNSUPPORTED otherwise).  The hash is taken
 * over the exponents as the caches hold them, one byte each, for every precision. */

/* Bytes of a HashCache for the whole plan (16 per block; units in table order), the offset of a
 * unit's first block in it, and the scratch ciera_encode_hashed needs (= ciera_plan_workspace_bytes). */
CIERA_API size_t ciera_plan_hash_cache_bytes(const ciera_plan* plan);
CIERA_API size_t ciera_plan_unit_hash_offset(const ciera_plan* plan, uint32_t unit);
CIERA_API size_t ciera_plan_hashed_workspace_bytes(const ciera_plan* plan);

/* HashCache := Hash128 of every block of exponents(weights); of all-zero exponents when
 * weights_dev is NULL (the counterpart of a zero-initialised exponent cache).  Device pointers,
 * 16-byte aligned.  Asynchronous on `stream`. */
CIERA_API int ciera_hash_cache_init(const ciera_plan* plan, void* hash_cache_dev, const void* weights_dev, void* stream);

/* Sender step with HashCache.  Arguments, launch (one persistent kernel) and error behaviour as
 * for ciera_encode, with hash_cache_dev (in/out, ciera_plan_hash_cache_bytes) in place of the
 * exponent cache and a scratch of ciera_plan_hashed_workspace_bytes (all zero on entry and on return,
 * as for ciera_encode). */
CIERA_API int ciera_encode_hashed(const ciera_plan* plan, const void* weights_dev, void* hash_cache_dev,
                                  void* messages_dev, uint64_t* wire_bytes_dev, uint32_t* changed_blocks_dev,
                                  void* workspace_dev, int32_t* status_dev, void* stream);

/* ---- transport stand-in: Send / Recv of Algorithm 1 on one GPU ----------------------------- */

/* Copies, for every unit, the first wire_bytes_dev[u] bytes of its slot from `src_messages_dev`
 * to the same slot of `dst_messages_dev` (one kernel; the lengths are read on the device).  This
 * stands where the Allgather of the messages would be.  `workspace_dev`: scratch of
 * ciera_plan_workspace_bytes() (holds the counter tiles are handed out from: zero on entry -- see
 * ciera_workspace_init -- and handed back at zero; not to be shared by calls that can overlap on the GPU).  `status_dev`: device int32 or NULL; the
 * kernel's waits on its own copies are bounded and raise CIERA_ERR_TIMEOUT there. */
CIERA_API int ciera_transport(const ciera_plan* plan, const void* src_messages_dev, void* dst_messages_dev,
                    const uint64_t* wire_bytes_dev, void* workspace_dev, int32_t* status_dev, void* stream);

/* ---- receiver: Algorithm 1, receiver part; Section 3.1 ------------------------------------- */

/*
 * For every unit: read the bitmap, overwrite the cached exponents of changed blocks with the
 * payload, merge cache and sign-plus-mantissa into `weights_out_dev`.
 *   messages_dev        in   slots at units[].msg_off
 *   receiver_cache_dev  i/o  1 byte per value at units[].cache_off
 *   weights_out_dev     out  reconstructed values at units[].weights_off
 *   wire_bytes_dev      in   optional (may be NULL): lengths as reported by the sender; a unit
 *                            whose bitmap implies a different length raises CIERA_ERR_CORRUPT in
 *                            status_dev (its output is then unspecified)
 *   workspace_dev       scratch of ciera_plan_workspace_bytes(), 16-byte aligned: the counter tiles
 *                            are handed out from (zero on entry -- see ciera_workspace_init -- and handed
 *                            back at zero) and, when some unit has
 *                            more than 4096 blocks, the per-tile counts of a small prefix kernel that
 *                            runs first; the sender's part of the workspace is left alone.  Must not be
 *                            shared by calls that can overlap on the GPU.
 */
CIERA_API int ciera_decode(const ciera_plan* plan, const void* messages_dev, void* receiver_cache_dev,
                 void* weights_out_dev, const uint64_t* wire_bytes_dev, void* workspace_dev, int32_t* status_dev,
                 void* stream);

/* ---- whole step with host buffers ---------------------------------------------------------- */

/* Device buffers one ciera_roundtrip_host call works in; all caller-owned, sized as for the
 * separate calls above (weights_dev / weights_out_dev: weights_bytes each; workspace_dev initialised
 * with ciera_workspace_init as for ciera_encode). */
typedef struct ciera_device_buffers {
    void* weights_dev;
    void* sender_cache_dev;
    void* msg_send_dev;
    void* msg_recv_dev;
    void* receiver_cache_dev;
    void* weights_out_dev;
    uint64_t* wire_bytes_dev;
    uint32_t* changed_blocks_dev;
    void* workspace_dev;
    int32_t* status_dev;
} ciera_device_buffers;

/* One sender + receiver step of Algorithm 1 on weights that live in HOST memory:
 * copy `weights_host` (weights_bytes, ideally pinned) to the device, ciera_encode,
 * ciera_transport, ciera_decode, copy the reconstructed weights to `weights_out_host` and the
 * per-unit wire lengths to `wire_bytes_host` ([n_units], may be NULL).  Everything is enqueued on
 * `stream`; the host buffers must stay valid until the stream has drained. */
CIERA_API int ciera_roundtrip_host(const ciera_plan* plan, const void* weights_host, size_t weights_bytes,
                         void* weights_out_host, uint64_t* wire_bytes_host, const ciera_device_buffers* bufs,
                         void* stream);

/* ---- entropy stage (Section 3.1; Algorithm 1: ANSEncode on the sender, ANSDecode on the receiver) ---
 *
 * Between ciera_encode (or ciera_encode_hashed) and the transport, ciera_entropy_encode replaces the
 * payload of every message -- the exponents of the changed blocks -- by its rANS-coded form if that
 * is strictly shorter, and lowers the unit's wire_bytes accordingly; bitmap and sign-plus-mantissa
 * stay as they are.  Between the transport and ciera_decode, ciera_entropy_decode restores the raw
 * payload in place (the receiver knows the raw length from the bitmap: a message of exactly that
 * length carries the raw form) and sets wire_bytes back to the raw length, so that ciera_decode
 * sees what the sender step had written.  The paper names a vendor library whose format is not
 * public; coder and layout are this library's own: static model per unit (a symbol = an exponent:
 * 256 symbols for bf16 and fp32, 32 for fp16, whose 5-bit packing is undone before and redone after
 * the coder; probabilities in 1/4096), 32-bit rANS states with 16-bit words, segments of 4096
 * symbols coded by 32 interleaved coders each; coded section = [256 or 32 x u16 frequencies][per
 * segment a u32 word count][segments: 32 x u32 final states, the words, 2 zero bytes if their
 * number is odd].
 *   messages_dev    device, in/out
 *   wire_bytes_dev  device, n_units x uint64, in/out
 *   scratch_dev     device, ciera_plan_entropy_scratch_bytes(plan) bytes, 16-byte aligned; contents
 *                   need not be initialised
 *   status_dev      device int32 or NULL: CIERA_ERR_CORRUPT if a coded section is inconsistent
 *                   (that unit's payload is then left as received)
 * One launch each, one thread block per unit; nothing waits inside the kernels. */
CIERA_API size_t ciera_plan_entropy_scratch_bytes(const ciera_plan* plan);
CIERA_API int ciera_entropy_encode(const ciera_plan* plan, void* messages_dev, uint64_t* wire_bytes_dev, void* scratch_dev,
                                   void* stream);
CIERA_API int ciera_entropy_decode(const ciera_plan* plan, void* messages_dev, uint64_t* wire_bytes_dev, void* scratch_dev,
                                   int32_t* status_dev, void* stream);

/* ---- selective compression: the gain rule of Section 3.2 (host only) ----------------------- */

typedef struct ciera_gain_in {
    uint64_t n_values;    /* N^i                                                               */
    int32_t dtype;        /* ciera_dtype                                                        */
    uint32_t block;       /* B (any positive value; only sizes are computed)                    */
    double q;             /* block change rate q_i in [0, 1] (measured offline / by a previous encode) */
    int32_t world_size;   /* W, used by the alpha-beta model only                               */
    int32_t overlapped;   /* non-zero: T_hash = T_cmp = 0 on the critical path (pipelining)     */
    double alpha;         /* Comm(S) = alpha + (W-1) * S / beta when n_points < 2               */
    double beta;          /* bytes per second                                                   */
    const double* table_bytes; /* optional measured Comm(): n_points ascending payload sizes... */
    const double* table_secs;  /* ...and their latencies; linear interpolation, the first/last
                                  segment is extended outside the table                         */
    int32_t n_points;
    double t_hash;        /* seconds: change detection of the shard                             */
    double t_cmp;         /* seconds: sender-side packing                                       */
    double t_decmp;       /* seconds: receiver-side patch + merge                               */
} ciera_gain_in;

/* g = Comm(S) - ( Comm(S_{s+m} + S_bm + q S_e) + T_hash + T_cmp + T_decmp ), and the decision
 * "compress iff g > 0".  Either output pointer may be NULL. */
CIERA_API int ciera_should_compress(const ciera_gain_in* in, double* gain_seconds_out, int* decision_out);

/* Shard selection under a cache budget (Section 3.2, last paragraph): shard i costs
 * M_i = (W - 1) * S_e^i bytes of exponent cache per GPU (S_e^i = one byte per value); shards with
 * positive gain are ranked in descending order of g_i / M_i and selected down the ranking until the
 * first one that no longer fits into cache_budget_bytes (ties keep the input order; shards without
 * values are never selected).  with_sender_cache != 0 counts W * S_e^i instead, i.e. also the
 * sender-side exponent cache this library compares against.
 *   shards          host, n_shards entries (q_i, sizes, Comm() model and kernel times per shard)
 *   ranking_out     host, n_shards indices: the ranked positive-gain shards, then the others in
 *                   input order; may be NULL
 *   selected_out    host, n_shards flags (1 = compress this shard)
 *   gains_out, footprints_out   host, n_shards values g_i (seconds) and M_i (bytes); may be NULL
 *   used_bytes_out  host, sum of M_i over the selected shards; may be NULL
 * Returns CIERA_ERR_INVALID_ARG for a shard that ciera_should_compress would reject. */
CIERA_API int ciera_select_shards(const ciera_gain_in* shards, uint32_t n_shards, uint64_t cache_budget_bytes,
                                  int with_sender_cache, uint32_t* ranking_out, uint8_t* selected_out,
                                  double* gains_out, uint64_t* footprints_out, uint64_t* used_bytes_out);

/* ---- diagnostics ---------------------------------------------------------------------------- */

/* Self-test of the device-side failure path (no counterpart in the paper: Algorithm 1 has no failure
 * handling).  Every wait inside the persistent kernels -- on a look-back status word of another tile,
 * on a shared-memory barrier that a bulk copy or another warp completes -- is bounded: when the bound
 * runs out the waiting role raises CIERA_ERR_TIMEOUT in the caller's status word, the thread block
 * stops, and the kernel returns, so the context stays usable.  This call runs one tiny kernel (one
 * thread block) that performs both kinds of wait with a limit of `max_polls` polls (1 .. 4096; a
 * barrier poll suspends for at most 20 microseconds) on a word and a barrier that nothing completes.
 *   scratch_dev  device, 8 bytes, 8-byte aligned: the status word that is polled (cleared by the call)
 *   status_dev   device int32: receives CIERA_ERR_TIMEOUT if it was 0
 *   report_dev   device, 4 x int32 (cleared by the call): [0] = 1 the status-word wait gave up,
 *                [1] = 1 the barrier wait gave up, [2] = the block's abort flag, [3] = max_polls
 * Asynchronous on `stream`. */
CIERA_API int ciera_selftest_bounded_waits(uint32_t max_polls, void* scratch_dev, int32_t* status_dev,
                                           int32_t* report_dev, void* stream);

/* cudaError_t of the last failing runtime call made by the calling thread inside this library. */
CIERA_API int ciera_last_cuda_error(void);
/* Number of kernels this library has launched from the calling process (for launch accounting). */
CIERA_API uint64_t ciera_kernel_launch_count(void);
CIERA_API const char* ciera_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* CIERA_H */
