/*
 * CIERA exponent-reuse codec -- plain CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the hot path computes.  Only the test-suite, the smoke check and the
 * benchmark's cpu_baseline / reference legs may call it.  It shares no code, header,
 * table or constant with the CUDA library and neither side includes the other.
 *
 * What it states (the definitions are the paper's, the wording and structure are this file's):
 *   - Section 3.1: a value is cut into its exponent field and the rest (sign and mantissa).
 *     Blocks of B consecutive values are compared with what was last sent: a block counts as
 *     changed when any of its exponents differs.  A message holds one bit per block, the
 *     sign-and-mantissa part of every value, and the exponent fields of the changed blocks only.
 *   - Algorithm 1: the sender marks changed blocks, remembers their new exponents, and strings the
 *     exponents of the marked blocks together in ascending block order; the receiver goes through
 *     the marks in the same order, takes one block of exponents off the front of the payload for
 *     each mark to overwrite its cached copy, and rebuilds every value from cached exponent plus
 *     received sign-and-mantissa.
 *   - Section 3.2: the sizes S, S_e, S_{s+m}, S_b, S_bm, the expected message size, and the gain
 *     of compressing a shard (ora_gain).
 *
 * Readings taken where the paper is silent (each is listed in the design notes):
 *   - Change detection is the exact predicate the paper's 128-bit block hash
 *     approximates: compare each exponent with a sender-side cached exponent.
 *   - The changed exponents travel raw (the entropy-coding stage is left out); this
 *     is also what the paper's expected-payload formula charges (q * S_e).
 *   - sm = sign << (m-1) | mantissa, m = b - 8 bits; fp32 sm is 3 little-endian
 *     bytes per value; bitmap bit k lives in byte k>>3, bit k&7.
 *   - A short last block carries exactly its own values; N = 0 gives an empty message.
 *   - Wire layout of one unit: [bitmap][pad to 16][sm][pad to 16][payload]; pad bytes
 *     and the unused high bits of the last bitmap byte are zero.
 *
 * Pins: tests/test_oracle_*.py (IEEE field definition through frexp, exhaustive
 * bf16 x cache sweep, hand-worked fixtures, byte formula, closed forms (1-c)^B,
 * special cases, hand-computed gains).  The entropy stage for the changed exponents has an oracle of
 * its own (rans_oracle.c).  The hash-based sender (ora_encode_hashed) is pinned as a change detector (published
 * SplitMix64 streams, equality with the exact-comparison sender, certain detection of single-word
 * changes); the 128-bit hash VALUES follow a construction the paper does not print, so for them:
 * parity unpinned.
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORA_BF16 = 0, ORA_FP32 = 1, ORA_FP16 = 2 };

/* b = bits per value, e = exponent bits, m = b - e = sign+mantissa bits (Section 3.1: a value is
 * sign, exponent and mantissa bits).  bf16: 16 = 1 + 8 + 7; fp32: 32 = 1 + 8 + 23; fp16 (IEEE
 * binary16): 16 = 1 + 5 + 10.  Caches hold one byte per value for every precision; on the wire an
 * exponent takes e bits and a sign-plus-mantissa m bits, packed without gaps (reading: value j of a
 * section occupies bits [j*w, (j+1)*w) of the section's bytes, bit i of a section = byte i >> 3,
 * bit i & 7 -- for w = 8 and w = 24 this is one byte and three little-endian bytes per value). */
static int ora_b(int dtype) { return dtype == ORA_FP32 ? 32 : 16; }
static int ora_e(int dtype) { return dtype == ORA_FP16 ? 5 : 8; }
static int ora_m(int dtype) { return ora_b(dtype) - ora_e(dtype); }

static void put_bits(uint8_t* buf, uint64_t bitpos, int width, uint32_t value) {
    if (((bitpos | (uint64_t)width) & 7) == 0) { /* whole bytes (bf16, fp32): little-endian */
        for (int i = 0; i < width / 8; ++i) buf[(bitpos >> 3) + i] |= (uint8_t)(value >> (8 * i));
        return;
    }
    for (int i = 0; i < width; ++i) {
        uint64_t p = bitpos + (uint64_t)i;
        if ((value >> i) & 1u) buf[p >> 3] |= (uint8_t)(1u << (p & 7));
    }
}
static uint32_t get_bits(const uint8_t* buf, uint64_t bitpos, int width) {
    uint32_t v = 0;
    if (((bitpos | (uint64_t)width) & 7) == 0) {
        for (int i = 0; i < width / 8; ++i) v |= (uint32_t)buf[(bitpos >> 3) + i] << (8 * i);
        return v;
    }
    for (int i = 0; i < width; ++i) {
        uint64_t p = bitpos + (uint64_t)i;
        v |= (uint32_t)((buf[p >> 3] >> (p & 7)) & 1u) << i;
    }
    return v;
}

static uint64_t pad16(uint64_t x) { return (x + 15u) / 16u * 16u; }

/* S_b = ceil(N / B)  (Section 3.2). */
uint64_t ora_num_blocks(uint64_t n, uint32_t block) { return (n + block - 1) / block; }

/* S_bm = ceil(S_b / 8) bytes  (Section 3.2). */
uint64_t ora_bitmap_bytes(uint64_t n, uint32_t block) { return (ora_num_blocks(n, block) + 7) / 8; }

/* S_{s+m} = N * m / 8 bytes  (Section 3.2: S - S_e), rounded up to whole bytes. */
uint64_t ora_sm_bytes(uint64_t n, int dtype) { return (n * (uint64_t)ora_m(dtype) + 7) / 8; }

/* Exponent bytes of one block of len values on the wire: len * e / 8, rounded up (every block of
 * the payload starts on a byte boundary). */
uint64_t ora_block_payload_bytes(uint64_t len, int dtype) { return (len * (uint64_t)ora_e(dtype) + 7) / 8; }

uint64_t ora_sm_offset(uint64_t n, uint32_t block) { return pad16(ora_bitmap_bytes(n, block)); }

uint64_t ora_payload_offset(uint64_t n, int dtype, uint32_t block) {
    return ora_sm_offset(n, block) + pad16(ora_sm_bytes(n, dtype));
}

/* Worst case: every block changed (payload = N exponent bytes when e = 8). */
uint64_t ora_message_capacity(uint64_t n, int dtype, uint32_t block) {
    if (n == 0) return 0;
    uint64_t nb = ora_num_blocks(n, block);
    uint64_t last = n - (nb - 1) * block;
    return ora_payload_offset(n, dtype, block) + (nb - 1) * ora_block_payload_bytes(block, dtype) +
           ora_block_payload_bytes(last, dtype);
}

/* The paper's transmitted-byte count S_{s+m} + S_bm + (changed exponent bytes). */
uint64_t ora_paper_bytes(uint64_t n, int dtype, uint32_t block, uint64_t payload_bytes) {
    return ora_sm_bytes(n, dtype) + ora_bitmap_bytes(n, block) + payload_bytes;
}

static uint32_t load_bits(const void* w, uint64_t j, int dtype) {
    if (ora_b(dtype) == 16) {
        uint16_t v;
        memcpy(&v, (const uint8_t*)w + 2 * j, 2);
        return v;
    }
    uint32_t v;
    memcpy(&v, (const uint8_t*)w + 4 * j, 4);
    return v;
}

static void store_bits(void* w, uint64_t j, int dtype, uint32_t bits) {
    if (ora_b(dtype) == 16) {
        uint16_t v = (uint16_t)bits;
        memcpy((uint8_t*)w + 2 * j, &v, 2);
    } else {
        memcpy((uint8_t*)w + 4 * j, &bits, 4);
    }
}

/* One value -> exponent field and sign-plus-mantissa (the sender's first step in Algorithm 1). */
static void split_value(uint32_t bits, int dtype, uint8_t* exp, uint32_t* sm) {
    int b = ora_b(dtype), m = ora_m(dtype);
    uint32_t sign = (bits >> (b - 1)) & 1u;
    uint32_t expo = (bits >> (m - 1)) & ((1u << ora_e(dtype)) - 1u);
    uint32_t mant = bits & ((1u << (m - 1)) - 1u);
    *exp = (uint8_t)expo;
    *sm = (sign << (m - 1)) | mant;
}

/* Exponent field and sign-plus-mantissa -> one value (the receiver's last step in Algorithm 1). */
static uint32_t merge_value(uint8_t exp, uint32_t sm, int dtype) {
    int b = ora_b(dtype), m = ora_m(dtype);
    uint32_t sign = (sm >> (m - 1)) & 1u;
    uint32_t mant = sm & ((1u << (m - 1)) - 1u);
    return (sign << (b - 1)) | ((uint32_t)exp << (m - 1)) | mant;
}

/* Exposed so that tests can pin the per-value map on its own. */
void ora_split(const void* w, uint64_t n, int dtype, uint8_t* exp_out, uint32_t* sm_out) {
    for (uint64_t j = 0; j < n; ++j) split_value(load_bits(w, j, dtype), dtype, &exp_out[j], &sm_out[j]);
}

void ora_merge(const uint8_t* exp, const uint32_t* sm, uint64_t n, int dtype, void* w_out) {
    for (uint64_t j = 0; j < n; ++j) store_bits(w_out, j, dtype, merge_value(exp[j], sm[j], dtype));
}

/* Cache initialisation: exponents of W0 (as if W0 had been sent uncompressed), or all
 * zero when w == NULL (then the first encode marks every block holding a non-zero
 * exponent field as changed). */
void ora_cache_init(uint8_t* cache, const void* w, uint64_t n, int dtype) {
    for (uint64_t j = 0; j < n; ++j) {
        uint8_t e = 0;
        uint32_t sm;
        if (w) split_value(load_bits(w, j, dtype), dtype, &e, &sm);
        cache[j] = e;
    }
}

/*
 * Sender side of Algorithm 1 for one unit (one shard of one tensor).
 *   w        N values of dtype
 *   cache_s  N bytes, in/out: the exponents the sender last transmitted
 *   msg      out, at least ora_message_capacity(N, dtype, B) bytes
 * Outputs: wire_bytes (section-padded length that has to travel), payload_bytes
 * (sum of L_k over changed blocks), changed_blocks.
 * Returns 0, or -1 on allocation failure, -2 if msg_capacity is too small.
 */
int ora_encode(const void* w, uint8_t* cache_s, uint64_t n, int dtype, uint32_t block, uint8_t* msg,
               uint64_t msg_capacity, uint64_t* wire_bytes, uint64_t* payload_bytes, uint32_t* changed_blocks) {
    *wire_bytes = 0;
    *payload_bytes = 0;
    *changed_blocks = 0;
    if (n == 0) return 0;
    if (msg_capacity < ora_message_capacity(n, dtype, block)) return -2;

    int m = ora_m(dtype), e = ora_e(dtype);
    uint64_t nb = ora_num_blocks(n, block);
    uint64_t sm_off = ora_sm_offset(n, block);
    uint64_t pay_off = ora_payload_offset(n, dtype, block);

    /* every value cut into exponent field and sign-plus-mantissa */
    uint8_t* exp = (uint8_t*)malloc(n);
    uint32_t* sm = (uint32_t*)malloc(n * sizeof(uint32_t));
    if (!exp || !sm) {
        free(exp);
        free(sm);
        return -1;
    }
    ora_split(w, n, dtype, exp, sm);

    /* no block marked yet, nothing in the payload; the pads are zero as well */
    memset(msg, 0, pay_off);

    /* a block is marked when one of its exponents is not the cached one; its cached copy is then replaced */
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t lo = k * block;
        uint64_t hi = lo + block < n ? lo + block : n;
        int changed = 0;
        for (uint64_t j = lo; j < hi; ++j)
            if (exp[j] != cache_s[j]) changed = 1;
        if (changed) {
            msg[k >> 3] |= (uint8_t)(1u << (k & 7));
            for (uint64_t j = lo; j < hi; ++j) cache_s[j] = exp[j];
        }
    }

    /* sign-plus-mantissa of all values. */
    for (uint64_t j = 0; j < n; ++j) put_bits(msg + sm_off, j * (uint64_t)m, m, sm[j]);

    /* the exponents of the marked blocks, ascending */
    uint64_t plen = 0;
    uint32_t nchg = 0;
    for (uint64_t k = 0; k < nb; ++k) {
        if (!((msg[k >> 3] >> (k & 7)) & 1u)) continue;
        uint64_t lo = k * block;
        uint64_t hi = lo + block < n ? lo + block : n;
        uint64_t nbytes = ora_block_payload_bytes(hi - lo, dtype);
        memset(msg + pay_off + plen, 0, nbytes);
        for (uint64_t j = lo; j < hi; ++j) put_bits(msg + pay_off + plen, (j - lo) * (uint64_t)e, e, exp[j]);
        plen += nbytes;
        ++nchg;
    }

    *payload_bytes = plen;
    *changed_blocks = nchg;
    *wire_bytes = pay_off + plen;
    free(exp);
    free(sm);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Sender side with hash-based change detection (Section 3.1; Algorithm 1 as printed: the sender
 * keeps HashCache[i,k], a 128-bit hash per block, not the exponents themselves).
 *
 * The paper fixes only this much: the hash has 128 bits and is built from two independent 64-bit
 * SplitMix64 hashes.  The construction used here (a reading; the paper prints none):
 *   mix(z)  = the SplitMix64 output function: z ^= z >> 30; z *= 0xBF58476D1CE4E5B9;
 *             z ^= z >> 27; z *= 0x94D049BB133111EB; z ^= z >> 31
 *   a block of L exponent bytes is read as m = ceil(L / 8) little-endian 64-bit words x_0..x_{m-1}
 *   (the last one zero-padded);
 *   H_i     = mix( L + sum_j mix(s_i + (j + 1) * g_i + x_j) )      (all arithmetic mod 2^64)
 *   Hash128 = (H_1, H_2) with  s_1 = 0,                  g_1 = 0x9E3779B97F4A7C15 (the SplitMix64 increment),
 *                              s_2 = 0x6A09E667F3BCC908, g_2 = 0xD1342543DE82EF95 (another odd increment).
 * mix(s + (j + 1) * g) is the j-th output of a SplitMix64 generator with seed s and increment g, so each
 * word is added to that generator's state before the output function; summing the per-word terms
 * makes the hash independent of the order in which the words are visited.
 * The two hashes run on generators with different increments (as split instances of SplitMix64 do): with a
 * common increment, moving a word from position j to position i and adding (j - i) * g to it leaves the
 * multiset of per-word terms of BOTH hashes unchanged, whatever the seeds, so that the two would share a
 * family of collisions and not be independent; with different increments a rearrangement of that kind
 * collides one of them only (pinned in the tests).
 */
#define ORA_GAMMA 0x9E3779B97F4A7C15ull
#define ORA_GAMMA2 0xD1342543DE82EF95ull
#define ORA_SEED1 0x0000000000000000ull
#define ORA_SEED2 0x6A09E667F3BCC908ull

uint64_t ora_splitmix64_mix(uint64_t z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

/* next output of the SplitMix64 generator; *state is advanced (used by the pins only) */
uint64_t ora_splitmix64_next(uint64_t* state) {
    *state += ORA_GAMMA;
    return ora_splitmix64_mix(*state);
}

/* the same for a generator with another (odd) increment */
uint64_t ora_splitmix64_next_with(uint64_t* state, uint64_t gamma) {
    *state += gamma;
    return ora_splitmix64_mix(*state);
}

void ora_hash128(const uint8_t* exp, uint64_t len, uint64_t out[2]) {
    const uint64_t seeds[2] = {ORA_SEED1, ORA_SEED2};
    const uint64_t gammas[2] = {ORA_GAMMA, ORA_GAMMA2};
    for (int h = 0; h < 2; ++h) {
        uint64_t acc = 0;
        for (uint64_t j = 0; 8 * j < len; ++j) {
            uint64_t x = 0;
            for (uint64_t i = 0; i < 8 && 8 * j + i < len; ++i) x |= (uint64_t)exp[8 * j + i] << (8 * i);
            acc += ora_splitmix64_mix(seeds[h] + (j + 1) * gammas[h] + x);
        }
        out[h] = ora_splitmix64_mix(acc + len);
    }
}

/* HashCache := Hash128 of every block of exponents(w); of all-zero exponents when w == NULL.
 * hash_cache holds 2 * S_b words: (H_s1, H_s2) of block 0, of block 1, ... */
int ora_hash_cache_init(const void* w, uint64_t n, int dtype, uint32_t block, uint64_t* hash_cache) {
    if (n == 0) return 0;
    uint8_t* exp = (uint8_t*)calloc(n, 1);
    uint32_t* sm = (uint32_t*)malloc(n * sizeof(uint32_t));
    if (!exp || !sm) {
        free(exp);
        free(sm);
        return -1;
    }
    if (w) ora_split(w, n, dtype, exp, sm);
    uint64_t nb = ora_num_blocks(n, block);
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t lo = k * block;
        uint64_t hi = lo + block < n ? lo + block : n;
        ora_hash128(exp + lo, hi - lo, hash_cache + 2 * k);
    }
    free(exp);
    free(sm);
    return 0;
}

/* Same message layout and outputs as ora_encode; hash_cache (2 * S_b words) is in/out. */
int ora_encode_hashed(const void* w, uint64_t* hash_cache, uint64_t n, int dtype, uint32_t block, uint8_t* msg,
                      uint64_t msg_capacity, uint64_t* wire_bytes, uint64_t* payload_bytes,
                      uint32_t* changed_blocks) {
    *wire_bytes = 0;
    *payload_bytes = 0;
    *changed_blocks = 0;
    if (n == 0) return 0;
    if (msg_capacity < ora_message_capacity(n, dtype, block)) return -2;

    int m = ora_m(dtype), e = ora_e(dtype);
    uint64_t nb = ora_num_blocks(n, block);
    uint64_t sm_off = ora_sm_offset(n, block);
    uint64_t pay_off = ora_payload_offset(n, dtype, block);

    /* every value cut into exponent field and sign-plus-mantissa */
    uint8_t* exp = (uint8_t*)malloc(n);
    uint32_t* sm = (uint32_t*)malloc(n * sizeof(uint32_t));
    if (!exp || !sm) {
        free(exp);
        free(sm);
        return -1;
    }
    ora_split(w, n, dtype, exp, sm);
    memset(msg, 0, pay_off);

    /* a block is marked when its hash is not the cached one, which is then replaced */
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t lo = k * block;
        uint64_t hi = lo + block < n ? lo + block : n;
        uint64_t h[2];
        ora_hash128(exp + lo, hi - lo, h);
        if (h[0] != hash_cache[2 * k] || h[1] != hash_cache[2 * k + 1]) {
            msg[k >> 3] |= (uint8_t)(1u << (k & 7));
            hash_cache[2 * k] = h[0];
            hash_cache[2 * k + 1] = h[1];
        }
    }

    for (uint64_t j = 0; j < n; ++j) put_bits(msg + sm_off, j * (uint64_t)m, m, sm[j]);

    /* the exponents of the marked blocks, ascending (no entropy stage, as in ora_encode) */
    uint64_t plen = 0;
    uint32_t nchg = 0;
    for (uint64_t k = 0; k < nb; ++k) {
        if (!((msg[k >> 3] >> (k & 7)) & 1u)) continue;
        uint64_t lo = k * block;
        uint64_t hi = lo + block < n ? lo + block : n;
        uint64_t nbytes = ora_block_payload_bytes(hi - lo, dtype);
        memset(msg + pay_off + plen, 0, nbytes);
        for (uint64_t j = lo; j < hi; ++j) put_bits(msg + pay_off + plen, (j - lo) * (uint64_t)e, e, exp[j]);
        plen += nbytes;
        ++nchg;
    }
    *payload_bytes = plen;
    *changed_blocks = nchg;
    *wire_bytes = pay_off + plen;
    free(exp);
    free(sm);
    return 0;
}

/*
 * Receiver side of Algorithm 1 for one unit: patch ExpCache where bitmap[k] = 1,
 * then merge the cache with the received sign-plus-mantissa.
 *   msg      the unit's message (layout as written by the sender)
 *   cache_r  N bytes, in/out
 *   w_out    N values of dtype
 * Returns 0, or -1 on allocation failure.
 */
int ora_decode(const uint8_t* msg, uint8_t* cache_r, uint64_t n, int dtype, uint32_t block, void* w_out) {
    if (n == 0) return 0;
    int m = ora_m(dtype), e = ora_e(dtype);
    uint64_t nb = ora_num_blocks(n, block);
    uint64_t sm_off = ora_sm_offset(n, block);
    uint64_t pay_off = ora_payload_offset(n, dtype, block);

    uint64_t j_pay = 0; /* read position (bytes) in newExp */
    for (uint64_t k = 0; k < nb; ++k) {
        if (!((msg[k >> 3] >> (k & 7)) & 1u)) continue;
        uint64_t lo = k * block;
        uint64_t hi = lo + block < n ? lo + block : n;
        for (uint64_t j = lo; j < hi; ++j) cache_r[j] = (uint8_t)get_bits(msg + pay_off + j_pay, (j - lo) * (uint64_t)e, e);
        j_pay += ora_block_payload_bytes(hi - lo, dtype);
    }

    uint32_t* sm = (uint32_t*)malloc(n * sizeof(uint32_t));
    if (!sm) return -1;
    for (uint64_t j = 0; j < n; ++j) sm[j] = get_bits(msg + sm_off, j * (uint64_t)m, m);
    ora_merge(cache_r, sm, n, dtype, w_out);
    free(sm);
    return 0;
}

/*
 * Comm(.) of Section 3.2.  The paper profiles it at start-up and gives no closed
 * form; here it is either a caller-given table of (bytes, seconds) points, linearly
 * interpolated (and extended along the first / last segment outside the table), or,
 * with fewer than two points, the model alpha + (W - 1) * bytes / beta.
 */
static double comm_time(double bytes, int world, double alpha, double beta, const double* tb, const double* ts,
                        int n_points) {
    if (n_points < 2) return alpha + (double)(world - 1) * bytes / beta;
    int i = 0;
    while (i < n_points - 2 && bytes > tb[i + 1]) ++i;
    double t = (bytes - tb[i]) / (tb[i + 1] - tb[i]);
    return ts[i] + t * (ts[i + 1] - ts[i]);
}

/*
 * g_i = Comm(S) - ( Comm(S_{s+m} + S_bm + q S_e) + T_hash + T_cmp + T_decmp ).
 * With overlapped != 0 the sender-side terms are zero on the critical path
 * (Section 3.2, paragraph on pipelining).
 */
double ora_gain(uint64_t n, int dtype, uint32_t block, double q, int world, double alpha, double beta,
                const double* table_bytes, const double* table_secs, int n_points, double t_hash, double t_cmp,
                double t_decmp, int overlapped) {
    double S = (double)n * ora_b(dtype) / 8.0;
    double S_e = (double)n * ora_e(dtype) / 8.0; /* exponent bits per value / 8 */
    double S_sm = S - S_e;
    double S_bm = (double)ora_bitmap_bytes(n, block);
    double sent = S_sm + S_bm + q * S_e;
    if (overlapped) {
        t_hash = 0.0;
        t_cmp = 0.0;
    }
    return comm_time(S, world, alpha, beta, table_bytes, table_secs, n_points) -
           (comm_time(sent, world, alpha, beta, table_bytes, table_secs, n_points) + t_hash + t_cmp + t_decmp);
}
