/*
 * CPU oracle of the entropy stage: the exponents of changed blocks (the payload of a unit's
 * message) coded with a range variant of asymmetric numeral systems (rANS).
 *
 * TEST INFRASTRUCTURE ONLY -- never linked into, imported by or called from the CUDA library.
 *
 * What the paper says (Section 3.1; Algorithm 1): payload <- ANSEncode({exp[k] | bitmap[k] = 1})
 * on the sender, newExp <- ANSDecode(payload) on the receiver, done with a vendor library whose
 * stream format is not public.  Everything below is therefore this build's own reading of "ANS":
 * the published rANS recurrences (Duda 2013; the 32-bit-state, 16-bit-word form) and a stream
 * layout made for one warp per segment.  The coded bytes have no outside reference: parity
 * unpinned for the byte stream; the pins are the recurrences on a hand-worked example, exact
 * round trips, and the coded size against the empirical entropy.
 *
 * Model: one static table per unit.  h[s] = count of byte s in the raw payload of P bytes;
 *   f[s] = 0 if h[s] = 0, else max(1, floor(h[s] * 4096 / P));
 *   if sum f < 4096 the difference goes to the symbol with the largest count (lowest s on ties);
 *   if sum f > 4096, repeatedly take the symbol with the largest f (lowest s on ties) and lower
 *   it by min(f - 1, excess) until the sum is 4096;  c[s] = sum of f[s'] over s' < s.
 *
 * Coder: state x in [2^16, 2^32), probabilities in 1/4096.
 *   encode s:  if x >= f[s] * 2^20: emit the low 16 bits of x, x >>= 16;
 *              x <- floor(x / f[s]) * 4096 + (x mod f[s]) + c[s]
 *   decode:    slot = x mod 4096, s = the symbol with c[s] <= slot < c[s] + f[s];
 *              x <- f[s] * floor(x / 4096) + slot - c[s];  if x < 2^16: x <- x * 2^16 + next word
 *
 * Segments: the raw payload is cut into segments of 4096 bytes (the last one shorter).  Inside a
 * segment 32 coders ("lanes") work side by side: lane l owns the bytes at positions 32 t + l
 * (step t).  The encoder walks the steps from the last to the first, at each step the lanes in
 * ascending order, appending emitted words to the segment's word list; the decoder walks the steps
 * forwards and takes the words from the END of the list backwards: at a step the k lanes that
 * need a word read the k words before its read position, lanes in ascending order.
 *
 * Coded section of a unit (replaces the raw payload when it is strictly shorter, which is how the
 * receiver tells the two apart -- it knows P from the bitmap):
 *   [A x u16 f[s]] [n_seg x u32: number of 16-bit words of each segment] [segment 0] [segment 1] ...
 *   segment = [32 x u32 final lane states] [its 16-bit words] [2 zero bytes if their number is odd]
 * all little-endian; every segment starts on a 4-byte boundary of the section.
 *
 * Alphabet: Algorithm 1 codes the exponents themselves, {exp[k] | bitmap[k] = 1}.  For bf16 and fp32
 * an exponent is a byte and the raw payload is the symbol sequence (A = 256 table entries).  An fp16
 * exponent has five bits: the symbols are the exponents of the changed blocks in order, one per
 * entry of raw[], all below 32, and only A = 32 table entries travel (the five-bit packing of the raw
 * payload is undone before and redone after the coder by the caller; "raw length" in the rule above
 * is then the length of the packed payload, while segments are cut every 4096 SYMBOLS).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define RANS_PROB_BITS 12
#define RANS_PROB_SCALE 4096u
#define RANS_L 65536u
#define RANS_LANES 32
#define RANS_SEGMENT 4096u

/* Normalised frequencies of a histogram; total = sum h > 0. */
void rans_normalise(const uint64_t h[256], uint64_t total, uint16_t f[256]) {
    uint32_t sum = 0;
    int best = 0;
    for (int s = 0; s < 256; ++s) {
        uint32_t v = 0;
        if (h[s]) {
            v = (uint32_t)(h[s] * RANS_PROB_SCALE / total);
            if (v == 0) v = 1;
        }
        f[s] = (uint16_t)v;
        sum += v;
        if (h[s] > h[best]) best = s;
    }
    if (sum < RANS_PROB_SCALE) {
        f[best] = (uint16_t)(f[best] + (RANS_PROB_SCALE - sum));
    } else {
        uint32_t excess = sum - RANS_PROB_SCALE;
        while (excess) {
            int big = 0;
            for (int s = 1; s < 256; ++s)
                if (f[s] > f[big]) big = s;
            uint32_t take = (uint32_t)f[big] - 1u < excess ? (uint32_t)f[big] - 1u : excess;
            f[big] = (uint16_t)(f[big] - take);
            excess -= take;
        }
    }
}

static void put16(uint8_t* p, uint32_t v) {
    p[0] = (uint8_t)v;
    p[1] = (uint8_t)(v >> 8);
}
static void put32(uint8_t* p, uint32_t v) {
    put16(p, v & 0xFFFFu);
    put16(p + 2, v >> 16);
}
static uint32_t get16(const uint8_t* p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8); }
static uint32_t get32(const uint8_t* p) { return get16(p) | (get16(p + 2) << 16); }

/* One encoder step of one lane (exposed for the hand-worked pin).  Returns 1 and sets *word if a
 * word was emitted. */
int rans_encode_step(uint32_t* x, uint32_t f, uint32_t c, uint32_t* word) {
    int emitted = 0;
    if ((uint64_t)*x >= ((uint64_t)f << 20)) {
        *word = *x & 0xFFFFu;
        *x >>= 16;
        emitted = 1;
    }
    *x = (*x / f) * RANS_PROB_SCALE + (*x % f) + c;
    return emitted;
}

/* Upper bound on the coded size of P symbols with A table entries (what a caller must be able to hold). */
uint64_t rans_coded_bound_alphabet(uint64_t P, uint32_t A) {
    uint64_t nseg = (P + RANS_SEGMENT - 1) / RANS_SEGMENT;
    /* a symbol makes the state grow by at most 12 bits, a word takes 16 away */
    return 2 * (uint64_t)A + 4 * nseg + nseg * (4 * RANS_LANES + 4) + (P * RANS_PROB_BITS + 15) / 16 * 2;
}
uint64_t rans_coded_bound(uint64_t P) { return rans_coded_bound_alphabet(P, 256); }

/*
 * Codes the symbols raw[0..P), each below A (A = 256 or 32), into out (at least
 * rans_coded_bound_alphabet(P, A) bytes).  Returns the coded size in bytes, or 0 if P = 0 or a symbol
 * does not fit the alphabet.  The caller compares it with the raw length to decide which form travels.
 */
uint64_t rans_encode_alphabet(const uint8_t* raw, uint64_t P, uint8_t* out, uint32_t A) {
    if (P == 0 || (A != 256 && A != 32)) return 0;
    uint64_t h[256] = {0};
    for (uint64_t i = 0; i < P; ++i) {
        if (raw[i] >= A) return 0;
        h[raw[i]]++;
    }
    uint16_t f[256];
    uint32_t c[256];
    rans_normalise(h, P, f);
    uint32_t run = 0;
    for (uint32_t s = 0; s < 256; ++s) {
        c[s] = run;
        run += f[s];
        if (s < A) put16(out + 2 * s, f[s]);
    }
    uint64_t nseg = (P + RANS_SEGMENT - 1) / RANS_SEGMENT;
    uint8_t* dir = out + 2 * A;
    uint8_t* dst = dir + 4 * nseg;
    uint16_t* words = (uint16_t*)malloc(sizeof(uint16_t) * RANS_SEGMENT);
    for (uint64_t g = 0; g < nseg; ++g) {
        const uint8_t* seg = raw + g * RANS_SEGMENT;
        uint32_t n = (uint32_t)(P - g * RANS_SEGMENT < RANS_SEGMENT ? P - g * RANS_SEGMENT : RANS_SEGMENT);
        uint32_t steps = (n + RANS_LANES - 1) / RANS_LANES;
        uint32_t x[RANS_LANES];
        for (int l = 0; l < RANS_LANES; ++l) x[l] = RANS_L;
        uint32_t nw = 0;
        for (uint32_t t = steps; t-- > 0;) {
            for (uint32_t l = 0; l < RANS_LANES; ++l) {
                uint32_t i = RANS_LANES * t + l;
                if (i >= n) continue;
                uint32_t w;
                if (rans_encode_step(&x[l], f[seg[i]], c[seg[i]], &w)) words[nw++] = (uint16_t)w;
            }
        }
        for (int l = 0; l < RANS_LANES; ++l) put32(dst + 4 * l, x[l]);
        for (uint32_t k = 0; k < nw; ++k) put16(dst + 4 * RANS_LANES + 2 * k, words[k]);
        uint32_t size = 4 * RANS_LANES + 2 * nw;
        if (nw & 1u) {
            put16(dst + size, 0);
            size += 2;
        }
        put32(dir + 4 * g, nw);
        dst += size;
    }
    free(words);
    return (uint64_t)(dst - out);
}
uint64_t rans_encode(const uint8_t* raw, uint64_t P, uint8_t* out) { return rans_encode_alphabet(raw, P, out, 256); }

/* Decodes a coded section with A table entries back into the symbols raw[0..P).  Returns 0, or -1 if
 * the section is inconsistent (sizes that do not add up to coded_bytes, a table that does not sum to
 * 4096). */
int rans_decode_alphabet(const uint8_t* in, uint64_t coded_bytes, uint64_t P, uint8_t* raw, uint32_t A) {
    if (A != 256 && A != 32) return -1;
    if (P == 0) return coded_bytes == 0 ? 0 : -1;
    uint64_t nseg = (P + RANS_SEGMENT - 1) / RANS_SEGMENT;
    if (coded_bytes < 2 * (uint64_t)A + 4 * nseg) return -1;
    uint32_t f[256], c[256];
    uint8_t* sym = (uint8_t*)malloc(RANS_PROB_SCALE);
    uint32_t run = 0;
    for (uint32_t s = 0; s < A; ++s) {
        f[s] = get16(in + 2 * s);
        c[s] = run;
        if (run + f[s] > RANS_PROB_SCALE) {
            free(sym);
            return -1;
        }
        for (uint32_t k = 0; k < f[s]; ++k) sym[run + k] = (uint8_t)s;
        run += f[s];
    }
    if (run != RANS_PROB_SCALE) {
        free(sym);
        return -1;
    }
    const uint8_t* dir = in + 2 * A;
    const uint8_t* src = dir + 4 * nseg;
    int rc = 0;
    for (uint64_t g = 0; g < nseg && rc == 0; ++g) {
        uint32_t nw = get32(dir + 4 * g);
        uint64_t size = 4 * RANS_LANES + 2 * (uint64_t)nw + ((nw & 1u) ? 2 : 0);
        if ((uint64_t)(src - in) + size > coded_bytes) {
            rc = -1;
            break;
        }
        uint32_t n = (uint32_t)(P - g * RANS_SEGMENT < RANS_SEGMENT ? P - g * RANS_SEGMENT : RANS_SEGMENT);
        uint32_t steps = (n + RANS_LANES - 1) / RANS_LANES;
        uint32_t x[RANS_LANES];
        for (int l = 0; l < RANS_LANES; ++l) x[l] = get32(src + 4 * l);
        const uint8_t* wbase = src + 4 * RANS_LANES;
        uint32_t ptr = nw; /* read position: one past the last unread word */
        uint8_t* o = raw + g * RANS_SEGMENT;
        for (uint32_t t = 0; t < steps; ++t) {
            /* decode this step's symbols, then hand out words to the lanes that need one */
            uint32_t need[RANS_LANES], k = 0;
            for (uint32_t l = 0; l < RANS_LANES; ++l) {
                uint32_t i = RANS_LANES * t + l;
                if (i >= n) continue;
                uint32_t slot = x[l] & (RANS_PROB_SCALE - 1);
                uint32_t s = sym[slot];
                o[i] = (uint8_t)s;
                x[l] = f[s] * (x[l] >> RANS_PROB_BITS) + slot - c[s];
                if (x[l] < RANS_L) need[k++] = l;
            }
            if (k > ptr) {
                rc = -1;
                break;
            }
            for (uint32_t r = 0; r < k; ++r) x[need[r]] = (x[need[r]] << 16) | get16(wbase + 2 * (ptr - k + r));
            ptr -= k;
        }
        /* all words used and every lane back at its start state, or the section is damaged */
        if (rc == 0 && ptr != 0) rc = -1;
        for (int l = 0; l < RANS_LANES && rc == 0; ++l)
            if (x[l] != RANS_L) rc = -1;
        src += size;
    }
    if (rc == 0 && (uint64_t)(src - in) != coded_bytes) rc = -1;
    free(sym);
    return rc;
}
int rans_decode(const uint8_t* in, uint64_t coded_bytes, uint64_t P, uint8_t* raw) {
    return rans_decode_alphabet(in, coded_bytes, P, raw, 256);
}
