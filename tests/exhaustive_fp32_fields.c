/*
 * Test program (not part of the library, not part of the oracle): every one of the 2^32 binary32 bit patterns
 * through the oracle's split and merge, checked against the NUMERIC definition of the IEEE-754 fields taken
 * with frexpf / ldexpf from <math.h> -- no shifts or masks on this side, so a wrong field position or width in
 * the oracle cannot cancel out.  For a finite non-zero value |x| = m * 2^e with m in [0.5, 1):
 *   normal    (e >= -125): exponent field E = e + 126, mantissa field M = m * 2^24 - 2^23
 *   subnormal (e <  -125): E = 0, M = |x| * 2^149
 * zero: E = M = 0; infinity: E = 255, M = 0; NaN: E = 255 (its payload has no numeric definition: there the
 * round trip merge(split(x)) == x, checked for every pattern, is what pins the bits).
 * The oracle must return exp = E and sm = sign << 23 | M.
 *
 * Built and run by tests/test_oracle_pins.py together with oracle/ciera_oracle.c; prints "ok <count>" or the
 * first mismatch.  Usage: exhaustive_fp32_fields [first_pattern count]   (default: all 2^32)
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

void ora_split(const void* w, uint64_t n, int dtype, uint8_t* exp, uint32_t* sm);
void ora_merge(const uint8_t* exp, const uint32_t* sm, uint64_t n, int dtype, void* w);

enum { CHUNK = 1 << 20, FP32 = 1 };

int main(int argc, char** argv) {
    uint64_t first = 0, count = 1ull << 32;
    if (argc == 3) {
        first = strtoull(argv[1], NULL, 0);
        count = strtoull(argv[2], NULL, 0);
    }
    const uint64_t chunks = (count + CHUNK - 1) / CHUNK;
    int failed = 0;
#pragma omp parallel
    {
        uint32_t* bits = malloc(sizeof(uint32_t) * CHUNK);
        uint32_t* back = malloc(sizeof(uint32_t) * CHUNK);
        uint32_t* sm = malloc(sizeof(uint32_t) * CHUNK);
        uint8_t* ex = malloc(CHUNK);
#pragma omp for schedule(dynamic)
        for (uint64_t c = 0; c < chunks; ++c) {
            if (failed) continue;
            const uint64_t lo = first + c * CHUNK;
            const uint64_t n = (c + 1) * CHUNK <= count ? CHUNK : count - c * CHUNK;
            for (uint64_t i = 0; i < n; ++i) bits[i] = (uint32_t)(lo + i);
            ora_split(bits, n, FP32, ex, sm);
            ora_merge(ex, sm, n, FP32, back);
            for (uint64_t i = 0; i < n && !failed; ++i) {
                float x;
                memcpy(&x, &bits[i], 4);
                long E, M = -1;  /* M = -1: not defined numerically (NaN) */
                const long sign = signbit(x) ? 1 : 0;
                if (isnan(x)) {
                    E = 255;
                } else if (isinf(x)) {
                    E = 255;
                    M = 0;
                } else if (x == 0.0f) {
                    E = 0;
                    M = 0;
                } else {
                    int e;
                    const float m = frexpf(fabsf(x), &e);
                    if (e >= -125) {
                        E = e + 126;
                        M = (long)(ldexpf(m, 24) - 8388608.0f);
                    } else {
                        E = 0;
                        M = (long)ldexpf(fabsf(x), 149);
                    }
                }
                const int bad = ex[i] != E || (long)(sm[i] >> 23) != sign || (M >= 0 && (long)(sm[i] & 0x7FFFFFu) != M) ||
                                sm[i] >= (1u << 24) || back[i] != bits[i];
                if (bad) {
#pragma omp critical
                    {
                        if (!failed)
                            printf("mismatch at pattern 0x%08x: exp %u sm 0x%06x, expected E %ld sign %ld M %ld, merged 0x%08x\n",
                                   bits[i], ex[i], sm[i], E, sign, M, back[i]);
                        failed = 1;
                    }
                }
            }
        }
        free(bits);
        free(back);
        free(sm);
        free(ex);
    }
    if (failed) return 1;
    printf("ok %llu\n", (unsigned long long)count);
    return 0;
}
