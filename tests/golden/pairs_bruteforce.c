/*
 * Exhaustive check of the two-rank bf16 all-reduce of the oracle: all 2^32 pairs (a, b).
 *
 * The expected value is computed here by a route that shares nothing with the oracle's
 * arithmetic: both operands are widened to binary64, added there (exact whenever the
 * exponents differ by at most 45, and otherwise the smaller operand is far below half an
 * ulp of the larger one in binary32, so rounding the binary64 sum to binary32 still gives
 * the correctly rounded binary32 sum), rounded once to binary32, and then rounded to bf16
 * by comparing distances to the two neighbouring bf16 values (ties to the even one),
 * instead of the add-and-shift trick the oracle uses.  NaN results must be 0x7FFF.
 *
 * Usage: pairs_bruteforce [first_a last_a]   (default 0 65535).  Prints the number of pairs
 * checked and of mismatches; exit status 1 on any mismatch.  Links against the oracle's C
 * source (test infrastructure only).
 *
 *        pairs_bruteforce round first_hi last_hi
 * checks the oracle's binary32 -> bf16 rounding alone on every bit pattern whose upper 16 bits
 * lie in [first_hi, last_hi] (all 2^32 patterns for 0 65535) against the same distance rule.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

void oracle_allreduce_bf16(const uint16_t *const *x, int P, size_t n, uint16_t *out);
uint16_t oracle_f32_to_bf16(float f);

static double widen(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

static uint16_t nearest_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if (isnan(f)) return 0x7FFF;
    if (isinf(f)) return (uint16_t)(u >> 16);
    const uint32_t lo_bits = u & 0xFFFF0000u;                /* towards zero */
    const uint32_t hi_bits = lo_bits + 0x00010000u;          /* away from zero: may carry into the exponent, up to inf */
    if (lo_bits == u) return (uint16_t)(u >> 16);            /* already a bf16 value */
    float lo, hi;
    memcpy(&lo, &lo_bits, 4);
    memcpy(&hi, &hi_bits, 4);
    /* hi is inf when f lies beyond the largest finite bf16: distance measured to 2^128 of the same sign */
    const double dhi = isinf(hi) ? fabs(copysign(ldexp(1.0, 128), (double)f) - (double)f) : fabs((double)hi - (double)f);
    const double dlo = fabs((double)f - (double)lo);
    if (dlo < dhi) return (uint16_t)(lo_bits >> 16);
    if (dhi < dlo) return (uint16_t)(hi_bits >> 16);
    return (uint16_t)((((lo_bits >> 16) & 1u) == 0u ? lo_bits : hi_bits) >> 16);   /* tie: even mantissa */
}

static int check_rounding(unsigned first_hi, unsigned last_hi)
{
    unsigned long long checked = 0, bad = 0;
    for (unsigned hi = first_hi; hi <= last_hi && hi < 65536u; ++hi)
        for (unsigned lo = 0; lo < 65536u; ++lo) {
            const uint32_t u = (hi << 16) | lo;
            float f;
            memcpy(&f, &u, 4);
            const uint16_t got = oracle_f32_to_bf16(f), want = nearest_bf16(f);
            if (got != want) {
                if (bad < 10) fprintf(stderr, "bits=%08x oracle=%04x expected=%04x\n", u, got, want);
                ++bad;
            }
            ++checked;
        }
    printf("%llu %llu\n", checked, bad);
    return bad ? 1 : 0;
}

int main(int argc, char **argv)
{
    if (argc > 3 && strcmp(argv[1], "round") == 0)
        return check_rounding((unsigned)strtoul(argv[2], NULL, 0), (unsigned)strtoul(argv[3], NULL, 0));
    const unsigned first = argc > 2 ? (unsigned)strtoul(argv[1], NULL, 0) : 0u;
    const unsigned last = argc > 2 ? (unsigned)strtoul(argv[2], NULL, 0) : 65535u;
    enum { N = 65536 };
    uint16_t *xa = malloc(N * 2), *xb = malloc(N * 2), *out = malloc(N * 2);
    if (!xa || !xb || !out) return 2;
    for (unsigned b = 0; b < N; ++b) xb[b] = (uint16_t)b;
    unsigned long long checked = 0, bad = 0;
    for (unsigned a = first; a <= last && a < N; ++a) {
        for (unsigned i = 0; i < N; ++i) xa[i] = (uint16_t)a;
        const uint16_t *xs[2] = {xa, xb};
        oracle_allreduce_bf16(xs, 2, N, out);
        const double da = widen((uint16_t)a);
        for (unsigned b = 0; b < N; ++b) {
            const float s = (float)(da + widen((uint16_t)b));
            const uint16_t want = nearest_bf16(s);
            if (out[b] != want) {
                if (bad < 10) fprintf(stderr, "a=%04x b=%04x oracle=%04x expected=%04x\n", a, b, out[b], want);
                ++bad;
            }
        }
        checked += N;
    }
    printf("%llu %llu\n", checked, bad);
    free(xa); free(xb); free(out);
    return bad ? 1 : 0;
}
