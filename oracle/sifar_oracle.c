/*
 * CPU oracle for the emulated oneshot all-reduce and for the synthetic
 * decode-step workloads that drive it.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the GPU library can be
 * checked against a plain, slow, obviously correct restatement of what the
 * method computes.  Only the test-suite, the smoke check and the CPU-baseline
 * leg of the benchmark may call it.  It shares no source, header, table or
 * helper with the CUDA library and is never a fallback for it.
 *
 * What is computed (paper, Section 3.1 "Oneshot", phase 2, and the oneshot
 * half of the first listing of Section 4.2): every rank holds a partial of n
 * elements; the result is the element-wise sum over the ranks, peers visited
 * in the order 0..P-1.  The paper leaves precision and the starting value of
 * the accumulator open; the reading taken here is
 *
 *     acc    = widen(x_0[i])                       (exact, so P = 1 is the identity)
 *     acc    = acc + widen(x_r[i])   r = 1..P-1    (IEEE binary32 add, RNE, this order)
 *     out[i] = narrow(acc)                         (one RNE to bf16; identity for fp32)
 *
 * The barriers, dual buffering and speculation of Sections 3.3-3.5 and 4 change
 * WHEN the partials are read, never WHAT is computed, so this one function is
 * the expected value for all three modes of the library.
 *
 * Parity pins (tests/test_oracle_pins.py): P = 1 identity, P equal copies give
 * P*x, integer inputs against exact integer arithmetic in every rank order,
 * fp32 adds against float64 arithmetic, bf16 rounding against a rational-
 * arithmetic rounder and against torch's CPU cast, hand-derived ties
 * (tests/golden/bf16_ties.txt), and all 2^32 two-rank bf16 pairs against a
 * binary64 route with a distance-based rounding (tests/golden/pairs_bruteforce.c).  The workload generator below is a definition,
 * not a result: it is pinned by range, moment and frequency checks.
 *
 * Build: gcc -O1 -ffp-contract=off -fno-fast-math -fPIC -shared (see oracle/oracle.py).
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* bf16 <-> binary32                                                         */
/* ------------------------------------------------------------------------ */

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* bf16 is the upper half of a binary32: widening appends sixteen zero bits. */
float oracle_bf16_to_f32(uint16_t b) { return bits_f32((uint32_t)b << 16); }

/*
 * Round a binary32 to the nearest bf16, ties to the even bf16.
 * NaN maps to the canonical quiet NaN 0x7FFF (what the GPU's conversion
 * instruction returns); everything else, subnormals included, is rounded on
 * its bit pattern: the discarded 16 bits are compared with one half, and a
 * carry out of the mantissa correctly bumps the exponent (up to infinity).
 */
uint16_t oracle_f32_to_bf16(float f)
{
    uint32_t u = f32_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FFFu;
    uint32_t low = u & 0xFFFFu;          /* discarded part              */
    uint32_t keep = u >> 16;             /* truncated bf16              */
    if (low > 0x8000u) keep += 1;        /* above one half: round up    */
    else if (low == 0x8000u) keep += (keep & 1u);   /* tie: to even     */
    return (uint16_t)keep;
}

/* The same conversions over arrays (bit patterns in, bit patterns out). */
void oracle_f32_to_bf16_array(const float *f, size_t n, uint16_t *b)
{
    for (size_t i = 0; i < n; ++i) b[i] = oracle_f32_to_bf16(f[i]);
}

void oracle_bf16_to_f32_array(const uint16_t *b, size_t n, float *f)
{
    for (size_t i = 0; i < n; ++i) f[i] = oracle_bf16_to_f32(b[i]);
}

/* ------------------------------------------------------------------------ */
/* The reduction                                                             */
/* ------------------------------------------------------------------------ */

/* x: array of P pointers, each to n bf16 bit patterns.  out: n bf16. */
void oracle_allreduce_bf16(const uint16_t *const *x, int P, size_t n, uint16_t *out)
{
    for (size_t i = 0; i < n; ++i) {
        float acc = oracle_bf16_to_f32(x[0][i]);
        for (int r = 1; r < P; ++r)
            acc = acc + oracle_bf16_to_f32(x[r][i]);
        out[i] = oracle_f32_to_bf16(acc);
    }
}

/* x: array of P pointers, each to n binary32 values.  out: n binary32. */
void oracle_allreduce_f32(const float *const *x, int P, size_t n, float *out)
{
    for (size_t i = 0; i < n; ++i) {
        float acc = x[0][i];
        for (int r = 1; r < P; ++r)
            acc = acc + x[r][i];
        out[i] = acc;
    }
}

/* ------------------------------------------------------------------------ */
/* Counter-based generator of the synthetic workloads                        */
/* ------------------------------------------------------------------------ */
/*
 * The decode-step workloads (64 or 120 dependent all-reduces, each rank's next
 * partial derived from the previous result plus seeded noise) need the same
 * random numbers on the CPU and on the GPU.  Both sides therefore restate this
 * integer-only counter generator; every real value derived from it is exact in
 * binary32, so the two restatements agree bit for bit.
 *
 * mix():  a 32-bit avalanche (xor-shift / odd multiply, the "lowbias32"
 *         constants).
 * word(): six chained mixes over (seed, stream, rank, step, element, lane).
 */
static uint32_t mix(uint32_t x)
{
    x ^= x >> 16; x *= 0x7FEB352Du;
    x ^= x >> 15; x *= 0x846CA68Bu;
    x ^= x >> 16;
    return x;
}

enum { STREAM_VALUE = 1, STREAM_OUTLIER = 2, STREAM_DELAY = 3 };

uint32_t oracle_gen_word(uint32_t seed, uint32_t stream, uint32_t r, uint32_t t,
                         uint32_t i, uint32_t k)
{
    uint32_t h = mix(seed);
    h = mix(h ^ stream);
    h = mix(h + r);
    h = mix(h ^ (t * 0x9E3779B9u));
    h = mix(h + i);
    h = mix(h ^ k);
    return h;
}

/* Uniform on [-1, 1): a 24-bit integer centred on zero, scaled by 2^-23. */
float oracle_gen_uniform(uint32_t seed, uint32_t r, uint32_t t, uint32_t i)
{
    uint32_t w = oracle_gen_word(seed, STREAM_VALUE, r, t, i, 0);
    int32_t c = (int32_t)(w >> 8) - (1 << 23);
    return (float)c * (1.0f / 8388608.0f);
}

/*
 * Approximately standard normal: the sum of twelve independent 16-bit
 * uniforms (the two halves of six words) has mean 12*65535/2 = 393210 and
 * standard deviation ~65536, so (sum - 393210) * 2^-16 is ~N(0,1), |z| < 6.
 */
float oracle_gen_gauss(uint32_t seed, uint32_t r, uint32_t t, uint32_t i)
{
    int32_t s = 0;
    for (uint32_t k = 0; k < 6; ++k) {
        uint32_t w = oracle_gen_word(seed, STREAM_VALUE, r, t, i, k);
        s += (int32_t)(w & 0xFFFFu) + (int32_t)(w >> 16);
    }
    return (float)(s - 393210) * (1.0f / 65536.0f);
}

/* Integer in [0, 128]. */
int32_t oracle_gen_int129(uint32_t seed, uint32_t r, uint32_t t, uint32_t i)
{
    return (int32_t)(oracle_gen_word(seed, STREAM_VALUE, r, t, i, 0) % 129u);
}

/* 1 if element (r, i) is an outlier: one element in outlier_mod. */
int oracle_gen_is_outlier(uint32_t seed, uint32_t r, uint32_t i, uint32_t outlier_mod)
{
    if (outlier_mod == 0) return 0;
    return oracle_gen_word(seed, STREAM_OUTLIER, r, 0, i, 0) % outlier_mod == 0;
}

/* Producer delay of rank r at step t, in nanoseconds, uniform on [0, max]. */
uint32_t oracle_gen_delay_ns(uint32_t seed, uint32_t r, uint32_t t, uint32_t delay_max_ns)
{
    if (delay_max_ns == 0) return 0;
    return oracle_gen_word(seed, STREAM_DELAY, r, t, 0, 0) % (delay_max_ns + 1u);
}

/* ------------------------------------------------------------------------ */
/* The workloads: first partials and the producer's elementwise update       */
/* ------------------------------------------------------------------------ */
/*
 * Between two all-reduces of a decode step each rank runs "the next operation"
 * on the reduced tensor and produces its next partial (paper, Section 2.3,
 * two all-reduces per layer, each fed by the previous one's result).  The
 * weights are not available, so the operation is a seeded elementwise update:
 *
 *   kind 0 (gauss) / kind 2 (uniform), noise z ~ N(0,1) resp. U(-1,1):
 *       x_r^1[i]     = narrow( z(r,1,i) * (outlier ? 100 : 1) )
 *       x_r^{t+1}[i] = narrow( widen(out^t[i]) * scale  +  z(r,t+1,i) * sigma )
 *     with every product and the sum rounded separately (no fused multiply-add).
 *   kind 1 (integers, for the skewed-arrival stress):
 *       x_r^1[i]     = k(r,1,i) - 64
 *       x_r^{t+1}[i] = ((int(out^t[i]) + k(r,t+1,i)) mod 129, taken in [0,128]) - 64
 *     so every partial is an integer in [-64, 64], exact in bf16 and binary32.
 */
typedef struct {
    int32_t  kind;          /* 0 gauss, 1 integers, 2 uniform              */
    uint32_t seed;
    float    scale;         /* multiplies the previous result (kinds 0, 2) */
    float    sigma;         /* multiplies the fresh noise     (kinds 0, 2) */
    uint32_t outlier_mod;   /* 0: none; m: one first partial in m is x100  */
    uint32_t delay_max_ns;  /* producer spin before storing; values unaffected */
} oracle_workload;

static float noise_of(const oracle_workload *w, uint32_t r, uint32_t t, uint32_t i)
{
    return w->kind == 2 ? oracle_gen_uniform(w->seed, r, t, i)
                        : oracle_gen_gauss(w->seed, r, t, i);
}

static int32_t wrap129(int32_t v) { return ((v % 129) + 129) % 129; }

/* First partial of rank r (step t = 1), as binary32 before narrowing. */
static float first_value(const oracle_workload *w, uint32_t r, uint32_t i)
{
    if (w->kind == 1)
        return (float)(oracle_gen_int129(w->seed, r, 1, i) - 64);
    float z = noise_of(w, r, 1, i);
    if (oracle_gen_is_outlier(w->seed, r, i, w->outlier_mod))
        z = z * 100.0f;
    return z;
}

/* Partial of rank r at step t >= 2 from the previous result, before narrowing. */
static float next_value(const oracle_workload *w, uint32_t r, uint32_t t, uint32_t i, float prev)
{
    if (w->kind == 1)
        return (float)(wrap129((int32_t)prev + oracle_gen_int129(w->seed, r, t, i)) - 64);
    float a = prev * w->scale;
    float b = noise_of(w, r, t, i) * w->sigma;
    return a + b;
}

/* x_r^1 for one rank, bf16. */
void oracle_workload_first_bf16(const oracle_workload *w, int r, size_t n, uint16_t *x)
{
    for (size_t i = 0; i < n; ++i)
        x[i] = oracle_f32_to_bf16(first_value(w, (uint32_t)r, (uint32_t)i));
}

void oracle_workload_first_f32(const oracle_workload *w, int r, size_t n, float *x)
{
    for (size_t i = 0; i < n; ++i)
        x[i] = first_value(w, (uint32_t)r, (uint32_t)i);
}

/* x_r^t (t >= 2) for one rank from out^{t-1}, bf16. */
void oracle_workload_next_bf16(const oracle_workload *w, int r, uint32_t t, size_t n,
                               const uint16_t *prev_out, uint16_t *x)
{
    for (size_t i = 0; i < n; ++i)
        x[i] = oracle_f32_to_bf16(
            next_value(w, (uint32_t)r, t, (uint32_t)i, oracle_bf16_to_f32(prev_out[i])));
}

void oracle_workload_next_f32(const oracle_workload *w, int r, uint32_t t, size_t n,
                              const float *prev_out, float *x)
{
    for (size_t i = 0; i < n; ++i)
        x[i] = next_value(w, (uint32_t)r, t, (uint32_t)i, prev_out[i]);
}

/*
 * A whole chain: `steps` dependent all-reduces starting at step t0 (1-based).
 * If t0 == 1 the first partials are generated, otherwise `out_prev` must hold
 * out^{t0-1}.  `outs` receives out^{t0} .. out^{t0+steps-1} back to back
 * (steps * n elements).  `scratch` holds P * n elements.  dtype: 0 bf16, 1 fp32.
 */
void oracle_chain(const oracle_workload *w, int P, size_t n, int dtype, uint32_t t0,
                  int steps, const void *out_prev, void *outs, void *scratch)
{
    const void *prev = out_prev;
    for (int s = 0; s < steps; ++s) {
        uint32_t t = t0 + (uint32_t)s;
        if (dtype == 0) {
            uint16_t *x = (uint16_t *)scratch;
            const uint16_t *xs[16];
            for (int r = 0; r < P; ++r) {
                xs[r] = x + (size_t)r * n;
                if (t == 1) oracle_workload_first_bf16(w, r, n, x + (size_t)r * n);
                else oracle_workload_next_bf16(w, r, t, n, (const uint16_t *)prev, x + (size_t)r * n);
            }
            uint16_t *o = (uint16_t *)outs + (size_t)s * n;
            oracle_allreduce_bf16(xs, P, n, o);
            prev = o;
        } else {
            float *x = (float *)scratch;
            const float *xs[16];
            for (int r = 0; r < P; ++r) {
                xs[r] = x + (size_t)r * n;
                if (t == 1) oracle_workload_first_f32(w, r, n, x + (size_t)r * n);
                else oracle_workload_next_f32(w, r, t, n, (const float *)prev, x + (size_t)r * n);
            }
            float *o = (float *)outs + (size_t)s * n;
            oracle_allreduce_f32(xs, P, n, o);
            prev = o;
        }
    }
}
