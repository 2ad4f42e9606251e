/*
 * sifar_gen.cuh - device restatement of the seeded workload generator and of the
 * update rules of a rank's "next operation" (include/sifar_workload.h), shared by
 * the chain kernels.  Integer-only counter generator; every floating-point step is
 * a single correctly rounded operation, so the CPU restatements agree bit for bit.
 */
#ifndef SIFAR_GEN_CUH
#define SIFAR_GEN_CUH

#include "sifar_internal.cuh"
#include "sifar_workload.h"

namespace sifar {

/* ------------------------------------------------------------------------ */
/* counter generator (device restatement; integer-only, exact in binary32)   */
/* ------------------------------------------------------------------------ */
__host__ __device__ __forceinline__ uint32_t mix32(uint32_t x)
{
    x ^= x >> 16; x *= 0x7FEB352Du;
    x ^= x >> 15; x *= 0x846CA68Bu;
    x ^= x >> 16;
    return x;
}

enum { kStreamValue = 1, kStreamOutlier = 2, kStreamDelay = 3 };

/* The first four of the six chained mixes depend only on (seed, stream, rank, step). */
__host__ __device__ __forceinline__ uint32_t gen_prefix(uint32_t seed, uint32_t stream, uint32_t r, uint32_t t)
{
    uint32_t h = mix32(seed);
    h = mix32(h ^ stream);
    h = mix32(h + r);
    return mix32(h ^ (t * 0x9E3779B9u));
}

__host__ __device__ __forceinline__ uint32_t gen_word(uint32_t prefix, uint32_t i, uint32_t k)
{
    return mix32(mix32(prefix + i) ^ k);
}

struct Gen {
    uint32_t value_prefix;     /* (seed, value stream, rank, step)   */
    uint32_t outlier_prefix;   /* (seed, outlier stream, rank, 0)    */
    int kind;
    float scale, sigma;
    uint32_t outlier_mod;
};

__device__ __forceinline__ Gen make_gen(const sifar_workload &w, uint32_t r, uint32_t t)
{
    Gen g;
    g.value_prefix = gen_prefix(w.seed, kStreamValue, r, t);
    g.outlier_prefix = gen_prefix(w.seed, kStreamOutlier, r, 0u);
    g.kind = w.kind; g.scale = w.scale; g.sigma = w.sigma; g.outlier_mod = w.outlier_mod;
    return g;
}

__device__ __forceinline__ float gen_uniform(const Gen &g, uint32_t i)
{
    const int32_t c = (int32_t)(gen_word(g.value_prefix, i, 0u) >> 8) - (1 << 23);
    return __fmul_rn((float)c, 1.0f / 8388608.0f);
}

__device__ __forceinline__ float gen_gauss(const Gen &g, uint32_t i)
{
    int32_t s = 0;
#pragma unroll
    for (uint32_t k = 0; k < 6; ++k) {
        const uint32_t w = gen_word(g.value_prefix, i, k);
        s += (int32_t)(w & 0xFFFFu) + (int32_t)(w >> 16);
    }
    return __fmul_rn((float)(s - 393210), 1.0f / 65536.0f);
}

__device__ __forceinline__ int32_t gen_int129(const Gen &g, uint32_t i)
{
    return (int32_t)(gen_word(g.value_prefix, i, 0u) % 129u);
}

__device__ __forceinline__ uint32_t gen_delay_ns(const sifar_workload &w, uint32_t r, uint32_t t)
{
    if (w.delay_max_ns == 0u) return 0u;
    return gen_word(gen_prefix(w.seed, kStreamDelay, r, t), 0u, 0u) % (w.delay_max_ns + 1u);
}

__device__ __forceinline__ float first_value(const Gen &g, uint32_t i)
{
    if (g.kind == 1) return (float)(gen_int129(g, i) - 64);
    float z = (g.kind == 2) ? gen_uniform(g, i) : gen_gauss(g, i);
    if (g.outlier_mod != 0u && gen_word(g.outlier_prefix, i, 0u) % g.outlier_mod == 0u) z = __fmul_rn(z, 100.0f);
    return z;
}

__device__ __forceinline__ float next_value(const Gen &g, uint32_t i, float prev)
{
    if (g.kind == 1) {
        int32_t v = ((int32_t)prev + gen_int129(g, i)) % 129;
        if (v < 0) v += 129;
        return (float)(v - 64);
    }
    const float z = (g.kind == 2) ? gen_uniform(g, i) : gen_gauss(g, i);
    return __fadd_rn(__fmul_rn(prev, g.scale), __fmul_rn(z, g.sigma));
}

/*
 * A unit of a rank's partial is NW 32-bit words starting at element i0 (bf16: two
 * elements per word); elements at or past n are zero.  It is computed in two
 * halves so that the half that does not depend on the previous result can run
 * while that result is still being reduced:
 *   unit_noise()   the seeded part: the whole first partial, or sigma * z
 *                  (kinds 0, 2), or the integer k (kind 1);
 *   unit_combine() loads out^{t-1} and applies the update rule.
 * out^{t-1} is read with strong loads: inside the persistent kernel it was
 * written by another CTA of the same launch.
 */
template <int DT, int NW>
__device__ __forceinline__ void unit_noise(const Gen &g, bool first, size_t i0, size_t n,
                                           float (&z)[NW * ((DT == SIFAR_BF16) ? 2 : 1)])
{
    constexpr int NE = NW * ((DT == SIFAR_BF16) ? 2 : 1);
#pragma unroll
    for (int k = 0; k < NE; ++k) {
        const size_t i = i0 + k;
        z[k] = 0.0f;
        if (i < n) {
            if (first) z[k] = first_value(g, (uint32_t)i);
            else if (g.kind == 1) z[k] = (float)gen_int129(g, (uint32_t)i);
            else z[k] = __fmul_rn((g.kind == 2) ? gen_uniform(g, (uint32_t)i) : gen_gauss(g, (uint32_t)i), g.sigma);
        }
    }
}

__device__ __forceinline__ float apply_update(const Gen &g, bool first, float prev, float z)
{
    if (first) return z;
    if (g.kind == 1) {
        int32_t v = ((int32_t)prev + (int32_t)z) % 129;
        if (v < 0) v += 129;
        return (float)(v - 64);
    }
    return __fadd_rn(__fmul_rn(prev, g.scale), z);
}

/* The update rule applied to the NW words `pw` of the previous result (ignored when `first`). */
template <int DT, int NW>
__device__ __forceinline__ void unit_apply(const Gen &g, bool first, const uint32_t (&pw)[NW], size_t i0, size_t n,
                                           const float (&z)[NW * ((DT == SIFAR_BF16) ? 2 : 1)], uint32_t (&w)[NW])
{
#pragma unroll
    for (int j = 0; j < NW; ++j) {
        if (DT == SIFAR_BF16) {
            const size_t ia = i0 + 2 * j, ib = ia + 1;
            const float a = (ia < n) ? apply_update(g, first, bf16lo_to_f32(pw[j]), z[2 * j]) : 0.0f;
            const float b = (ib < n) ? apply_update(g, first, bf16hi_to_f32(pw[j]), z[2 * j + 1]) : 0.0f;
            w[j] = f32x2_to_bf16x2(a, b);
            if (ia >= n) w[j] = 0u;
            else if (ib >= n) w[j] &= 0xFFFFu;
        } else {
            const size_t ia = i0 + j;
            w[j] = (ia < n) ? __float_as_uint(apply_update(g, first, __uint_as_float(pw[j]), z[j])) : 0u;
        }
    }
}

template <int DT, int NW>
__device__ __forceinline__ void unit_combine(const Gen &g, bool first, const void *prev, size_t i0, size_t n,
                                             const float (&z)[NW * ((DT == SIFAR_BF16) ? 2 : 1)], uint32_t (&w)[NW],
                                             size_t n_readable = 0)
{
    constexpr int EPW = (DT == SIFAR_BF16) ? 2 : 1;
    uint32_t pw[NW];
#pragma unroll
    for (int j = 0; j < NW; ++j) pw[j] = 0u;
    /* n_readable > n: the row behind `prev` is padded, so a ragged last unit can be loaded whole */
    const bool full = (i0 + (size_t)NW * EPW <= (n_readable > n ? n_readable : n));
    if (!first) {
        if (full) {
            const uint32_t *p32 = reinterpret_cast<const uint32_t *>(prev) + i0 / EPW;
            if (NW == 4) {
                const uint4 v = ld_slot(reinterpret_cast<const uint4 *>(p32));
                pw[0] = v.x; pw[1] = v.y; pw[2] = v.z; pw[NW - 1] = v.w;
            } else {
#pragma unroll
                for (int j = 0; j < NW; ++j) pw[j] = ld_relaxed_u32(p32 + j);
            }
        } else if (DT == SIFAR_BF16) {
            /* ragged last unit: element loads, all issued before any is used (a loop that tests the bound
               between loads serialises up to six L2 round trips on the chain's critical path) */
            const uint16_t *p16 = reinterpret_cast<const uint16_t *>(prev);
            uint16_t h[NW * 2];
#pragma unroll
            for (int k = 0; k < NW * 2; ++k) h[k] = (i0 + k < n) ? ld_relaxed_u16(p16 + i0 + k) : (uint16_t)0;
#pragma unroll
            for (int k = 0; k < NW * 2; ++k) pw[k >> 1] |= (uint32_t)h[k] << ((k & 1) * 16);
        } else {
            const uint32_t *p32 = reinterpret_cast<const uint32_t *>(prev);
#pragma unroll
            for (int k = 0; k < NW; ++k) pw[k] = (i0 + k < n) ? ld_relaxed_u32(p32 + i0 + k) : 0u;
        }
    }
    unit_apply<DT, NW>(g, first, pw, i0, n, z, w);
}

template <int DT, int NW>
__device__ __forceinline__ void produce_words(const Gen &g, bool first, const void *prev, size_t i0, size_t n,
                                              uint32_t (&w)[NW])
{
    float z[NW * ((DT == SIFAR_BF16) ? 2 : 1)];
    unit_noise<DT, NW>(g, first, i0, n, z);
    unit_combine<DT, NW>(g, first, prev, i0, n, z, w);
}

/* Busy-wait `ns` nanoseconds on the global timer (ns is small and bounded by the caller). */
__device__ __forceinline__ void spin_ns(uint32_t ns)
{
    if (ns == 0u) return;
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < (unsigned long long)ns) { }
}

}  /* namespace sifar */
#endif
