/*
 * sifar_device.cuh - device-side building blocks of the producer store path and
 * of the reducer, header-only, for kernels that want to store their partial
 * directly (a fused producer) instead of going through sifar_pack().
 *
 * Memory-model notes.  Ranks and reducer talk only through global memory of one
 * GPU, so every access below is a STRONG access at .gpu scope (never a plain
 * cached load: a kernel that outlives its producers must not read a stale L1
 * line; the paper meets the same issue and bypasses L1 on retry, Section 4.2
 * "Verification Logic Correctness").
 *
 *  - A slot is 16 aligned bytes {w0, w1, w2, tag}.  It is written and read with
 *    ONE scalar 128-bit access (.b128), so data and tag arrive together: a slot
 *    whose tag equals the current call number carries that call's data, without
 *    any fence and without the ordering assumption between payload and flag that
 *    the paper's separate validation buffer needs (Section 8.1).
 *  - Arrival / done flags follow release -> acquire: all stores of the CTA, then
 *    bar.sync, then one thread publishes with st.release.gpu; the reader polls
 *    with ld.acquire.gpu, then bar.sync, then reads the payload.
 */
#ifndef SIFAR_DEVICE_CUH
#define SIFAR_DEVICE_CUH

#include <cuda_runtime.h>
#include <stdint.h>

namespace sifar {

__device__ __forceinline__ uint4 ld_slot(const uint4 *p)
{
    uint4 v;
    asm volatile("{\n\t.reg .b128 q;\n\tld.relaxed.gpu.global.b128 q, [%4];\n\tmov.b128 {%0, %1, %2, %3}, q;\n\t}"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint4 ld_slot_acquire(const uint4 *p)
{
    uint4 v;
    asm volatile("{\n\t.reg .b128 q;\n\tld.acquire.gpu.global.b128 q, [%4];\n\tmov.b128 {%0, %1, %2, %3}, q;\n\t}"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_slot(uint4 *p, uint4 v)
{
    asm volatile("{\n\t.reg .b128 q;\n\tmov.b128 q, {%0, %1, %2, %3};\n\tst.relaxed.gpu.global.b128 [%4], q;\n\t}"
                 :: "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(p) : "memory");
}

__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint16_t ld_relaxed_u16(const uint16_t *p)
{
    uint16_t v;
    asm volatile("ld.relaxed.gpu.global.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint2 ld_relaxed_u32x2(const void *p)
{
    uint2 v;
    asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ void st_relaxed_u32(uint32_t *p, uint32_t v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ uint32_t atom_add_acq_rel_u32(uint32_t *p, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

__device__ __forceinline__ uint32_t atom_add_relaxed_u32(uint32_t *p, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.relaxed.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

/* Fire-and-forget increment: the issuing thread does not wait for the result. */
__device__ __forceinline__ void red_add_relaxed_u32(uint32_t *p, uint32_t v)
{
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

/* One tagged slot: three data words and the call number, in one 16-byte store. */
__device__ __forceinline__ void store_slot(uint4 *slots, size_t i, uint32_t w0, uint32_t w1,
                                           uint32_t w2, uint32_t tag)
{
    st_slot(slots + i, make_uint4(w0, w1, w2, tag));
}

/*
 * Arrival of one rank in the barrier modes.  Every thread of every CTA that
 * stored part of the rank's partial calls this after its last store.  `counter`
 * counts the CTAs of the rank that are done; the last one re-arms it and
 * releases the flag.  `nctas` = number of CTAs that call this for the rank.
 */
__device__ __forceinline__ void signal_arrival(uint32_t *counter, uint32_t nctas, uint32_t *flag,
                                               uint32_t epoch)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t done = (nctas > 1) ? atom_add_acq_rel_u32(counter, 1u) + 1u : 1u;
        if (done == nctas) {
            if (nctas > 1) st_relaxed_u32(counter, 0u);
            st_release_u32(flag, epoch);
        }
    }
}

/*
 * Arrival of one block of the flagged-tile format (speculative mode, large payloads; see
 * sifar_spec_format() and sifar_tile_flags()).  Every thread of the CTA that stored the block calls this
 * after its last store of the block; one thread releases the block's flag.
 */
__device__ __forceinline__ void signal_block(uint32_t *flags, size_t stride_words, size_t block, uint32_t epoch)
{
    __syncthreads();
    if (threadIdx.x == 0) st_release_u32(flags + block * stride_words, epoch);
}

/* bf16 pair <-> binary32 (the low half of a word is the element with the lower index). */
__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

/* Two binary32 -> packed bf16x2, each rounded to nearest even (NaN -> 0x7FFF). */
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi)
{
    uint32_t w;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(hi), "f"(lo));
    return w;
}

__device__ __forceinline__ uint16_t f32_to_bf16(float f)
{
    return (uint16_t)(f32x2_to_bf16x2(f, 0.0f) & 0xFFFFu);
}

}  /* namespace sifar */
#endif /* SIFAR_DEVICE_CUH */
