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

/*
 * Slot format.  Default ("S12"): {w0, w1, w2, tag}, written and read with one 16-byte access; a slot counts
 * iff its tag is the call number.  Fallback, compiled with -DSIFAR_SLOT_S8X2: two halves {w0, tag} and
 * {w1, tag}, each written with one 8-byte store and valid on its own, so that only 64-bit single-copy
 * atomicity is relied on (the memory model's scalar guarantee); 8 data bytes per 16-byte slot instead of 12.
 * Should the 16-byte check (sifar_tear_check) ever report a torn slot, this is the layout to build.
 */
#ifdef SIFAR_SLOT_S8X2
constexpr int kSlotDataWords = 2;
#else
constexpr int kSlotDataWords = 3;
#endif

/* Does the slot image carry call number `tag` (in the fallback format: both of its halves)? */
__device__ __forceinline__ bool slot_valid(const uint4 &v, uint32_t tag)
{
#ifdef SIFAR_SLOT_S8X2
    return v.y == tag && v.w == tag;
#else
    return v.w == tag;
#endif
}

/* Data word j (0 .. kSlotDataWords - 1) of a slot image. */
__device__ __forceinline__ uint32_t slot_word(const uint4 &v, int j)
{
#ifdef SIFAR_SLOT_S8X2
    return j == 0 ? v.x : v.z;
#else
    return j == 0 ? v.x : j == 1 ? v.y : v.z;
#endif
}

/* One tagged slot: kSlotDataWords data words and the call number. */
__device__ __forceinline__ void store_slot_words(uint4 *slots, size_t i, const uint32_t (&w)[kSlotDataWords], uint32_t tag)
{
#ifdef SIFAR_SLOT_S8X2
    uint32_t *p = reinterpret_cast<uint32_t *>(slots + i);
    asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" :: "l"(p), "r"(w[0]), "r"(tag) : "memory");
    asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" :: "l"(p + 2), "r"(w[1]), "r"(tag) : "memory");
#else
    st_slot(slots + i, make_uint4(w[0], w[1], w[2], tag));
#endif
}

#ifndef SIFAR_SLOT_S8X2
/* The default format spelled out: three data words and the call number, in one 16-byte store. */
__device__ __forceinline__ void store_slot(uint4 *slots, size_t i, uint32_t w0, uint32_t w1,
                                           uint32_t w2, uint32_t tag)
{
    st_slot(slots + i, make_uint4(w0, w1, w2, tag));
}
#endif

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
