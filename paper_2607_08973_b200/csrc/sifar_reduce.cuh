/*
 * Device-side pieces shared by the discrete reducer kernels and by the
 * persistent decode-step chain: bounded flag waits, rank-order accumulation,
 * slot validation with retry, masked result stores.
 */
#ifndef SIFAR_REDUCE_CUH
#define SIFAR_REDUCE_CUH

#include "sifar_internal.cuh"

namespace sifar {

/* ------------------------------------------------------------------------ */
/* bounded waits                                                             */
/* ------------------------------------------------------------------------ */

/*
 * Time limit of a polling loop.  The clock (%globaltimer) is read on every
 * kPollsPerClockCheck-th failed poll only: reading it on every poll measurably
 * slows the poll loops of the persistent chain.  A poll costs at least one L2
 * round trip (~0.3 us), so a limit is overshot by a few microseconds at most.
 */
constexpr unsigned kPollsPerClockCheck = 8;
constexpr unsigned kPollStaggerNs = 120;         /* spacing of the polls a waiting lane keeps in flight */

struct Deadline {
    unsigned long long t0 = 0;
    unsigned polls = 0;
    /* Call after a failed poll; true once the limit has passed. */
    __device__ __forceinline__ bool expired(unsigned long long timeout_ns)
    {
        if ((++polls % kPollsPerClockCheck) != 1u) return false;
        const unsigned long long now = globaltimer_ns();
        if (t0 == 0) { t0 = now; return false; }
        return now - t0 > timeout_ns;
    }
};

/* Bounded poll of a flag until it equals `want` (acquire).  Returns the number of failed polls, or -1 on time-out. */
__device__ __forceinline__ int wait_flag_eq(const uint32_t *flag, uint32_t want, unsigned long long timeout_ns)
{
    Deadline d;
    while (ld_acquire_u32(flag) != want)
        if (d.expired(timeout_ns)) return -1;
    return (int)d.polls;
}

/* Same until the flag has reached `base` (call numbers never wrap inside a context's life). */
__device__ __forceinline__ int wait_flag_ge(const uint32_t *flag, uint32_t base, unsigned long long timeout_ns)
{
    Deadline d;
    while (ld_acquire_u32(flag) < base)
        if (d.expired(timeout_ns)) return -1;
    return (int)d.polls;
}

/*
 * Bounded acquire wait of the persistent kernels: until the flag equals (or, GE, has reached) `want`.  Records
 * SIFAR_ERR_TIMEOUT when the limit passes, and also gives up when another CTA has already recorded a failure.
 */
template <bool GE>
__device__ __forceinline__ bool wait_flag_or_fail(const uint32_t *flag, uint32_t want, DevState *st, int *host_status,
                                                  unsigned long long timeout_ns)
{
    Deadline d;
    for (;;) {
        const uint32_t v = ld_acquire_u32(flag);
        if (GE ? (v >= want) : (v == want)) return true;
        if (d.expired(timeout_ns)) { fail(st, host_status, SIFAR_ERR_TIMEOUT); return false; }
        if ((d.polls % 64u) == 0u && ld_relaxed_u32(&st->status) != 0u) return false;
    }
}

/* ------------------------------------------------------------------------ */
/* rank-order accumulation                                                   */
/* ------------------------------------------------------------------------ */
template <int DT, int P>
__device__ __forceinline__ uint32_t sum_word(const uint32_t (&w)[P])
{
    if (DT == SIFAR_BF16) {
        float lo = bf16lo_to_f32(w[0]), hi = bf16hi_to_f32(w[0]);
#pragma unroll
        for (int r = 1; r < P; ++r) {
            lo = __fadd_rn(lo, bf16lo_to_f32(w[r]));
            hi = __fadd_rn(hi, bf16hi_to_f32(w[r]));
        }
        return f32x2_to_bf16x2(lo, hi);
    } else {
        float acc = __uint_as_float(w[0]);
#pragma unroll
        for (int r = 1; r < P; ++r) acc = __fadd_rn(acc, __uint_as_float(w[r]));
        return __float_as_uint(acc);
    }
}

template <int DT, int P>
__device__ __forceinline__ uint4 sum_vec(const uint4 (&x)[P], bool with_w)
{
    uint32_t a[P], b[P], c[P], d[P];
#pragma unroll
    for (int r = 0; r < P; ++r) { a[r] = x[r].x; b[r] = x[r].y; c[r] = x[r].z; d[r] = x[r].w; }
    uint4 o;
    o.x = sum_word<DT, P>(a);
    o.y = sum_word<DT, P>(b);
    o.z = sum_word<DT, P>(c);
    o.w = with_w ? sum_word<DT, P>(d) : 0u;
    return o;
}

/* The data words of P slot images, summed in rank order: word j of the result in .x, .y (, .z). */
template <int DT, int P>
__device__ __forceinline__ uint4 sum_slot(const uint4 (&x)[P])
{
    uint32_t o[3] = {0u, 0u, 0u};
#pragma unroll
    for (int j = 0; j < kSlotDataWords; ++j) {
        uint32_t a[P];
#pragma unroll
        for (int r = 0; r < P; ++r) a[r] = slot_word(x[r], j);
        o[j] = sum_word<DT, P>(a);
    }
    return make_uint4(o[0], o[1], o[2], 0u);
}

/* Vectors (plain) or slots (speculative) a thread keeps in flight per rank. */
template <int P> struct Unroll { static constexpr int value = (P <= 2) ? 4 : (P <= 4) ? 2 : 1; };

/* ------------------------------------------------------------------------ */
/* slot validation (speculative mode)                                        */
/* ------------------------------------------------------------------------ */
/*
 * x[r] holds rank r's slot `s` as first loaded.  A slot counts iff its tag equals
 * the call number e (Section 4.2: validation after the speculative read).  On
 * mis-speculation only the stale ranks of this slot are loaded again until
 * every tag matches or the time limit passes.  Returns false on time-out.
 * `reloads` counts the extra loads.
 *
 * Polling shapes (WIDE, pace_ns):
 *   wide    every stale rank is re-loaded each round: the last arrival is seen one
 *           L2 round trip later, at up to P loads per waiting thread and round.
 *   narrow  only the lowest stale rank is polled; when it turns valid one wide
 *           round follows.  One more round trip after the last arrival, 1/P of
 *           the polling traffic.
 *   pace_ns sleep between rounds.
 * A large waiting grid that polls wide and unpaced takes L2 bandwidth away from
 * the very producers it waits for; the host picks the shape from the grid size.
 */
template <int P, bool WIDE>
__device__ __forceinline__ bool revalidate(uint4 (&x)[P], uint32_t stale, const uint4 *const *src, size_t s,
                                           uint32_t e, unsigned long long timeout_ns, uint32_t pace_ns,
                                           unsigned &reloads, unsigned long long *round_stamps = nullptr)
{
    Deadline d;
    bool burst = WIDE;
    unsigned round = 0;
    do {
        /* issue every pending load before looking at any result, so that the re-loads overlap */
        const uint32_t pending = (WIDE || burst) ? stale : (stale & (0u - stale));
#pragma unroll
        for (int r = 0; r < P; ++r)
            if (pending & (1u << r)) x[r] = ld_slot(src[r] + s);
        const uint32_t before = stale;
#pragma unroll
        for (int r = 0; r < P; ++r)
            if ((pending & (1u << r)) && slot_valid(x[r], e)) stale &= ~(1u << r);
        reloads += __popc(pending);
        if (!WIDE) burst = !burst && stale != before;    /* the polled rank arrived: look at all others once */
        if (round_stamps && round < 8u) round_stamps[round] = globaltimer_ns();
        ++round;
        if (stale) {
            if (d.expired(timeout_ns)) return false;
            if (pace_ns) __nanosleep(pace_ns);
        }
    } while (stale);
    return true;
}

struct PollShape {
    uint32_t wide;
    uint32_t pace_ns;
    uint32_t sentinel;     /* wait on one slot per rank and warp before touching the warp's other slots */
    uint32_t forced;       /* measurement knob: re-load every slot this many times although it may be valid */
};

/*
 * Sentinel wait of a warp (all 32 lanes call): lane r < P polls rank r's copy of the warp's first slot
 * until it carries the call number; the other lanes idle.  A producer warp writes 32 consecutive slots
 * with one store instruction, so once the first is visible the rest follow within the same few hundred
 * nanoseconds, and the warp's 32 x P bulk loads can go out and will almost always validate at once.
 * Compared with every lane polling its own P slots this costs one extra L2 round trip after the last
 * arrival, but it keeps 31/32 of the lines free of poll traffic while the producers are storing into
 * them, which is what large waiting grids need.  Returns false on time-out (any lane).
 */
template <int P>
__device__ __forceinline__ bool sentinel_wait(const uint4 *const *src, size_t warp_first_slot, uint32_t e,
                                              unsigned long long timeout_ns, unsigned &reloads)
{
    const unsigned lane = threadIdx.x & 31u;
    bool ok = true;
    if (lane < (unsigned)P) {
        const uint4 *p = nullptr;
#pragma unroll
        for (int r = 0; r < P; ++r)
            if (lane == (unsigned)r) p = src[r] + warp_first_slot;
        /* Three polls in flight, issued a third of a round trip apart: a poll loop that waits for each answer
           before it asks again sees an arrival up to a whole round trip late, and in a chain whose steps all
           look alike that delay does not average out (the same code was 0.6 us per step faster or slower
           depending on where its polls happened to fall). */
        Deadline d;
        uint4 v0 = ld_slot(p);
        if (!slot_valid(v0, e)) {                     /* already there (a thread's later units usually are): one look */
        v0 = ld_slot(p);
        __nanosleep(kPollStaggerNs);
        uint4 v1 = ld_slot(p);
        __nanosleep(kPollStaggerNs);
        uint4 v2 = ld_slot(p);
        ++reloads;
        for (;;) {
            if (slot_valid(v0, e)) break;
            v0 = ld_slot(p);
            if (slot_valid(v1, e)) break;
            v1 = ld_slot(p);
            if (slot_valid(v2, e)) break;
            v2 = ld_slot(p);
            reloads += 3;
            if (d.expired(timeout_ns)) { ok = false; break; }
        }
        }
    }
    return __all_sync(0xFFFFFFFFu, ok);
}

template <int P>
__device__ __forceinline__ bool validate_once(uint4 (&x)[P], const uint4 *const *src, size_t s, uint32_t e,
                                              unsigned long long timeout_ns, PollShape shape, unsigned &reloads,
                                              unsigned long long *round_stamps)
{
    uint32_t stale = 0;
#pragma unroll
    for (int r = 0; r < P; ++r) stale |= (uint32_t)(!slot_valid(x[r], e)) << r;
    if (stale == 0u) return true;
    return shape.wide ? revalidate<P, true>(x, stale, src, s, e, timeout_ns, shape.pace_ns, reloads, round_stamps)
                      : revalidate<P, false>(x, stale, src, s, e, timeout_ns, shape.pace_ns, reloads, round_stamps);
}

template <int P>
__device__ __forceinline__ bool validate_slot(uint4 (&x)[P], const uint4 *const *src, size_t s, uint32_t e,
                                              unsigned long long timeout_ns, PollShape shape, unsigned &reloads,
                                              unsigned long long *round_stamps = nullptr)
{
    if (!validate_once<P>(x, src, s, e, timeout_ns, shape, reloads, round_stamps)) return false;
    if (shape.forced == 0u) return true;
    /* Forced retries (the retry-latency experiment of Section 6.3, "Retry Overhead"): the attempt that found
       every copy valid is treated as mis-speculated, `forced` times: each round loads all P copies again.
       The address of a round depends on the previous round's tags through a zero the compiler cannot see,
       so the rounds run one after another as real retries do.  The last copies are validated as usual
       (a valid slot stays valid until its producer's store for call e + 2, which waits for this result). */
    for (uint32_t k = 0; k < shape.forced; ++k) {
        uint32_t dep = 0;
#pragma unroll
        for (int r = 0; r < P; ++r) dep |= x[r].w;
        asm volatile("and.b32 %0, %0, 0;" : "+r"(dep));
#pragma unroll
        for (int r = 0; r < P; ++r) x[r] = ld_slot(src[r] + s + dep);
        reloads += P;
    }
    return validate_once<P>(x, src, s, e, timeout_ns, shape, reloads, nullptr);
}

/* ------------------------------------------------------------------------ */
/* result stores                                                             */
/* ------------------------------------------------------------------------ */
/* The data bytes of reduced slot s go to elements [s*EPS, s*EPS+EPS) of out; a short last slot is masked. */
template <int DT>
__device__ __forceinline__ void store_slot_result(void *out, size_t s, size_t n, const uint4 &o)
{
    constexpr int EPS = kSlotDataWords * ((DT == SIFAR_BF16) ? 2 : 1);
    const size_t i0 = s * EPS;
    if (i0 + EPS <= n) {
        uint32_t *dst = reinterpret_cast<uint32_t *>(out) + s * kSlotDataWords;
        dst[0] = o.x; dst[1] = o.y;
        if (kSlotDataWords == 3) dst[2] = o.z;
    } else if (DT == SIFAR_BF16) {
        uint16_t *dst = reinterpret_cast<uint16_t *>(out) + i0;
        const uint32_t w[3] = {o.x, o.y, o.z};
        for (int k = 0; k < EPS && i0 + k < n; ++k)
            dst[k] = (uint16_t)((w[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu);
    } else {
        uint32_t *dst = reinterpret_cast<uint32_t *>(out) + i0;
        const uint32_t w[3] = {o.x, o.y, o.z};
        for (int k = 0; k < EPS && i0 + k < n; ++k) dst[k] = w[k];
    }
}

/* Reduced 16-byte vector v goes to elements [v*EPV, v*EPV+EPV) of out; a short last vector is masked. */
template <int DT>
__device__ __forceinline__ void store_vec_result(void *out, size_t v, size_t n, const uint4 &o)
{
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
    const size_t i0 = v * EPV;
    if (i0 + EPV <= n) {
        reinterpret_cast<uint4 *>(out)[v] = o;
    } else if (DT == SIFAR_BF16) {
        uint16_t *dst = reinterpret_cast<uint16_t *>(out) + i0;
        const uint32_t w[4] = {o.x, o.y, o.z, o.w};
        for (int k = 0; k < EPV && i0 + k < n; ++k)
            dst[k] = (uint16_t)((w[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu);
    } else {
        uint32_t *dst = reinterpret_cast<uint32_t *>(out) + i0;
        const uint32_t w[4] = {o.x, o.y, o.z, o.w};
        for (int k = 0; k < EPV && i0 + k < n; ++k) dst[k] = w[k];
    }
}

}  /* namespace sifar */
#endif
