/*
 * sifar_symmetric.cu - the decode-step chain with P readers: every emulated rank
 * runs its own operation AND its own pull-and-reduce, as every GPU of the paper's
 * system does (Section 3.1: each GPU pulls all peers' partials and reduces them
 * locally; Listing of Section 4.2).
 *
 * One cooperative kernel of P x C CTAs.  CTA (r, c) is rank r's share c of the
 * machine: in every step it
 *   1. computes chunk c of rank r's next partial from chunk c of ITS OWN copy of the
 *      previous result (registers: the same threads reduced it a moment ago),
 *   2. stores it into rank r's buffer (tagged slots, or plain data + arrival flag),
 *   3. pulls chunk c of all P partials, its own included, and reduces it in rank
 *      order into rank r's copy of the result.
 * Nothing orders a rank behind another rank except the mode's own protocol:
 *   BARRIER_ONESHOT : [wait until all P readers are done with the single buffer]
 *                     store, arrival flag; wait for P arrival flags; load, sum;
 *                     done flag                      (top and bottom barrier, P x P flags)
 *   DUALBUF         : store into parity buffer, arrival flag; wait for P flags; load, sum
 *   SPECULATIVE     : store tagged slots; load all P copies at once, accept a slot iff
 *                     its tag is this call's number, re-load the stale ones
 *   TWOSHOT         : the paper's other baseline (Section 3.1): store, arrival flag; wait for P flags;
 *                     reduce 1/P of the chunk for everybody (reduce-scatter); second barrier; read the
 *                     whole reduced chunk (all-gather).  The second barrier also covers the reuse of the
 *                     single buffer: a rank passes it only after every rank's reads of the partials.
 *   FLAGVAL         : the paper's own validation scheme (Section 4.2, "Speculative Reduction" and
 *                     "Verification Logic Correctness"): plain payload, one validation flag per threadblock
 *                     written after the payload, one extra warp that pulls the P flags while the other
 *                     warps pull the payload, success iff the flags sum to P x flag, else the whole
 *                     threadblock runs again; the flag buffer is dual-buffered like the payload (k_symv).
 *   FLAGVAL_ORDERED : the same objects, but the payload is pulled only after the extra warp has seen all P
 *                     flags (acquire): the ordering that is sound on one GPU without any assumption.
 * so ranks drift against each other as real GPUs do, and a rank mis-speculates
 * exactly when a peer is behind it.  A thread keeps the same units in every step;
 * the speculative mode needs no CTA-wide barrier at all: the write-after-read
 * safety of the two parity buffers holds per thread (a thread overwrites a slot for
 * call e + 2 only after it has validated call e + 1 of every rank, whose threads
 * had finished reading call e before they stored call e + 1).
 * All P copies of every result are bit-identical and equal to the one-reader chains'.
 */
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "sifar_internal.cuh"
#ifdef SIFAR_SLOT_S8X2
#error "the decode-step chains are written for the default slot format; the fallback format is built for libsifar only"
#endif
#include "sifar_reduce.cuh"
#include "sifar_gen.cuh"
#include "sifar_workload.h"

namespace sifar {

constexpr int kSymThreads = 128;
constexpr int kSymNoAllreduce = SIFAR_CHAIN_NO_ALLREDUCE;
constexpr int kSymTwoshot = SIFAR_SYMCHAIN_TWOSHOT;
constexpr int kSymFlagval = SIFAR_SYMCHAIN_FLAGVAL;
constexpr int kSymFlagvalOrdered = SIFAR_SYMCHAIN_FLAGVAL_ORDERED;
constexpr int kSymUnchecked = SIFAR_SYMCHAIN_UNCHECKED;
constexpr int kSymvThreads = kSymThreads + 32;       /* the payload warps and one validation warp */

/* Flags of one chunk: what the P CTAs that own it tell each other. */
struct __align__(128) SymFlags {
    uint32_t arrive[2][8];          /* [parity][rank]: chunk of the rank's partial of call e stored      */
    uint32_t pad0[16];
    uint32_t done[8];               /* [rank]: the rank's reader has finished reading the chunk of call e */
    uint32_t pad1[24];
};

struct __align__(128) SymDev {
    uint32_t exit_count;            /* CTAs that left the kernel (monotonic over runs) */
    uint32_t pad[31];
};

struct SymArgs {
    DevState *st;
    int *host_status;
    unsigned long long timeout_ns;
    sifar_workload w;
    unsigned long long n;
    char *plain;                    /* [parity][rank] plain buffers */
    unsigned long long plain_stride;
    char *slots;                    /* [parity][rank] slot buffers  */
    unsigned long long slot_stride;
    char *rings;                    /* [rank][ring_len] result rows */
    unsigned long long ring_stride;
    uint32_t ring_len;
    uint32_t e0;                    /* calls completed before this run */
    uint32_t base_epoch;
    uint32_t steps;
    uint32_t C, K;
    uint32_t exit_base;
    PollShape poll;
    SymDev *cs;
    SymFlags *flags;                /* C */
    unsigned long long *stamps;     /* [rank][chunk][warp][steps + 1] */
    uint32_t *retry_marks;          /* [rank][steps]: 1 if the rank re-loaded a slot in that step */
    unsigned long long *rank_retries; /* [P] cumulative (rank, step) pairs with a re-load */
};

template <int DT, int P, int MODE>
__global__ void __launch_bounds__(kSymThreads, 6) k_sym(const SymArgs a)
{
    DevState *st = a.st;
    constexpr bool no_ar = (MODE == kSymNoAllreduce);
    constexpr bool spec = (MODE == SIFAR_SPECULATIVE);
    constexpr bool two = (MODE == kSymTwoshot);
    constexpr bool single = (MODE == SIFAR_BARRIER_ONESHOT || two);      /* one buffer per rank instead of two */
    constexpr int NW = spec ? 3 : 4;                                  /* words per unit */
    constexpr int NE = NW * ((DT == SIFAR_BF16) ? 2 : 1);             /* elements per unit */
    const uint32_t rank = blockIdx.x % (uint32_t)P;                   /* the P CTAs of a chunk are neighbours (one cluster) */
    const uint32_t chunk = blockIdx.x / (uint32_t)P;
    SymFlags *cf = a.flags + chunk;
    const size_t n = (size_t)a.n;
    /* whole warps of units (a partly filled warp was measured to slow its chunk down); units past the last
       element carry zeros, and the rank buffers and result rows have room for them */
    const size_t nunits = ((n + NE - 1) / NE + 31) / 32 * 32;
    const size_t n_io = nunits * NE;                                  /* result rows are padded to whole units */
    const size_t unit0 = (size_t)chunk * kSymThreads * a.K + threadIdx.x;
    char *my_ring = a.rings + (size_t)rank * a.ring_len * a.ring_stride;
    /* Stamps per warp: without a CTA-wide barrier (speculative mode has none) the warps of a CTA are pipelines
       of their own, and a chunk of a result is complete when the last of them is; the host takes the maximum. */
    constexpr uint32_t kWarps = kSymThreads / 32;
    const bool stamper = (threadIdx.x & 31u) == 0u;
    unsigned long long *my_stamps = a.stamps + (((size_t)rank * a.C + chunk) * kWarps + (threadIdx.x >> 5)) * (a.steps + 1u);
    __shared__ int s_ok;
    unsigned reloads = 0;
    bool alive = true;
    uint32_t prevw[NW];                                               /* this thread's first unit of the previous result */
#pragma unroll
    for (int j = 0; j < NW; ++j) prevw[j] = 0u;
    if (stamper) my_stamps[0] = globaltimer_ns();

    for (uint32_t s = 0; s < a.steps && alive; ++s) {
        const uint32_t e = a.e0 + 1u + s;
        const uint32_t t = e - a.base_epoch;
        const uint32_t p = e & 1u;
        const bool first = (t == 1u);
        const Gen g = make_gen(a.w, rank, t);
        char *row = my_ring + (size_t)((t - 1u) % a.ring_len) * a.ring_stride;
        /* where the previous result (without all-reduce: the rank's previous partial) lies in memory */
        const char *prev_mem = no_ar ? a.plain + ((size_t)(p ^ 1u) * P + rank) * a.plain_stride
                                     : my_ring + (size_t)((t + a.ring_len - 2u) % a.ring_len) * a.ring_stride;
        uint4 *dst = spec ? reinterpret_cast<uint4 *>(a.slots + ((size_t)p * P + rank) * a.slot_stride)
                          : reinterpret_cast<uint4 *>(a.plain + ((size_t)(single ? 0u : p) * P + rank) * a.plain_stride);

        /* ---- 1. the rank's next operation: the seeded half first, it needs nothing from anybody ---- */
        float z0[NE];
        if (unit0 < nunits) unit_noise<DT, NW>(g, first, unit0 * NE, n, z0);
        if (MODE == SIFAR_BARRIER_ONESHOT || a.w.delay_max_ns != 0u) {
            if (threadIdx.x < 32) {
                bool ok = true;
                /* bottom barrier, writer side: all P readers are done with the single buffer (Section 3.1, phase 3) */
                if (MODE == SIFAR_BARRIER_ONESHOT && !first && threadIdx.x < P)
                    ok = wait_flag_or_fail<true>(&cf->done[threadIdx.x], e - 1u, st, a.host_status, a.timeout_ns);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (threadIdx.x == 0) {
                    if (ok) spin_ns(gen_delay_ns(a.w, rank, t));          /* seeded skew between the ranks */
                    s_ok = ok;
                }
            }
            __syncthreads();
            if (!s_ok) { alive = false; break; }
        }
        /* ---- 2. store the partial ---- */
        for (uint32_t k = 0; k < a.K; ++k) {
            const size_t u = unit0 + (size_t)k * kSymThreads;
            if (u >= nunits) break;
            uint32_t w[NW];
            if (k == 0 && s > 0u) {
                unit_apply<DT, NW>(g, first, prevw, u * NE, n, z0, w);
            } else if (k == 0) {
                unit_combine<DT, NW>(g, first, prev_mem, u * NE, n, z0, w, n_io);
            } else {
                float z[NE];
                unit_noise<DT, NW>(g, first, u * NE, n, z);
                unit_combine<DT, NW>(g, first, prev_mem, u * NE, n, z, w, n_io);
            }
            if (spec) store_slot(dst, u, w[0], w[1], w[2], e);
            else st_slot(dst + u, make_uint4(w[0], w[1], w[2], w[NW - 1]));
            if (no_ar && k == 0) {
#pragma unroll
                for (int j = 0; j < NW; ++j) prevw[j] = w[j];
            }
        }
        if constexpr (no_ar) {
            __syncthreads();
            if (stamper) my_stamps[s + 1u] = globaltimer_ns();
        } else {
        const uint4 *src[P];
#pragma unroll
        for (int r = 0; r < P; ++r)
            src[r] = spec ? reinterpret_cast<const uint4 *>(a.slots + ((size_t)p * P + r) * a.slot_stride)
                          : reinterpret_cast<const uint4 *>(a.plain + ((size_t)(single ? 0u : p) * P + r) * a.plain_stride);
        if (!spec) {
            /* arrival flag of this rank (release), then the top barrier: all P ranks' flags (acquire) */
            __syncthreads();
            if (threadIdx.x == 0) st_release_u32(&cf->arrive[p][rank], e);
            if (threadIdx.x < 32) {
                bool ok = true;
                if (threadIdx.x < P)
                    ok = wait_flag_or_fail<false>(&cf->arrive[p][threadIdx.x], e, st, a.host_status, a.timeout_ns);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (threadIdx.x == 0) s_ok = ok;
            }
            __syncthreads();
            if (!s_ok) { alive = false; break; }
        }
        if constexpr (two) {
            /* ---- 3a. reduce-scatter: this rank reduces its share of the chunk's units for everybody ---- */
            uint4 *red = reinterpret_cast<uint4 *>(a.plain + (size_t)P * a.plain_stride);   /* parity 1, rank 0: unused here */
            const bool mine = (threadIdx.x * (uint32_t)P / kSymThreads == rank);
            for (uint32_t k = 0; k < a.K; ++k) {
                const size_t u = unit0 + (size_t)k * kSymThreads;
                if (u >= nunits) break;
                if (mine) {
                    uint4 x[P];
#pragma unroll
                    for (int r = 0; r < P; ++r) x[r] = ld_slot(src[r] + u);
                    st_slot(red + u, sum_vec<DT, P>(x, true));
                }
            }
            /* second barrier: all P shares of the chunk are reduced (the done flags serve as its arrival flags) */
            __syncthreads();
            if (threadIdx.x == 0) st_release_u32(&cf->done[rank], e);
            if (threadIdx.x < 32) {
                bool ok = true;
                if (threadIdx.x < P)
                    ok = wait_flag_or_fail<false>(&cf->done[threadIdx.x], e, st, a.host_status, a.timeout_ns);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (threadIdx.x == 0) s_ok = ok;
            }
            __syncthreads();
            if (!s_ok) { alive = false; break; }
            /* ---- 3b. all-gather: every rank takes the whole reduced chunk ---- */
            for (uint32_t k = 0; k < a.K; ++k) {
                const size_t u = unit0 + (size_t)k * kSymThreads;
                if (u >= nunits) break;
                const uint4 o = ld_slot(red + u);
                store_vec_result<DT>(row, u, n_io, o);
                if (k == 0) { prevw[0] = o.x; prevw[1] = o.y; prevw[2] = o.z; prevw[NW - 1] = o.w; }
            }
        } else {
        /* ---- 3. pull all P partials and reduce in rank order ---- */
        bool retried = false;
        for (uint32_t k = 0; k < a.K; ++k) {
            const size_t u = unit0 + (size_t)k * kSymThreads;
            if (u >= nunits) break;
            uint4 x[P];
#pragma unroll
            for (int r = 0; r < P; ++r) x[r] = ld_slot(src[r] + u);
            uint4 o;
            if (spec) {
                const unsigned before = reloads;
                if (!validate_slot<P>(x, src, u, e, a.timeout_ns, a.poll, reloads)) {
                    fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
                    alive = false;
                    break;
                }
                retried |= (reloads != before);
                o = sum_vec<DT, P>(x, false);
                store_slot_result<DT>(row, u, n_io, o);
            } else {
                o = sum_vec<DT, P>(x, true);
                store_vec_result<DT>(row, u, n_io, o);
            }
            if (k == 0) { prevw[0] = o.x; prevw[1] = o.y; prevw[2] = o.z; prevw[NW - 1] = spec ? o.z : o.w; }
        }
        if (spec) {
            /* a rank mis-speculated in this step if any of its threads had to load a slot again */
            if (__any_sync(0xFFFFFFFFu, retried) && (threadIdx.x & 31) == 0)
                st_relaxed_u32(&a.retry_marks[(size_t)rank * a.steps + s], 1u);
            if (!__all_sync(0xFFFFFFFFu, alive)) alive = false;
        }
        if (MODE == SIFAR_BARRIER_ONESHOT) {
            /* bottom barrier, reader side: this rank's loads of the chunk have returned */
            __syncthreads();
            if (threadIdx.x == 0) st_release_u32(&cf->done[rank], e);
        }
        }   /* !two */
        if (stamper) my_stamps[s + 1u] = globaltimer_ns();
        }   /* !no_ar */
    }

    /* leave: statistics, then the last CTA out books the run and publishes the call number */
    const unsigned warp_reloads = __reduce_add_sync(0xFFFFFFFFu, reloads);
    if (warp_reloads && (threadIdx.x & 31) == 0)
        atomicAdd(&st->stats[kStatSlotReloads], (unsigned long long)warp_reloads);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const uint32_t left = atom_add_acq_rel_u32(&a.cs->exit_count, 1u) + 1u;
        s_ok = (left == a.exit_base + gridDim.x && !no_ar && ld_relaxed_u32(&st->status) == 0u);
    }
    __syncthreads();
    if (s_ok) {
        if (spec) {
            unsigned long long any_steps = 0;
            for (uint32_t s = threadIdx.x; s < a.steps; s += kSymThreads) {
                uint32_t any = 0;
                for (int r = 0; r < P; ++r) {
                    const uint32_t m = ld_relaxed_u32(&a.retry_marks[(size_t)r * a.steps + s]);
                    if (m) {
                        atomicAdd(&a.rank_retries[r], 1ull);
                        st_relaxed_u32(&a.retry_marks[(size_t)r * a.steps + s], 0u);
                    }
                    any |= m;
                }
                any_steps += any ? 1ull : 0ull;
            }
            if (any_steps) atomicAdd(&st->stats[kStatCallsWithRetry], any_steps);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            atomicAdd(&st->stats[kStatCalls], (unsigned long long)a.steps);
            st_release_u32(&st->epoch, a.e0 + a.steps);
        }
    }
}

/*
 * The paper's validation scheme in the chain with P readers (Section 4.2, "Speculative Reduction").
 *
 * Per step, CTA (r, c):
 *   1. the rank's operation: chunk c of its next partial, plain stores into the parity buffer;
 *   2. bar.sync, then ONE thread writes the threadblock's validation flag = call number, with release
 *      (the flag follows the payload; the flag buffer alternates with the parity like the payload);
 *   3. the four payload warps pull chunk c of all P partials and reduce it, storing the result into the
 *      rank's own row at once (nobody else reads that row), while the FIFTH warp pulls the P validation
 *      flags of the chunk and adds them up;
 *   4. bar.sync; if the sum is not P x flag the whole CTA runs step 3 again (every load is a strong
 *      access that bypasses the L1, which is what the paper's .cg on retry is for).
 * ORDERED = false issues the payload loads and the flag loads together, as the paper does: a stale
 * payload read followed by a fresh flag read would pass the check, and nothing in the memory model
 * forbids that order; the paper's "monotonicity assumption" (Section 8.1) is what rules it out in
 * practice, here for the two loads of one CTA.  ORDERED = true lets the payload warps wait until the
 * validation warp has seen all P flags (acquire): sound on any schedule, and the flag round trip is
 * back on the critical path, which makes it the dual-buffered mode with the paper's objects.
 *
 * UNCHECKED = the same pull with no flag and no check at all: the paper's idealized configuration "no
 * barriers" (Section 6.3, "Mis-Speculation and Verification Overhead"), whose results are whatever was in
 * the buffers.  A timing floor for the verification overhead, never a result.
 * Forced retries (the context's measurement knob): the first attempts that pass the check are treated as
 * failed, as many as asked for, so that the cost of a rerun can be measured (Section 6.3, "Retry Overhead").
 */
enum { kVariantConcurrent = 0, kVariantOrdered = 1, kVariantUnchecked = 2 };

template <int DT, int P, int VARIANT>
__global__ void __launch_bounds__(kSymvThreads, 4) k_symv(const SymArgs a)
{
    constexpr bool ORDERED = (VARIANT == kVariantOrdered);
    constexpr bool UNCHECKED = (VARIANT == kVariantUnchecked);
    DevState *st = a.st;
    constexpr int NW = 4;
    constexpr int NE = NW * ((DT == SIFAR_BF16) ? 2 : 1);
    const uint32_t rank = blockIdx.x % (uint32_t)P;
    const uint32_t chunk = blockIdx.x / (uint32_t)P;
    SymFlags *cf = a.flags + chunk;
    const size_t n = (size_t)a.n;
    const size_t nunits = ((n + NE - 1) / NE + 31) / 32 * 32;
    const size_t n_io = nunits * NE;
    const bool worker = threadIdx.x < (unsigned)kSymThreads;          /* payload warps; the last warp validates */
    const unsigned lane = threadIdx.x & 31u;
    const size_t unit0 = (size_t)chunk * kSymThreads * a.K + threadIdx.x;
    char *my_ring = a.rings + (size_t)rank * a.ring_len * a.ring_stride;
    constexpr uint32_t kWarps = kSymThreads / 32;
    const bool stamper = worker && lane == 0u;
    unsigned long long *my_stamps = a.stamps + (((size_t)rank * a.C + chunk) * kWarps + (threadIdx.x >> 5)) * (a.steps + 1u);
    __shared__ int s_ok;
    __shared__ int s_valid;
    __shared__ int s_giveup;
    unsigned reloads = 0;
    bool alive = true;
    uint32_t prevw[NW];
#pragma unroll
    for (int j = 0; j < NW; ++j) prevw[j] = 0u;
    if (stamper) my_stamps[0] = globaltimer_ns();

    for (uint32_t s = 0; s < a.steps && alive; ++s) {
        const uint32_t e = a.e0 + 1u + s;
        const uint32_t t = e - a.base_epoch;
        const uint32_t p = e & 1u;
        const bool first = (t == 1u);
        const Gen g = make_gen(a.w, rank, t);
        char *row = my_ring + (size_t)((t - 1u) % a.ring_len) * a.ring_stride;
        const char *prev_mem = my_ring + (size_t)((t + a.ring_len - 2u) % a.ring_len) * a.ring_stride;
        uint4 *dst = reinterpret_cast<uint4 *>(a.plain + ((size_t)p * P + rank) * a.plain_stride);

        /* ---- 1. the rank's operation ---- */
        float z0[NE];
        if (worker && unit0 < nunits) unit_noise<DT, NW>(g, first, unit0 * NE, n, z0);
        if (a.w.delay_max_ns != 0u) {
            if (threadIdx.x == 0) spin_ns(gen_delay_ns(a.w, rank, t));       /* seeded skew between the ranks */
            __syncthreads();
        }
        if (worker) {
            for (uint32_t k = 0; k < a.K; ++k) {
                const size_t u = unit0 + (size_t)k * kSymThreads;
                if (u >= nunits) break;
                uint32_t w[NW];
                if (k == 0 && s > 0u) {
                    unit_apply<DT, NW>(g, first, prevw, u * NE, n, z0, w);
                } else if (k == 0) {
                    unit_combine<DT, NW>(g, first, prev_mem, u * NE, n, z0, w, n_io);
                } else {
                    float z[NE];
                    unit_noise<DT, NW>(g, first, u * NE, n, z);
                    unit_combine<DT, NW>(g, first, prev_mem, u * NE, n, z, w, n_io);
                }
                st_slot(dst + u, make_uint4(w[0], w[1], w[2], w[3]));
            }
        }
        /* ---- 2. the threadblock's validation flag, after its payload ---- */
        if (!UNCHECKED) {
            __syncthreads();
            if (threadIdx.x == 0) st_release_u32(&cf->arrive[p][rank], e);
        }

        /* ---- 3./4. pull payload and flags, validate, run again on mis-speculation ---- */
        const uint4 *src[P];
#pragma unroll
        for (int r = 0; r < P; ++r)
            src[r] = reinterpret_cast<const uint4 *>(a.plain + ((size_t)p * P + r) * a.plain_stride);
        Deadline dl;                                                /* kept by thread 0, which decides for the CTA */
        bool retried = false;
        const auto pull_flags = [&]() {
            /* validation warp: pull-and-local-reduce of the P flags; success iff they add up to P x flag */
            uint32_t f = 0u;
            if (lane < (unsigned)P) f = ORDERED ? ld_acquire_u32(&cf->arrive[p][lane]) : ld_relaxed_u32(&cf->arrive[p][lane]);
            const uint32_t valid_out = __reduce_add_sync(0xFFFFFFFFu, f);
            if (lane == 0) s_valid = (valid_out == (uint32_t)P * e);
        };
        const auto pull_payload = [&]() {
            for (uint32_t k = 0; k < a.K; ++k) {
                const size_t u = unit0 + (size_t)k * kSymThreads;
                if (u >= nunits) break;
                uint4 x[P];
#pragma unroll
                for (int r = 0; r < P; ++r) x[r] = ld_slot(src[r] + u);
                const uint4 o = sum_vec<DT, P>(x, true);
                store_vec_result<DT>(row, u, n_io, o);              /* own row: rewritten if the check fails */
                if (k == 0) { prevw[0] = o.x; prevw[1] = o.y; prevw[2] = o.z; prevw[3] = o.w; }
            }
        };
        const auto give_up = [&]() {                                /* thread 0, after a failed check */
            const bool out_of_time = dl.expired(a.timeout_ns);
            if (out_of_time) fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
            return out_of_time || ((dl.polls % 64u) == 0u && ld_relaxed_u32(&st->status) != 0u);
        };
        uint32_t forced_left = a.poll.forced;
        for (;;) {
            if (UNCHECKED) { if (worker) pull_payload(); break; }
            if (!worker) pull_flags();
            if (!ORDERED && worker) pull_payload();                 /* at the same time as the flags, as the paper does */
            __syncthreads();                                        /* the verdict (and, unordered, the payload) */
            if (s_valid && forced_left == 0u) break;                /* uniform over the CTA */
            if (s_valid) --forced_left;                             /* a passed check counted as failed (measurement) */
            retried = true;
            if (!ORDERED) reloads += (unsigned)P;
            if (threadIdx.x == 0) s_giveup = give_up();
            __syncthreads();                                        /* s_valid may be rewritten from here on */
            if (s_giveup) { alive = false; break; }
        }
        if (ORDERED && alive && worker) pull_payload();             /* only after all P flags were seen */
        if (!alive) break;
        if (retried && threadIdx.x == 0) st_relaxed_u32(&a.retry_marks[(size_t)rank * a.steps + s], 1u);
        if (stamper) my_stamps[s + 1u] = globaltimer_ns();
    }

    /* leave: statistics, then the last CTA out books the run and publishes the call number */
    const unsigned warp_reloads = __reduce_add_sync(0xFFFFFFFFu, reloads);
    if (warp_reloads && lane == 0)
        atomicAdd(&st->stats[kStatSlotReloads], (unsigned long long)warp_reloads);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const uint32_t left = atom_add_acq_rel_u32(&a.cs->exit_count, 1u) + 1u;
        s_ok = (left == a.exit_base + gridDim.x && ld_relaxed_u32(&st->status) == 0u);
    }
    __syncthreads();
    if (s_ok) {
        unsigned long long any_steps = 0;
        for (uint32_t s = threadIdx.x; s < a.steps; s += kSymvThreads) {
            uint32_t any = 0;
            for (int r = 0; r < P; ++r) {
                const uint32_t m = ld_relaxed_u32(&a.retry_marks[(size_t)r * a.steps + s]);
                if (m) {
                    atomicAdd(&a.rank_retries[r], 1ull);
                    st_relaxed_u32(&a.retry_marks[(size_t)r * a.steps + s], 0u);
                }
                any |= m;
            }
            any_steps += any ? 1ull : 0ull;
        }
        if (any_steps) atomicAdd(&st->stats[kStatCallsWithRetry], any_steps);
        __syncthreads();
        if (threadIdx.x == 0) {
            atomicAdd(&st->stats[kStatCalls], (unsigned long long)a.steps);
            st_release_u32(&st->epoch, a.e0 + a.steps);
        }
    }
}

template <int DT, int P>
static const void *sym_kernel_p(int mode)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: return (const void *)k_sym<DT, P, SIFAR_BARRIER_ONESHOT>;
    case SIFAR_DUALBUF:         return (const void *)k_sym<DT, P, SIFAR_DUALBUF>;
    case SIFAR_SPECULATIVE:     return (const void *)k_sym<DT, P, SIFAR_SPECULATIVE>;
    case kSymTwoshot:           return (const void *)k_sym<DT, P, kSymTwoshot>;
    case kSymFlagval:           return (const void *)k_symv<DT, P, kVariantConcurrent>;
    case kSymFlagvalOrdered:    return (const void *)k_symv<DT, P, kVariantOrdered>;
    case kSymUnchecked:         return (const void *)k_symv<DT, P, kVariantUnchecked>;
    default:                    return (const void *)k_sym<DT, P, kSymNoAllreduce>;
    }
}

template <int DT>
static const void *sym_kernel_dt(int P, int mode)
{
    switch (P) {
    case 1: return sym_kernel_p<DT, 1>(mode);
    case 2: return sym_kernel_p<DT, 2>(mode);
    case 3: return sym_kernel_p<DT, 3>(mode);
    case 4: return sym_kernel_p<DT, 4>(mode);
    case 5: return sym_kernel_p<DT, 5>(mode);
    case 6: return sym_kernel_p<DT, 6>(mode);
    case 7: return sym_kernel_p<DT, 7>(mode);
    default: return sym_kernel_p<DT, 8>(mode);
    }
}

}  /* namespace sifar */

using namespace sifar;

struct sifar_symchain {
    sifar_ctx *ctx;
    sifar_workload w;
    size_t n;
    int mode;
    char *rings;
    int ring_len;
    size_t ring_stride;
    int steps;
    uint32_t base_epoch;
    uint32_t runs;
    uint32_t C, K;
    int grid;
    bool clustered;                 /* the P CTAs of a chunk as one thread-block cluster (placement only) */
    SymDev *d_cs;
    SymFlags *d_flags;
    unsigned long long *d_stamps;
    uint32_t *d_marks;
    unsigned long long *d_rank_retries;
};

/* Threads per CTA: the flag-validation modes run one extra warp. */
static int sym_threads(int mode) { return mode >= kSymFlagval ? kSymvThreads : kSymThreads; }

static const void *sym_kernel(const sifar_symchain *ch)
{
    return ch->ctx->dtype == SIFAR_BF16 ? sym_kernel_dt<SIFAR_BF16>(ch->ctx->P, ch->mode)
                                        : sym_kernel_dt<SIFAR_F32>(ch->ctx->P, ch->mode);
}

static void sym_free(sifar_symchain *ch)
{
    if (!ch) return;
    if (ch->d_cs) cudaFree(ch->d_cs);
    if (ch->d_flags) cudaFree(ch->d_flags);
    if (ch->d_stamps) cudaFree(ch->d_stamps);
    if (ch->d_marks) cudaFree(ch->d_marks);
    if (ch->d_rank_retries) cudaFree(ch->d_rank_retries);
    delete ch;
}

static int sym_setup(sifar_symchain *ch)
{
    sifar_ctx *c = ch->ctx;
    const int P = c->P;
    int coop = 0;
    SIFAR_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device));
    if (!coop) { set_error("sifar_symchain_create: device lacks cooperative launch"); return SIFAR_ERR_CUDA; }
    const size_t units = (ch->mode == SIFAR_SPECULATIVE) ? slots_for(c->dtype, ch->n)
                                                         : (ch->n * elem_size(c->dtype) + 15) / 16;
    int per_sm = 0;
    const int threads = sym_threads(ch->mode);
    SIFAR_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sym_kernel(ch), threads, 0));
    const size_t resident = (size_t)per_sm * c->sm_count;
    const size_t budget = resident > (size_t)P ? resident : (size_t)P;
    uint32_t K = 1;
    size_t C = (units + kSymThreads - 1) / kSymThreads;
    while (C * P > budget) {
        ++K;
        C = (units + (size_t)kSymThreads * K - 1) / ((size_t)kSymThreads * K);
    }
    ch->K = K; ch->C = (uint32_t)C; ch->grid = (int)(C * P);
    ch->clustered = false;
    const char *env_cluster = getenv("SIFAR_CHAIN_CLUSTER");
    if (!(env_cluster && atoi(env_cluster) == 0) && P >= 2) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3((unsigned)ch->grid);
        cfg.blockDim = dim3((unsigned)threads);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)P;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int max_clusters = 0;
        cudaError_t err = cudaOccupancyMaxActiveClusters(&max_clusters, sym_kernel(ch), &cfg);
        if (err == cudaSuccess && (size_t)max_clusters >= C) ch->clustered = true;
        else cudaGetLastError();
    }
    const size_t nstamps = (size_t)P * C * (kSymThreads / 32) * (ch->steps + 1);
    SIFAR_CUDA(cudaMalloc(&ch->d_cs, sizeof(SymDev)));
    SIFAR_CUDA(cudaMalloc(&ch->d_flags, sizeof(SymFlags) * C));
    SIFAR_CUDA(cudaMalloc(&ch->d_stamps, sizeof(unsigned long long) * nstamps));
    SIFAR_CUDA(cudaMalloc(&ch->d_marks, sizeof(uint32_t) * P * ch->steps));
    SIFAR_CUDA(cudaMalloc(&ch->d_rank_retries, sizeof(unsigned long long) * kMaxRanks));
    SIFAR_CUDA(cudaMemset(ch->d_cs, 0, sizeof(SymDev)));
    SIFAR_CUDA(cudaMemset(ch->d_flags, 0, sizeof(SymFlags) * C));
    SIFAR_CUDA(cudaMemset(ch->d_stamps, 0, sizeof(unsigned long long) * nstamps));
    SIFAR_CUDA(cudaMemset(ch->d_marks, 0, sizeof(uint32_t) * P * ch->steps));
    SIFAR_CUDA(cudaMemset(ch->d_rank_retries, 0, sizeof(unsigned long long) * kMaxRanks));
    return SIFAR_OK;
}

extern "C" sifar_symchain *sifar_symchain_create(sifar_ctx *c, const sifar_workload *w, size_t n, int mode,
                                                 void *out_rings, int ring_len, int steps_per_run)
{
    if (!c || !w || w->kind < 0 || w->kind > 2 || w->delay_max_ns > 1000000u || n == 0 || n > c->max_elems ||
        mode < 0 || mode > kSymUnchecked || !out_rings || ((uintptr_t)out_rings & 15u) || ring_len < 2 ||
        steps_per_run < 2 || (steps_per_run & 1) || steps_per_run % ring_len != 0) {
        set_error("sifar_symchain_create: bad argument (need 1 <= n <= max_elems, ring_len >= 2 dividing an even "
                  "steps_per_run, delay_max_ns <= 1000000)");
        return nullptr;
    }
    if (*c->h_status != 0) { set_error("sifar_symchain_create: context carries a device error"); return nullptr; }
    if ((uint64_t)c->h_epoch + (uint64_t)steps_per_run >= kEpochLimit) {
        set_error("sifar_symchain_create: call numbers exhausted");
        return nullptr;
    }
    sifar_symchain *ch = new (std::nothrow) sifar_symchain();
    if (!ch) { set_error("sifar_symchain_create: out of host memory"); return nullptr; }
    memset(ch, 0, sizeof *ch);
    ch->ctx = c; ch->w = *w; ch->n = n; ch->mode = mode;
    ch->rings = (char *)out_rings; ch->ring_len = ring_len;
    ch->ring_stride = sifar_chain_ring_stride(c->dtype, n);
    ch->steps = steps_per_run; ch->base_epoch = c->h_epoch; ch->runs = 0;
    cudaSetDevice(c->device);
    if (sym_setup(ch) != SIFAR_OK) { cudaGetLastError(); sym_free(ch); return nullptr; }
    return ch;
}

extern "C" int sifar_symchain_run(sifar_symchain *ch, void *stream)
{
    if (!ch) { set_error("sifar_symchain_run: NULL chain"); return SIFAR_ERR_INVALID; }
    sifar_ctx *c = ch->ctx;
    const int s0 = *c->h_status;
    if (s0) { set_error("sifar_symchain_run: context carries device status %d", s0); return s0; }
    const bool no_ar = (ch->mode == kSymNoAllreduce);
    const uint32_t expect = ch->base_epoch + (no_ar ? 0u : ch->runs * (uint32_t)ch->steps);
    if (c->h_epoch != expect) {
        set_error("sifar_symchain_run: the context was used outside the chain (call number %u, expected %u)",
                  c->h_epoch, expect);
        return SIFAR_ERR_EPOCH;
    }
    if ((uint64_t)expect + (uint64_t)ch->steps >= kEpochLimit) {
        set_error("sifar_symchain_run: call numbers exhausted");
        return SIFAR_ERR_EPOCH;
    }
    SymArgs a;
    memset(&a, 0, sizeof a);
    a.st = c->d_state; a.host_status = c->d_status_alias; a.timeout_ns = c->timeout_ns;
    a.w = ch->w; a.n = ch->n;
    a.plain = c->d_plain; a.plain_stride = c->plain_stride;
    a.slots = c->d_slots; a.slot_stride = c->slot_stride;
    a.rings = ch->rings; a.ring_stride = ch->ring_stride; a.ring_len = (uint32_t)ch->ring_len;
    a.e0 = ch->base_epoch + ch->runs * (uint32_t)ch->steps;
    a.base_epoch = ch->base_epoch; a.steps = (uint32_t)ch->steps;
    a.C = ch->C; a.K = ch->K;
    a.exit_base = ch->runs * (uint32_t)ch->grid;
    a.poll = poll_shape_for(c, ch->n);
    a.poll.sentinel = 0u;
    a.cs = ch->d_cs; a.flags = ch->d_flags; a.stamps = ch->d_stamps;
    a.retry_marks = ch->d_marks; a.rank_retries = ch->d_rank_retries;
    void *params[] = {&a};
    const void *fn = sym_kernel(ch);
    cudaStream_t s = (cudaStream_t)stream;
    if (ch->clustered) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3((unsigned)ch->grid);
        cfg.blockDim = dim3((unsigned)sym_threads(ch->mode));
        cfg.stream = s;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)c->P;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        SIFAR_CUDA(cudaLaunchKernelExC(&cfg, fn, params));
    } else {
        SIFAR_CUDA(cudaLaunchCooperativeKernel(fn, dim3((unsigned)ch->grid), dim3((unsigned)sym_threads(ch->mode)), params, 0, s));
    }
    ch->runs += 1;
    if (!no_ar) c->h_epoch += (uint32_t)ch->steps;
    c->last_mode0_epoch = 0;        /* the chain keeps its own done flags; when it has run, nothing reads the buffers */
    return SIFAR_OK;
}

/* Per step the latest stamp over the chunks of ranks [r0, r1); the run starts with the earliest CTA. */
static int sym_stamps(sifar_symchain *ch, int r0, int r1, unsigned long long *stamps)
{
    SIFAR_CUDA(cudaDeviceSynchronize());
    const size_t per = (size_t)ch->steps + 1;
    const size_t pipes = (size_t)ch->C * (kSymThreads / 32);         /* chunks x warps of one rank */
    std::vector<unsigned long long> all(per * pipes * ch->ctx->P);
    SIFAR_CUDA(cudaMemcpy(all.data(), ch->d_stamps, sizeof(unsigned long long) * all.size(), cudaMemcpyDeviceToHost));
    for (size_t s = 0; s < per; ++s) {
        unsigned long long v = 0;
        bool have = false;
        for (int r = r0; r < r1; ++r)
            for (size_t c = 0; c < pipes; ++c) {
                const unsigned long long x = all[((size_t)r * pipes + c) * per + s];
                if (!have) { v = x; have = true; }
                else v = (s == 0) ? (x < v ? x : v) : (x > v ? x : v);
            }
        stamps[s] = v;
    }
    return SIFAR_OK;
}

extern "C" int sifar_symchain_stamps(sifar_symchain *ch, unsigned long long *stamps)
{
    if (!ch || !stamps) { set_error("sifar_symchain_stamps: needs a chain and a destination"); return SIFAR_ERR_INVALID; }
    return sym_stamps(ch, 0, ch->ctx->P, stamps);
}

extern "C" int sifar_symchain_rank_stamps(sifar_symchain *ch, int rank, unsigned long long *stamps)
{
    if (!ch || !stamps || rank < 0 || rank >= ch->ctx->P) {
        set_error("sifar_symchain_rank_stamps: needs a chain, a rank below P and a destination");
        return SIFAR_ERR_INVALID;
    }
    return sym_stamps(ch, rank, rank + 1, stamps);
}

extern "C" int sifar_symchain_retries(sifar_symchain *ch, unsigned long long *per_rank)
{
    if (!ch || !per_rank) { set_error("sifar_symchain_retries: needs a chain and a destination"); return SIFAR_ERR_INVALID; }
    SIFAR_CUDA(cudaDeviceSynchronize());
    SIFAR_CUDA(cudaMemcpy(per_rank, ch->d_rank_retries, sizeof(unsigned long long) * ch->ctx->P, cudaMemcpyDeviceToHost));
    return SIFAR_OK;
}

extern "C" int sifar_symchain_destroy(sifar_symchain *ch)
{
    if (!ch) return SIFAR_OK;
    cudaSetDevice(ch->ctx->device);
    cudaError_t e = cudaDeviceSynchronize();
    sym_free(ch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
    return SIFAR_OK;
}
