/*
 * sifar_core.cu - context, producer-side store path and reducer kernels of the
 * emulated oneshot all-reduce (sm_100a).
 *
 * Protocol per call number e (parity p = e & 1), after the paper's Sections 3.1,
 * 3.3, 3.5 and 4.2, mapped onto one GPU:
 *
 *   BARRIER_ONESHOT  producer r : wait done[r] (bottom barrier, producer side);
 *                                 plain stores into the rank's single buffer;
 *                                 release arrive[p][r] = e.
 *                    reducer    : poll arrive[p][0..P) == e (top barrier);
 *                                 load, sum, store; all CTAs arrive on a counter,
 *                                 the last one releases done[0..P) = e.
 *   DUALBUF          producer r : plain stores into buffer p; release arrive.
 *                    reducer    : top barrier; load, sum, store.
 *   SPECULATIVE      producer r : one 16-byte store {12 B data, tag = e} per slot.
 *                    reducer    : load all P slots at once, accept tag == e,
 *                                 re-load only the stale ones (bounded); sum; store.
 *     large payloads (flagged tiles): the tags would cost a third more traffic, so
 *                    producer r : plain stores; one arrival flag = e per 16 KiB block,
 *                                 released as soon as that block is stored.
 *                    reducer    : a CTA acquires the P flags of its own tile only,
 *                                 then loads, sums, stores: tiles are reduced as
 *                                 they land, there is no call-wide barrier.
 *
 * What orders a reducer.  Its READS are ordered by the protocol alone (arrival
 * flags with release/acquire, or tags inside the slots), never by the stream: a
 * reducer launched with programmatic stream serialization polls and loads while
 * the kernel before it on its stream is still draining.  Its WRITES (the result,
 * the CTA count, the call number) wait for that kernel (griddepcontrol.wait), so
 * the stream order of results is what the caller expects.
 *
 * The call number lives in device memory (DevState::epoch) and is read by every
 * kernel at entry, so a replayed CUDA graph advances it without new arguments.
 * Every wait is bounded by a time limit; on expiry the kernel records a sticky
 * status and returns.
 */
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "sifar_internal.cuh"
#include "sifar_reduce.cuh"

namespace sifar {

/* ------------------------------------------------------------------------ */
/* errors                                                                    */
/* ------------------------------------------------------------------------ */
static thread_local char g_error[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char *what)
{
    set_error("%s: %s", what, cudaGetErrorString(e));
    return SIFAR_ERR_CUDA;
}

/* ------------------------------------------------------------------------ */
/* kernel arguments                                                          */
/* ------------------------------------------------------------------------ */
struct ReduceArgs {
    const uint4 *src[kMaxRanks];
    void *out;
    unsigned long long n;
    DevState *st;
    int *host_status;
    unsigned long long timeout_ns;
    uint32_t parity;
    uint32_t check_parity;
    PollShape poll;          /* speculative: how stale slots are re-polled (see validate_slot)        */
    uint32_t two_phase;      /* 1: deferring regime (see "the reducer kernel")                       */
    uint32_t janitors;       /* G: how many of the last CTAs sweep up the deferred tiles              */
    unsigned long long spin_ns;
    uint32_t *defer;         /* [0] = number of queued tiles, [1..] = their indices */
    /* arrival flags a CTA waits for before it loads plain partials: rank r's flag of tile t is
       flags[(t >> flag_shift) * kFlagStride + r] (one flag per rank and call: flag_shift = 31) */
    const uint32_t *flags;
    uint32_t flag_shift;
    uint32_t early;          /* 1: reads do not wait for the stream's previous kernel, writes do     */
    uint32_t e_host;         /* the call number the host expects, or 0: take it from device memory   */
    uint32_t pdl;            /* host side only: launch with programmatic stream serialization         */
    uint32_t sweeper;        /* 1: k_sweep follows on the stream: this grid keeps no count and no janitors */
};

struct PackArgs {
    const void *src;
    void *dst;
    unsigned long long n;
    DevState *st;
    int *host_status;
    unsigned long long timeout_ns;
    uint32_t rank;
    uint32_t parity;
    uint32_t wait_delta;     /* 0: no bottom-barrier wait; d: wait for done[rank] >= e - d */
    uint32_t *tile_flags;    /* flagged-tile format: the flag array of this call's parity ([block][kFlagStride]) */
};

/* Internal fourth mode of the plain reducer and of the pack kernel: SPECULATIVE in the flagged-tile format. */
constexpr int kModeTiles = 3;

__device__ __forceinline__ void gdc_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void gdc_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

constexpr int kThreads = 256;

/* ------------------------------------------------------------------------ */
/* exit of a reducer CTA                                                     */
/* ------------------------------------------------------------------------ */

/*
 * Completion of a call, by the one thread that knows every CTA is done: statistics,
 * the done flags of the baseline (bottom barrier, reducer side: every CTA has
 * finished reading) and the new call number.
 */
template <int MODE>
__device__ __forceinline__ void publish_call(DevState *st, uint32_t e, int P)
{
    st_relaxed_u32(&st->cta_arrive[(e + 1u) & 1u], 0u);               /* re-arm the next call's count (see DevState) */
    atomicAdd(&st->stats[kStatCalls], 1ull);                          /* result unused: fire and forget */
    if ((MODE == SIFAR_SPECULATIVE || MODE == kModeTiles) && ld_relaxed_u32(&st->retry_epoch) == e)
        atomicAdd(&st->stats[kStatCallsWithRetry], 1ull);
    if (MODE == SIFAR_BARRIER_ONESHOT) {
        /* one fence, then the P done flags: P release stores in a row would each wait for the one before */
        __threadfence();
        for (int r = 0; r < P; ++r) st_relaxed_u32(&st->done[r], e);
    }
    /* readers of the call number are ordered after this kernel by the stream or by an event */
    st_relaxed_u32(&st->epoch, e);
}

/* ------------------------------------------------------------------------ */
/* reducer tiles                                                             */
/* ------------------------------------------------------------------------ */
/*
 * A tile is kThreads * U consecutive units (16-byte vectors of plain elements,
 * or slots) and is reduced by one CTA: every thread issues its U * P coalesced
 * 16-byte loads before the first add.
 */
/* Ragged tail of a plain partial (fewer elements than a 16-byte vector holds): one element per thread, with the
   last tile. */
template <int DT, int P>
__device__ __forceinline__ void ragged_tail(const ReduceArgs &a)
{
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
    const size_t i = (size_t)a.n / EPV * EPV + threadIdx.x;
    if (i >= a.n) return;
    uint32_t w[P];
    if (DT == SIFAR_BF16) {
#pragma unroll
        for (int r = 0; r < P; ++r)
            w[r] = ld_relaxed_u16(reinterpret_cast<const uint16_t *>(a.src[r]) + i);
        reinterpret_cast<uint16_t *>(a.out)[i] = (uint16_t)(sum_word<DT, P>(w) & 0xFFFFu);
    } else {
#pragma unroll
        for (int r = 0; r < P; ++r)
            w[r] = ld_relaxed_u32(reinterpret_cast<const uint32_t *>(a.src[r]) + i);
        reinterpret_cast<uint32_t *>(a.out)[i] = sum_word<DT, P>(w);
    }
}

template <int DT, int P>
__device__ __forceinline__ void tile_plain(const ReduceArgs &a, size_t tile, size_t ntiles, bool wait_before_stores)
{
    constexpr int U = Unroll<P>::value;
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;       /* elements per 16-byte vector */
    const size_t nvec = (size_t)a.n / EPV;
    uint4 *out = reinterpret_cast<uint4 *>(a.out);
    const size_t base = tile * kThreads * U + threadIdx.x;
    uint4 x[U][P];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t v = base + (size_t)u * kThreads;
        if (v < nvec) {
#pragma unroll
            for (int r = 0; r < P; ++r) x[u][r] = ld_slot(a.src[r] + v);
        }
    }
    if (wait_before_stores) gdc_wait();                    /* the loads are in flight; nothing was written yet */
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t v = base + (size_t)u * kThreads;
        if (v < nvec) out[v] = sum_vec<DT, P>(x[u], true);
    }
    if (tile == ntiles - 1) ragged_tail<DT, P>(a);
}

/* Returns false if a slot of this thread was still stale after `limit_ns`. */
template <int DT, int P>
__device__ __forceinline__ bool tile_spec(const ReduceArgs &a, size_t tile, size_t nslots, uint32_t e,
                                          unsigned long long limit_ns, unsigned &reloads)
{
    constexpr int U = Unroll<P>::value;
    const size_t base = tile * kThreads * U + threadIdx.x;
    bool ok = true;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t s = base + (size_t)u * kThreads;
        if (s >= nslots || !ok) continue;
        uint4 x[P];
#pragma unroll
        for (int r = 0; r < P; ++r) x[r] = ld_slot(a.src[r] + s);
        /* validation (Section 4.2): a slot counts iff it carries this call's tag; stale ones are re-loaded */
        if (!validate_slot<P>(x, a.src, s, e, limit_ns, a.poll, reloads)) { ok = false; continue; }
        store_slot_result<DT>(a.out, s, (size_t)a.n, sum_slot<DT, P>(x));
    }
    return ok;
}

__host__ __device__ inline size_t tiles_for(size_t units, int per_thread)
{
    const size_t per_cta = (size_t)kThreads * per_thread;
    const size_t t = (units + per_cta - 1) / per_cta;
    return t ? t : 1;
}

constexpr uint32_t kQueuedBit = 0x80000000u;      /* in the CTA count: some CTA has queued its tile */

/* Call number, status and parity check at kernel entry.  Returns 0 if the kernel must not run. */
__device__ __forceinline__ uint32_t entry_epoch(const ReduceArgs &a, uint2 es)
{
    if (es.y != 0u) return 0u;
    const uint32_t e = es.x + 1u;
    if (a.check_parity && (e & 1u) != a.parity) {
        fail(a.st, a.host_status, SIFAR_ERR_EPOCH);
        return 0u;
    }
    return e;
}

/*
 * An early reducer may find the call number one short: the kernel before it on its stream is this
 * context's previous reducer and has not published yet.  Then, and only then, the parity is off by one.
 */
__device__ __forceinline__ bool predecessor_unpublished(const ReduceArgs &a, uint2 es)
{
    return a.early && es.y == 0u && ((es.x + 1u) & 1u) != a.parity;
}

/*
 * Top barrier (Section 3.1, phase 1) by warp 0: lane r < P loads rank r's arrival flag of this tile
 * (acquire).  The flag is the rank's single arrival flag of the call (barrier modes) or the flag of the
 * 16 KiB block the tile lies in (flagged tiles).
 *
 * Fast path: the host passed the call number it expects (a.e_host) and all P flags carry it: one load
 * per lane, one line, one round trip through the L2, nothing else is touched.  (Every word that each
 * CTA of a large grid reads is a hot spot in its L2 slice: the call-number line and the CTA-count line
 * cost 0.6 and 0.35 us per 16 MiB call when every CTA read them.)
 * Slow path (flags not there yet, or no call number from the host because the launch is being captured
 * into a graph whose replays advance it): lane P loads call number and status from device memory, lane
 * P + 1 the CTA count, whose top bit says that some CTA of this grid has already given up waiting; then
 * the bounded wait.
 *
 * Returns the call number, or 0 with `give_up` telling why: 1 = not arrived within limit_ns, 2 = error
 * or dead context.  `first` = the CTA's own tile (not a janitor's sweep).
 */
template <int P, int MODE>
__device__ __forceinline__ uint32_t top_barrier(const ReduceArgs &a, size_t tile, unsigned long long limit_ns,
                                                int &give_up, bool first)
{
    __shared__ uint32_t s_epoch;
    __shared__ int s_why;
    DevState *st = a.st;
    __syncthreads();                                  /* the shared words may still be read from an earlier use */
    if (threadIdx.x < 32) {
        const unsigned lane = threadIdx.x;
        const uint32_t *fp = a.flags + (tile >> a.flag_shift) * kFlagStride + (lane < (unsigned)P ? lane : 0u);
        uint32_t e = a.e_host, f = 0u;
        int why = 0, polls = 0;
        bool slow = (e == 0u);
        if (!slow) {
            if (lane < (unsigned)P) f = ld_acquire_u32(fp);
            slow = !__all_sync(0xFFFFFFFFu, lane >= (unsigned)P || f == e);
        }
        if (slow) {
            /* the relaxed loads first: an acquire load holds back what follows it in its thread */
            uint2 es = make_uint2(0u, 0u);
            uint32_t count = 0u;
            if (lane == (unsigned)P) es = ld_relaxed_u32x2(&st->epoch);
            if (lane == (unsigned)P + 1u) count = ld_relaxed_u32(&st->cta_arrive[a.parity]);
            if (lane < (unsigned)P) f = ld_acquire_u32(fp);
            es.x = __shfl_sync(0xFFFFFFFFu, es.x, P);
            es.y = __shfl_sync(0xFFFFFFFFu, es.y, P);
            count = __shfl_sync(0xFFFFFFFFu, count, P + 1);
            if (first && predecessor_unpublished(a, es)) {
                /* wait for the stream's previous kernel (this context's previous reducer), then look again */
                gdc_wait();
                if (lane == (unsigned)P) es = ld_relaxed_u32x2(&st->epoch);
                es.x = __shfl_sync(0xFFFFFFFFu, es.x, P);
                es.y = __shfl_sync(0xFFFFFFFFu, es.y, P);
            }
            e = entry_epoch(a, es);
            why = e ? 0 : 2;
            if (e && a.e_host && e != a.e_host) {     /* host and device disagree about the call number */
                fail(st, a.host_status, SIFAR_ERR_EPOCH);
                e = 0u; why = 2;
            }
            if (e) {
                const bool ready = lane >= (unsigned)P || f == e;
                if (!__all_sync(0xFFFFFFFFu, ready)) {
                    if (first && a.two_phase && (count & kQueuedBit)) {
                        why = 1;       /* the grid runs ahead of its producers: do not hold the SM, queue at once */
                    } else if (!ready) {
                        polls = wait_flag_eq(fp, e, limit_ns);
                        if (polls < 0) { why = 1; polls = 0; }
                        polls += 1;    /* the first look counts */
                    }
                }
            }
            why = __reduce_max_sync(0xFFFFFFFFu, why);
            polls = __reduce_add_sync(0xFFFFFFFFu, polls);
        }
        if (lane == 0) {
            s_epoch = why ? 0u : e;
            s_why = why;
            if (polls) {
                atomicAdd(&st->stats[kStatFlagPolls], (unsigned long long)polls);
                /* flagged tiles: a tile whose flags were not there at the first look is a mis-speculation */
                if (MODE == kModeTiles && e) st_relaxed_u32(&st->retry_epoch, e);
            }
        }
    }
    __syncthreads();
    give_up = s_why;
    return s_epoch;
}

/* ------------------------------------------------------------------------ */
/* the reducer kernel                                                        */
/* ------------------------------------------------------------------------ */
/*
 * One CTA per tile.  Two regimes, chosen by the host from the grid size:
 *
 * in place (grid <= one CTA per SM): a CTA waits for its data as long as the
 *   time limit allows; it cannot keep the producers off the machine.
 *
 * deferring (larger grids): a reducer that fills every SM and then waits would
 *   keep the very producers it waits for from being scheduled.  So a CTA waits
 *   only spin_ns; if its tile is still not ready it queues the tile and leaves.
 *   The G CTAs with the highest indices (G <= one per SM) stay as janitors: they
 *   wait until everybody has arrived, split the queued tiles among themselves
 *   and reduce them with the full time limit.  With producers that are on time
 *   the queue is empty and the janitors cost a short wait at the very end.
 *   Where the host appends the sweep kernel (a.sweeper, see k_sweep) there are no
 *   janitors and no count: a CTA reduces or queues its tile and leaves, and the
 *   sweep kernel, ordered behind the whole grid, does the rest.
 *
 * Either way the last CTA out publishes the call (publish_call).
 */
struct Roles {
    uint32_t janitor;      /* 0: leave; k+1: janitor number k                       */
    uint32_t ndefer;       /* queued tiles (valid for janitors)                     */
    uint32_t ok;
};

/* Thread 0 of a CTA in the deferring regime: queue the CTA's tile (made visible before the CTA's arrival). */
__device__ __forceinline__ void defer_tile(const ReduceArgs &a, size_t tile)
{
    const uint32_t slot = atomicAdd(a.defer, 1u);
    st_relaxed_u32(a.defer + 1u + slot, (uint32_t)tile);
    __threadfence();
    /* "something is queued" travels in the top bit of the arrival count, set before this thread counts its
       CTA: who sees the count complete knows from the same word whether the queue needs a look */
    asm volatile("red.relaxed.gpu.global.or.b32 [%0], %1;" :: "l"(&a.st->cta_arrive[a.parity]), "r"(kQueuedBit) : "memory");
}

/*
 * End of a CTA's own tile (all threads call; `alive` = no error seen).  Returns
 * the CTA's role.
 *   In place: CTAs count themselves with an atomic whose result they read; the
 *   last arrival publishes the call.
 *   Deferring: a CTA's SM slot is worth more than the answer, so it counts itself
 *   with a fire-and-forget increment and leaves.  The G CTAs with the highest
 *   indices (dispatched last) are the janitors: they wait until the count is
 *   complete and then learn from the same word whether anything was queued.
 *   Nothing queued (the usual case): janitor 1 publishes, the others just leave.
 * The count is polled with relaxed loads (half the round trip of an acquire); a
 * fence follows only if the queue has to be read.  A relaxed count is enough in
 * both regimes: the CTA's loads have returned (its stores depended on them),
 * which is all the bottom barrier asks; `out` is handed over by the kernel
 * boundary; a queued tile was fenced by defer_tile().  The word counts this
 * call only (the other parity's word is re-armed by the CTA that publishes), so a
 * janitor that looks late still finds it complete.
 */
template <int MODE>
__device__ __forceinline__ Roles cta_arrive(const ReduceArgs &a, uint32_t e, int P, bool alive, bool want_defer,
                                            size_t tile)
{
    __shared__ Roles s_roles;
    DevState *st = a.st;
    uint32_t *counter = &st->cta_arrive[a.parity];
    const uint32_t n = gridDim.x;
    const bool janitor = a.two_phase && blockIdx.x + a.janitors >= n;
    /* One barrier: every thread's loads are done.  In place it also collects "somebody saw an error"; in
       the deferring regime errors are uniform over the CTA and the barrier collects "somebody wants to defer". */
    int dead;
    if (a.two_phase) {
        dead = !alive;
        if (__syncthreads_or(want_defer) && !dead && threadIdx.x == 0) defer_tile(a, tile);
    } else {
        dead = __syncthreads_or(!alive);
    }
    if (a.two_phase && !janitor) {
        if (!dead && threadIdx.x == 0) red_add_relaxed_u32(counter, 1u);
        return Roles{0u, 0u, (uint32_t)!dead};
    }
    if (threadIdx.x == 0) {
        Roles r = {0u, 0u, (uint32_t)!dead};
        if (!dead && !a.two_phase) {
            const uint32_t arrived = (n > 1u) ? atom_add_relaxed_u32(counter, 1u) + 1u : 1u;
            if (arrived == n) publish_call<MODE>(st, e, P);
        } else if (!dead) {
            r.janitor = blockIdx.x + a.janitors - n + 1u;              /* 1 .. G */
            red_add_relaxed_u32(counter, 1u);
            Deadline d;
            uint32_t count;
            for (;;) {
                count = ld_relaxed_u32(counter);
                if ((count & ~kQueuedBit) >= n) break;
                if (d.expired(a.timeout_ns)) { fail(st, a.host_status, SIFAR_ERR_TIMEOUT); r.ok = 0u; break; }
                if ((d.polls % 64u) == 0u && ld_relaxed_u32(&st->status) != 0u) { r.ok = 0u; break; }
            }
            if (r.ok && (count & kQueuedBit)) {
                __threadfence();                                       /* the queue entries of the CTAs counted */
                r.ndefer = ld_relaxed_u32(a.defer);
            }
            if (r.ok && r.ndefer == 0u) {
                if (r.janitor == 1u) publish_call<MODE>(st, e, P);
                r.janitor = 0u;
            }
        }
        s_roles = r;
    }
    __syncthreads();
    return s_roles;
}

/* Mis-speculation statistics of a CTA: one atomic per warp that re-loaded anything; must precede the arrival. */
__device__ __forceinline__ void flush_reloads(DevState *st, uint32_t e, unsigned &reloads)
{
    const unsigned warp_reloads = __reduce_add_sync(0xFFFFFFFFu, reloads);
    if (warp_reloads && (threadIdx.x & 31) == 0) {
        atomicAdd(&st->stats[kStatSlotReloads], (unsigned long long)warp_reloads);
        if (e) st_relaxed_u32(&st->retry_epoch, e);
    }
    reloads = 0;
}

/* A janitor is done with its share (all threads call).  The last janitor re-arms the queue and publishes. */
template <int MODE>
__device__ __forceinline__ void janitor_leave(const ReduceArgs &a, uint32_t e, int P, bool alive)
{
    DevState *st = a.st;
    if (!__syncthreads_and(alive)) return;
    if (threadIdx.x == 0) {
        const uint32_t left = atom_add_relaxed_u32(&st->janitor_done, 1u) + 1u;
        if (left == a.janitors) {
            st_relaxed_u32(&st->janitor_done, 0u);
            st_relaxed_u32(a.defer, 0u);
            publish_call<MODE>(st, e, P);
        }
    }
}

template <int DT, int P, int MODE>
__global__ void __launch_bounds__(kThreads, 4) k_reduce_plain(const ReduceArgs a)
{
    constexpr int U = Unroll<P>::value;
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
    const size_t ntiles = tiles_for((size_t)a.n / EPV, U);
    const size_t tile = blockIdx.x;
    /* Programmatic dependent launch: the next kernel of the stream may become resident as soon as every
       CTA of this one has started.  Whether this kernel's own reads wait for the kernel before it is the
       host's choice (a.early, see launch_reduce); its writes always do. */
    if (!a.early) gdc_wait();
    gdc_launch_dependents();
    int give_up = 0;
    if (a.early && !a.sweeper && (threadIdx.x & 7u) == 0u) {
        /* While warp 0 makes its round trip for the flags, ask the L2 for the tile's lines (one thread per
           128-byte line).  A prefetch returns nothing to the thread, so it cannot deliver stale data: the
           loads below still follow the flags, and the L2 is where the producers' stores arrive.  Not where
           the host saw the producers still busy (a.sweeper): a grid that runs ahead of its producers would
           read every partial once for nothing, beside the very kernels that are storing them. */
        constexpr int EPVp = (DT == SIFAR_BF16) ? 8 : 4;
        const size_t nvec = (size_t)a.n / EPVp;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t v = tile * kThreads * U + (size_t)u * kThreads + threadIdx.x;
            if (v < nvec) {
#pragma unroll
                for (int r = 0; r < P; ++r) asm volatile("prefetch.global.L2 [%0];" :: "l"(a.src[r] + v));
            }
        }
    }
    if (MODE == kModeTiles && a.early && !a.sweeper && threadIdx.x == 33u) {
        /* and for the flags of the CTA that takes this CTA's place a wave from now: block flags are read once
           each, so unlike the one arrival line of the barrier modes they are not in the L2 when asked for */
        const size_t later = tile + 4u * (size_t)a.janitors;
        if (later < gridDim.x)
            asm volatile("prefetch.global.L2 [%0];" :: "l"(a.flags + (later >> a.flag_shift) * kFlagStride));
    }
    uint32_t e = top_barrier<P, MODE>(a, tile, a.two_phase ? a.spin_ns : a.timeout_ns, give_up, true);
    bool alive = true;
    if (e == 0u) {
        if (a.early) gdc_wait();                                       /* before anything is written */
        if (give_up == 2) return;                                      /* dead context */
        if (!a.two_phase) {
            if (threadIdx.x == 0) fail(a.st, a.host_status, SIFAR_ERR_TIMEOUT);
            return;
        }
        /* the ranks are late: queue the tile and free the SM; the call number is still needed to arrive */
        if (threadIdx.x == 0) defer_tile(a, tile);
        if (a.sweeper) return;
        e = entry_epoch(a, ld_relaxed_u32x2(&a.st->epoch));         /* after the wait: the predecessor has published */
        alive = (e != 0u);
    } else {
        tile_plain<DT, P>(a, tile, ntiles, a.early != 0u);             /* pull and reduce (phase 2) */
    }
    /* a sweep kernel follows on the stream: it is ordered after this whole grid, reduces what was queued
       and closes the call */
    if (a.sweeper) return;
    /* phase 3 (bottom barrier, baseline only) and publication of the call number by the last CTA out */
    const Roles role = cta_arrive<MODE>(a, e, P, alive, false, tile);
    if (!role.janitor) return;
    alive = (role.ok != 0u);
    for (uint32_t i = role.janitor - 1u; i < role.ndefer && alive; i += a.janitors) {
        const size_t t = ld_relaxed_u32(a.defer + 1u + i);
        /* flagged tiles: the flags of each queued tile; barrier modes: the same P flags every time */
        if (MODE == kModeTiles || i == role.janitor - 1u) {
            alive = (top_barrier<P, MODE>(a, t, a.timeout_ns, give_up, false) != 0u);
            if (!alive && give_up == 1 && threadIdx.x == 0) fail(a.st, a.host_status, SIFAR_ERR_TIMEOUT);
        }
        if (alive) tile_plain<DT, P>(a, t, ntiles, false);
    }
    janitor_leave<MODE>(a, e, P, alive);
}

/*
 * The sweep kernel: second half of a large call in plain format whose producers are still busy on other
 * streams when the call is enqueued.
 *
 * The janitors of k_reduce_plain sweep queued tiles with the registers of one quarter-occupancy CTA per
 * SM: P loads of 16 bytes per thread, 32 KB per SM in flight, a third of the machine's bandwidth (42 us
 * for the 134 MB of a 16 MiB/rank call at P = 8).  Such a call gets this kernel behind its reducer grid
 * instead, and the grid keeps neither a CTA count nor janitors.  One CTA per SM as well, so that the late
 * producers find room beside it, but compiled for one CTA per SM: a thread keeps kSweepTiles tiles in flight
 * (128 KB per SM; 28 us for the same sweep).  It starts when the reducer grid is over (griddepcontrol.wait:
 * the queue is complete and visible).  Nothing queued: CTA 0 closes the call and that is all.  Otherwise a
 * CTA takes kSweepTiles queue entries per round, warp 0 checks all their flags with one round trip
 * (lane = (tile, rank)), the CTA reduces them, and the last CTA out closes the call.
 *
 * (The same sweep out of shared memory - two stages of three tiles filled with cp.async, 56 registers, so
 * that its CTAs fit beside a full reducer grid - was built and measured: 36 us instead of 28, the producers
 * beside it 40 us slower, and no cheaper on ready data, where what this kernel costs is its place in the
 * stream's chain of dependent launches, 1.1-1.8 us per call.)
 */
constexpr int kSweepTiles = 4;
constexpr int kSweepFromTilesPerSm = 8;      /* below 8 queued tiles per janitor the janitors are as fast */
constexpr unsigned long long kSweepSpinNs = 500;   /* how long a CTA of the grid before it waits for its tile */

template <int DT, int P, int MODE>
__global__ void __launch_bounds__(kThreads, 1) k_sweep(const ReduceArgs a)
{
    constexpr int U = Unroll<P>::value;
    constexpr int K = kSweepTiles;
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
    static_assert(K * P <= 32, "one lane of warp 0 per (tile, rank)");
    __shared__ uint32_t s_e, s_n, s_tile[K];
    __shared__ int s_ok;
    DevState *st = a.st;
    gdc_launch_dependents();
    gdc_wait();
    if (threadIdx.x == 0) {
        uint32_t e = entry_epoch(a, ld_relaxed_u32x2(&st->epoch));
        if (e && a.e_host && e != a.e_host) { fail(st, a.host_status, SIFAR_ERR_EPOCH); e = 0u; }
        s_e = e;
        s_n = e ? ld_relaxed_u32(a.defer) : 0u;
    }
    __syncthreads();
    const uint32_t e = s_e, ndefer = s_n;
    if (e == 0u) return;
    if (ndefer == 0u) {
        if (blockIdx.x == 0 && threadIdx.x == 0) publish_call<MODE>(st, e, P);
        return;
    }
    const size_t nvec = (size_t)a.n / EPV;
    const size_t ntiles = tiles_for(nvec, U);
    uint4 *out = reinterpret_cast<uint4 *>(a.out);
    bool alive = true, checked = false;
    for (uint32_t g = blockIdx.x; (size_t)g * K < ndefer && alive; g += gridDim.x) {
        const uint32_t first = g * K;
        const int cnt = (ndefer - first < (uint32_t)K) ? (int)(ndefer - first) : K;
        if (threadIdx.x < 32) {
            const int lane = (int)threadIdx.x, j = lane / P, r = lane % P;
            const bool mine = j < cnt;
            const uint32_t t = mine ? ld_relaxed_u32(a.defer + 1u + first + (uint32_t)j) : 0u;
            if (mine && r == 0) s_tile[j] = t;
            int why = 0, polls = 0;
            /* flagged tiles: the flags of every queued tile; barrier modes: the same P flags, once */
            if (mine && (MODE == kModeTiles || !checked)) {
                const uint32_t *fp = a.flags + (size_t)(t >> a.flag_shift) * kFlagStride + r;
                if (ld_acquire_u32(fp) != e) {
                    polls = wait_flag_eq(fp, e, a.timeout_ns);
                    if (polls < 0) { why = 1; polls = 0; }
                    polls += 1;
                }
            }
            why = __reduce_max_sync(0xFFFFFFFFu, why);
            polls = __reduce_add_sync(0xFFFFFFFFu, polls);
            if (lane == 0) {
                s_ok = !why;
                if (polls) atomicAdd(&st->stats[kStatFlagPolls], (unsigned long long)polls);
                if (why) fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
            }
        }
        __syncthreads();
        alive = (s_ok != 0);
        checked = true;
        if (alive) {
            uint4 x[K][U][P];
#pragma unroll
            for (int j = 0; j < K; ++j) {
                if (j < cnt) {
                    const size_t base = (size_t)s_tile[j] * kThreads * U + threadIdx.x;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const size_t v = base + (size_t)u * kThreads;
                        if (v < nvec) {
#pragma unroll
                            for (int r = 0; r < P; ++r) x[j][u][r] = ld_slot(a.src[r] + v);
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < K; ++j) {
                if (j < cnt) {
                    const size_t base = (size_t)s_tile[j] * kThreads * U + threadIdx.x;
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const size_t v = base + (size_t)u * kThreads;
                        if (v < nvec) out[v] = sum_vec<DT, P>(x[j][u], true);
                    }
                    if (s_tile[j] == ntiles - 1) ragged_tail<DT, P>(a);
                }
            }
        }
        __syncthreads();                                    /* s_tile and s_ok are written again next round */
    }
    if (!__syncthreads_and(alive)) return;
    if (threadIdx.x == 0) {
        const uint32_t left = atom_add_relaxed_u32(&st->janitor_done, 1u) + 1u;
        if (left == gridDim.x) {
            st_relaxed_u32(&st->janitor_done, 0u);
            st_relaxed_u32(a.defer, 0u);
            /* flagged tiles: a tile that had to be queued was not there at the first look (mis-speculation) */
            if (MODE == kModeTiles) st_relaxed_u32(&st->retry_epoch, e);
            publish_call<MODE>(st, e, P);
        }
    }
}

template <int DT, int P>
__global__ void __launch_bounds__(kThreads, 4) k_reduce_spec(const ReduceArgs a)
{
    constexpr int U = Unroll<P>::value;
    constexpr int EPS = kSlotDataWords * ((DT == SIFAR_BF16) ? 2 : 1);
    DevState *st = a.st;
    const size_t nslots = ((size_t)a.n + EPS - 1) / EPS;
    const size_t tile = blockIdx.x;
    const unsigned long long limit_ns = a.two_phase ? a.spin_ns : a.timeout_ns;
    unsigned reloads = 0;
    /* programmatic dependent launch, as in k_reduce_plain: the slots validate themselves, so the loads
       need not wait for the kernel before this one on the stream unless the host says so */
    if (!a.early) gdc_wait();
    gdc_launch_dependents();

    /* The call number is loaded together with the slots (no dependent round trip before the data), by one
       thread per CTA: a word that every warp of a large grid loads becomes a hot spot in its L2 slice. */
    __shared__ uint2 s_es;
    if (threadIdx.x == 0) s_es = a.e_host ? make_uint2(a.e_host - 1u, 0u) : ld_relaxed_u32x2(&st->epoch);
    const size_t base = tile * kThreads * U + threadIdx.x;
    uint4 x[U][P];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t s = base + (size_t)u * kThreads;
        if (s < nslots) {
#pragma unroll
            for (int r = 0; r < P; ++r) x[u][r] = ld_slot(a.src[r] + s);
        }
    }
    __syncthreads();
    if (!a.e_host && predecessor_unpublished(a, s_es)) {    /* uniform over the CTA */
        /* this context's previous reducer is still running ahead of us on the stream: wait for it and read
           the call number again (what was loaded above is then stale and is loaded again by the validation) */
        gdc_wait();
        __syncthreads();
        if (threadIdx.x == 0) s_es = ld_relaxed_u32x2(&st->epoch);
        __syncthreads();
    }
    const uint32_t e = entry_epoch(a, s_es);
    bool alive = (e != 0u);
    bool ok = true;
    if (alive) {
        /* validation (Section 4.2): a slot counts iff it carries this call's tag; stale ones are re-loaded */
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t s = base + (size_t)u * kThreads;
            if (s >= nslots || !ok) continue;
            ok = validate_slot<P>(x[u], a.src, s, e, limit_ns, a.poll, reloads);
        }
    }
    if (a.early) gdc_wait();                                /* everything from here on writes */
    if (alive) {
        if (ok) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t s = base + (size_t)u * kThreads;
                if (s < nslots) store_slot_result<DT>(a.out, s, (size_t)a.n, sum_slot<DT, P>(x[u]));
            }
        } else if (!a.two_phase) {
            fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
            alive = false;
        }
    }
    flush_reloads(st, e, reloads);
    /* deferring regime: a slot that stayed stale past the short limit sends the whole tile to a janitor */
    const Roles role = cta_arrive<SIFAR_SPECULATIVE>(a, e, P, alive, a.two_phase && !ok, tile);
    if (!role.janitor) return;
    alive = (role.ok != 0u);
    for (uint32_t i = role.janitor - 1u; i < role.ndefer && alive; i += a.janitors) {
        if (!tile_spec<DT, P>(a, ld_relaxed_u32(a.defer + 1u + i), nslots, e, a.timeout_ns, reloads)) {
            fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
            alive = false;
        }
    }
    flush_reloads(st, e, reloads);
    janitor_leave<SIFAR_SPECULATIVE>(a, e, P, alive);
}

/* ------------------------------------------------------------------------ */
/* producer-side store path                                                  */
/* ------------------------------------------------------------------------ */
constexpr int kPackUnroll = 4;

template <int DT, int MODE>
__device__ __forceinline__ void pack_body(const PackArgs &a)
{
    DevState *st = a.st;
    __shared__ uint32_t s_epoch;
    /* a reducer that follows on the same stream may become resident now; it waits for this grid's completion */
    asm volatile("griddepcontrol.launch_dependents;");
    if (threadIdx.x == 0) {
        const uint2 es = ld_relaxed_u32x2(&st->epoch);
        uint32_t e = es.x + 1u;
        bool ok = (es.y == 0u);
        /* The call number is the device's, so this producer must be ordered after the previous call's reducer
           (stream, event or graph edge).  One that was not reads a call number that is one short: its parity
           differs from what the host enqueued it for. */
        if (ok && (e & 1u) != a.parity) {
            fail(st, a.host_status, SIFAR_ERR_EPOCH);
            ok = false;
        }
        /* Bottom barrier, producer side: the previous reader of this single buffer must be done. */
        if (ok && MODE == SIFAR_BARRIER_ONESHOT && a.wait_delta) {
            if (wait_flag_ge(&st->done[a.rank], e - a.wait_delta, a.timeout_ns) < 0) {
                fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
                ok = false;
            }
        }
        s_epoch = ok ? e : 0u;
    }
    __syncthreads();
    const uint32_t e = s_epoch;
    if (e == 0u) return;

    const size_t tid = (size_t)blockIdx.x * kThreads + threadIdx.x;
    const size_t nthreads = (size_t)gridDim.x * kThreads;
    if (MODE == kModeTiles) {
        /* Flagged tiles: plain data, and one arrival flag per block of kFlagBlockVecs vectors, released as soon
           as the block is stored, so that the reducer can start on it while the rest is still being written.
           One block per CTA and round, four vectors per thread in flight.  The releasing thread changes from
           round to round: its fence then overlaps the next round's loads of the other warps. */
        constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
        constexpr int VPT = (int)(kFlagBlockVecs / kThreads);
        const size_t nvec = (size_t)a.n / EPV;
        const size_t nblocks = nvec ? (nvec + kFlagBlockVecs - 1) / kFlagBlockVecs : 1;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.src);
        uint4 *dst = reinterpret_cast<uint4 *>(a.dst);
        unsigned round = 0;
        for (size_t b = blockIdx.x; b < nblocks; b += gridDim.x, ++round) {
            const size_t v0 = b * kFlagBlockVecs + threadIdx.x;
            uint4 x[VPT];
#pragma unroll
            for (int j = 0; j < VPT; ++j)
                if (v0 + (size_t)j * kThreads < nvec) x[j] = __ldcs(src + v0 + (size_t)j * kThreads);
#pragma unroll
            for (int j = 0; j < VPT; ++j)
                if (v0 + (size_t)j * kThreads < nvec) st_slot(dst + v0 + (size_t)j * kThreads, x[j]);
            const size_t i = nvec * EPV + threadIdx.x;                 /* ragged tail, with the last block */
            if (b == nblocks - 1 && i < a.n) {
                if (DT == SIFAR_BF16)
                    reinterpret_cast<uint16_t *>(a.dst)[i] = reinterpret_cast<const uint16_t *>(a.src)[i];
                else
                    reinterpret_cast<uint32_t *>(a.dst)[i] = reinterpret_cast<const uint32_t *>(a.src)[i];
            }
            __syncthreads();
            if (threadIdx.x == ((round * 32u) % kThreads)) st_release_u32(a.tile_flags + b * kFlagStride + a.rank, e);
        }
    } else if (MODE != SIFAR_SPECULATIVE) {
        constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
        const size_t nvec = (size_t)a.n / EPV;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.src);
        uint4 *dst = reinterpret_cast<uint4 *>(a.dst);
        /* kPackUnroll independent loads in flight per thread, then their stores */
        size_t v = tid;
        for (; v + (kPackUnroll - 1) * nthreads < nvec; v += kPackUnroll * nthreads) {
            uint4 x[kPackUnroll];
#pragma unroll
            for (int j = 0; j < kPackUnroll; ++j) x[j] = __ldcs(src + v + j * nthreads);
#pragma unroll
            for (int j = 0; j < kPackUnroll; ++j) st_slot(dst + v + j * nthreads, x[j]);
        }
        for (; v < nvec; v += nthreads) st_slot(dst + v, src[v]);
        const size_t i = nvec * EPV + threadIdx.x;
        if (blockIdx.x == 0 && i < a.n) {
            if (DT == SIFAR_BF16)
                reinterpret_cast<uint16_t *>(a.dst)[i] = reinterpret_cast<const uint16_t *>(a.src)[i];
            else
                reinterpret_cast<uint32_t *>(a.dst)[i] = reinterpret_cast<const uint32_t *>(a.src)[i];
        }
        signal_arrival(&st->pack_count[a.rank], gridDim.x, &st->arrive[e & 1u][a.rank], e);
    } else {
        constexpr int EPS = kSlotDataWords * ((DT == SIFAR_BF16) ? 2 : 1);
        constexpr int NW = kSlotDataWords;
        const size_t nslots = ((size_t)a.n + EPS - 1) / EPS;
        uint4 *slots = reinterpret_cast<uint4 *>(a.dst);
        const uint32_t *src32 = reinterpret_cast<const uint32_t *>(a.src);
        /* whole slots first, kPackUnroll of them in flight per thread; the loop below takes the rest */
        const size_t nfull = (size_t)a.n / EPS;
        size_t s = tid;
        for (; s + (kPackUnroll - 1) * nthreads < nfull; s += kPackUnroll * nthreads) {
            uint32_t w[kPackUnroll][NW];
#pragma unroll
            for (int j = 0; j < kPackUnroll; ++j) {
                const uint32_t *p = src32 + (s + j * nthreads) * NW;
#pragma unroll
                for (int q = 0; q < NW; ++q) w[j][q] = __ldcs(p + q);
            }
#pragma unroll
            for (int j = 0; j < kPackUnroll; ++j) store_slot_words(slots, s + j * nthreads, w[j], e);
        }
        for (; s < nslots; s += nthreads) {
            uint32_t w[NW];
#pragma unroll
            for (int q = 0; q < NW; ++q) w[q] = 0u;
            const size_t i0 = s * EPS;
            if (i0 + EPS <= a.n) {
#pragma unroll
                for (int q = 0; q < NW; ++q) w[q] = src32[s * NW + q];
            } else if (DT == SIFAR_BF16) {
                const uint16_t *src16 = reinterpret_cast<const uint16_t *>(a.src);
                for (int k = 0; k < EPS && i0 + k < a.n; ++k)
                    w[k >> 1] |= (uint32_t)src16[i0 + k] << ((k & 1) * 16);
            } else {
                for (int k = 0; k < EPS && i0 + k < a.n; ++k) w[k] = src32[i0 + k];
            }
            store_slot_words(slots, s, w, e);
        }
    }
}

template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads) k_pack(const PackArgs a)
{
    pack_body<DT, MODE>(a);
}

/* All P ranks in one launch (blockIdx.y = rank): the host-buffer entry point packs straight from pinned host memory. */
struct PackAllArgs {
    const void *src[kMaxRanks];
    void *dst[kMaxRanks];
    PackArgs common;             /* src, dst and rank are filled in per rank */
};

template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads) k_pack_all(const PackAllArgs all)
{
    PackArgs a = all.common;
    a.rank = blockIdx.y;
    a.src = all.src[blockIdx.y];
    a.dst = all.dst[blockIdx.y];
    pack_body<DT, MODE>(a);
}

/* Release of one rank's arrival flag after caller-written plain partials. */
__global__ void k_arrive(DevState *st, int *host_status, uint32_t rank, uint32_t parity)
{
    const uint2 es = ld_relaxed_u32x2(&st->epoch);
    if (es.y != 0u) return;
    const uint32_t e = es.x + 1u;
    if ((e & 1u) != parity) { fail(st, host_status, SIFAR_ERR_EPOCH); return; }   /* not ordered after the previous call */
    __threadfence();
    st_release_u32(&st->arrive[e & 1u][rank], e);
}

/* Producer-side half of the bottom barrier as a kernel of its own. */
__global__ void k_wait_writable(DevState *st, int *host_status, uint32_t rank, uint32_t wait_delta, uint32_t parity,
                                unsigned long long timeout_ns)
{
    const uint2 es = ld_relaxed_u32x2(&st->epoch);
    if (es.y != 0u) return;
    const uint32_t e = es.x + 1u;
    if ((e & 1u) != parity) { fail(st, host_status, SIFAR_ERR_EPOCH); return; }
    if (wait_flag_ge(&st->done[rank], e - wait_delta, timeout_ns) < 0) fail(st, host_status, SIFAR_ERR_TIMEOUT);
}

/* n = 0: nothing to move, the call number still advances. */
__global__ void k_empty_call(DevState *st, int mode, int P)
{
    const uint2 es = ld_relaxed_u32x2(&st->epoch);
    if (es.y != 0u) return;
    const uint32_t e = es.x + 1u;
    st->stats[kStatCalls] += 1ull;
    st->cta_arrive[(e + 1u) & 1u] = 0u;             /* what the CTA that closes a call does for the next one */
    if (mode == SIFAR_BARRIER_ONESHOT) {
        __threadfence();
        for (int r = 0; r < P; ++r) st_relaxed_u32(&st->done[r], e);
    }
    st_release_u32(&st->epoch, e);
}

__global__ void k_set_epoch(DevState *st, uint32_t e) { st->epoch = e; st->cta_arrive[0] = 0u; st->cta_arrive[1] = 0u; }

/* ------------------------------------------------------------------------ */
/* launch geometry                                                           */
/* ------------------------------------------------------------------------ */
/*
 * Programmatic dependent launch: a reducer may become resident while the kernel before it on its stream
 * is still draining.  Its CTAs then sit in griddepcontrol.wait until that kernel has completed and its
 * writes are visible, so what they read is unchanged; what is saved is the launch gap and the ramp-up
 * between back-to-back kernels (about 2 us per pair).  Used for reducer grids above the SM count, where
 * bandwidth is what counts.  SIFAR_PDL=0 launches the plain way.
 */
static bool g_pdl = !(getenv("SIFAR_PDL") && atoi(getenv("SIFAR_PDL")) == 0);
/* SIFAR_BARRIER_EARLY=1: the baseline's reads may start early too (they are ordered by its arrival flags just as
   well); off by default: the baseline stands for the conventional design, which orders everything by the stream. */
static bool g_barrier_early = getenv("SIFAR_BARRIER_EARLY") && atoi(getenv("SIFAR_BARRIER_EARLY")) != 0;
/* SIFAR_SWEEP=0: contexts start with SIFAR_SWEEP_NEVER (the janitors of the reducer grid sweep, as for small grids). */
static bool g_sweep = !(getenv("SIFAR_SWEEP") && atoi(getenv("SIFAR_SWEEP")) == 0);

static thread_local cudaEvent_t g_programmatic_event = nullptr;   /* set by launch_reduce around the launch */

template <typename K>
static cudaError_t launch_k(K kernel, int grid, cudaStream_t s, const ReduceArgs &a)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(kThreads); cfg.stream = s;
    if (g_programmatic_event) {
        /* The event fires once every CTA has released its dependents (right after the kernel's own dependency
           wait), so kernels of other streams that wait for it can become resident while this one still runs;
           they call griddepcontrol.wait before they read anything. */
        cudaLaunchAttribute ev[1];
        ev[0].id = cudaLaunchAttributeProgrammaticEvent;
        ev[0].val.programmaticEvent.event = g_programmatic_event;
        ev[0].val.programmaticEvent.flags = 0;
        ev[0].val.programmaticEvent.triggerAtBlockStart = 0;
        cfg.attrs = ev; cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, a);
    }
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    /* for grids above the SM count, and for any grid whose producers are known to run on other streams: at
       decode payloads a reducer that becomes resident early beside the very kernels it waits for measurably
       slows the graph chains and the host path */
    cfg.attrs = at; cfg.numAttrs = (g_pdl && (a.two_phase || a.pdl)) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

template <int DT, int P>
static cudaError_t launch_sweep_p(int mode, int grid, cudaStream_t s, const ReduceArgs &a)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: return launch_k(k_sweep<DT, P, SIFAR_BARRIER_ONESHOT>, grid, s, a);
    case SIFAR_DUALBUF:         return launch_k(k_sweep<DT, P, SIFAR_DUALBUF>, grid, s, a);
    default:                    return launch_k(k_sweep<DT, P, kModeTiles>, grid, s, a);
    }
}

template <int DT>
static cudaError_t launch_sweep_dt(int P, int mode, int grid, cudaStream_t s, const ReduceArgs &a)
{
    switch (P) {
    case 1: return launch_sweep_p<DT, 1>(mode, grid, s, a);
    case 2: return launch_sweep_p<DT, 2>(mode, grid, s, a);
    case 3: return launch_sweep_p<DT, 3>(mode, grid, s, a);
    case 4: return launch_sweep_p<DT, 4>(mode, grid, s, a);
    case 5: return launch_sweep_p<DT, 5>(mode, grid, s, a);
    case 6: return launch_sweep_p<DT, 6>(mode, grid, s, a);
    case 7: return launch_sweep_p<DT, 7>(mode, grid, s, a);
    default: return launch_sweep_p<DT, 8>(mode, grid, s, a);
    }
}

template <int DT, int P>
static cudaError_t launch_reduce_p(int mode, int grid, cudaStream_t s, const ReduceArgs &a)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: return launch_k(k_reduce_plain<DT, P, SIFAR_BARRIER_ONESHOT>, grid, s, a);
    case SIFAR_DUALBUF:         return launch_k(k_reduce_plain<DT, P, SIFAR_DUALBUF>, grid, s, a);
    case kModeTiles:            return launch_k(k_reduce_plain<DT, P, kModeTiles>, grid, s, a);
    default:                    return launch_k(k_reduce_spec<DT, P>, grid, s, a);
    }
}

template <int DT>
static cudaError_t launch_reduce_dt(int P, int mode, int grid, cudaStream_t s, const ReduceArgs &a)
{
    switch (P) {
    case 1: return launch_reduce_p<DT, 1>(mode, grid, s, a);
    case 2: return launch_reduce_p<DT, 2>(mode, grid, s, a);
    case 3: return launch_reduce_p<DT, 3>(mode, grid, s, a);
    case 4: return launch_reduce_p<DT, 4>(mode, grid, s, a);
    case 5: return launch_reduce_p<DT, 5>(mode, grid, s, a);
    case 6: return launch_reduce_p<DT, 6>(mode, grid, s, a);
    case 7: return launch_reduce_p<DT, 7>(mode, grid, s, a);
    default: return launch_reduce_p<DT, 8>(mode, grid, s, a);
    }
}

}  /* namespace sifar */

/* Polling shape from the number of (slot, rank) pairs a waiting grid re-polls per round (see validate_slot). */
sifar::PollShape sifar::poll_shape_for(const sifar_ctx *ctx, size_t n)
{
    const size_t pairs = slots_for(ctx->dtype, n) * (size_t)ctx->P;
    PollShape p;
    p.wide = pairs <= ctx->poll_wide_max ? 1u : 0u;
    p.pace_ns = pairs <= ctx->poll_pace_min ? 0u : ctx->poll_pace_ns;
    p.sentinel = pairs <= ctx->poll_sentinel_min ? 0u : 1u;
    p.forced = ctx->force_retries;
    return p;
}

static int unroll_for(int P) { return P <= 2 ? 4 : P <= 4 ? 2 : 1; }

/* 16-byte units the reducer works on: slots, or vectors of plain elements (kernel mode, see kModeTiles). */
static size_t reduce_units(const sifar_ctx *ctx, size_t n, int kernel_mode)
{
    return kernel_mode == SIFAR_SPECULATIVE ? sifar::slots_for(ctx->dtype, n)
                                            : n * sifar::elem_size(ctx->dtype) / 16;
}

/* The chains use the slot format at every size. */
size_t sifar::reduce_tiles(const sifar_ctx *ctx, size_t n, int mode)
{
    return tiles_for(reduce_units(ctx, n, mode), unroll_for(ctx->P));
}

/*
 * Format of the speculative mode by size.  Slots carry their own tags (no flag, no dependent round trip)
 * but move a third more bytes; from 8 MiB for all P partials together (1 MiB per rank at P = 8: where the plain
 * reducer overtakes the slot reducer on ready data on B200), where bandwidth is what counts,
 * the partial travels as plain data with one arrival flag per 16 KiB block.
 */
static int spec_format(int P, int dtype, size_t n)
{
    constexpr size_t kTilesFromBytes = (size_t)8 << 20;
    return (size_t)P * n * sifar::elem_size(dtype) < kTilesFromBytes ? SIFAR_FORMAT_SLOTS : SIFAR_FORMAT_TILES;
}

static size_t flag_blocks(int dtype, size_t n)
{
    const size_t nvec = n * sifar::elem_size(dtype) / 16;
    return nvec ? (nvec + sifar::kFlagBlockVecs - 1) / sifar::kFlagBlockVecs : 1;
}

namespace sifar {

int launch_reduce(sifar_ctx *ctx, const ReduceLaunch &rl, cudaStream_t stream)
{
    if (rl.n == 0) {
        k_empty_call<<<1, 1, 0, stream>>>(ctx->d_state, rl.mode, ctx->P);
        SIFAR_CUDA(cudaGetLastError());
        return SIFAR_OK;
    }
    const int kernel_mode = (rl.mode == SIFAR_SPECULATIVE && rl.format == SIFAR_FORMAT_TILES) ? kModeTiles : rl.mode;
    ReduceArgs a;
    memset(&a, 0, sizeof a);
    for (int r = 0; r < ctx->P; ++r) a.src[r] = reinterpret_cast<const uint4 *>(rl.src[r]);
    a.out = rl.out;
    a.n = rl.n;
    a.st = ctx->d_state;
    a.host_status = ctx->d_status_alias;
    a.timeout_ns = ctx->timeout_ns;
    a.parity = rl.parity;
    a.check_parity = 1u;
    a.poll = poll_shape_for(ctx, rl.n);
    a.defer = ctx->d_defer;
    a.spin_ns = ctx->spin_ns < ctx->timeout_ns ? ctx->spin_ns : ctx->timeout_ns;
    /* One tile per CTA.  Up to one CTA per SM the reducer cannot crowd out the producers and waits in
       place; beyond that it runs at full occupancy, waits briefly, and its last CTAs sweep up: one
       janitor per SM.  Two per SM swept faster, but with two waiting CTAs of this kernel on every SM a
       producer that became ready after the reducer had started was not given a single CTA slot until the
       reducer gave up (seen with every stream on a hardware queue of its own; one per SM never showed it). */
    const int U = unroll_for(ctx->P);
    const size_t ntiles = tiles_for(reduce_units(ctx, rl.n, kernel_mode), U);
    a.two_phase = ntiles > (size_t)ctx->sm_count ? 1u : 0u;
    a.janitors = (uint32_t)ctx->sm_count;
    if (a.janitors > ntiles) a.janitors = (uint32_t)ntiles;
    if (kernel_mode == kModeTiles) {
        /* a tile is kThreads * U vectors, a flag block kFlagBlockVecs = 4 * kThreads vectors */
        a.flags = rl.tile_flags;
        a.flag_shift = U == 1 ? 2u : U == 2 ? 1u : 0u;
    } else {
        a.flags = &ctx->d_state->arrive[rl.parity][0];
        a.flag_shift = 31u;
    }
    /* The call number: the host's own count, unless this launch is being captured into a graph, whose
       replays advance the number in device memory. */
    a.e_host = 0u;
    if (rl.e_host) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusActive;
        if (cudaStreamIsCapturing(stream, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) a.e_host = rl.e_host;
        else cudaGetLastError();
    }
    /* Early reads need programmatic launch to mean anything, and the baseline keeps the plain stream order. */
    a.pdl = (rl.early && g_pdl && !rl.programmatic_event) ? 1u : 0u;
    a.early = (a.pdl && (rl.mode != SIFAR_BARRIER_ONESHOT || g_barrier_early)) ? 1u : 0u;
    /* Large plain-format call whose producers run on other streams and have not all finished: their data
       may be late, and what the grid then queues is swept by a kernel of its own (see k_sweep) instead of
       the grid's janitors.  Not while capturing (a stream may not be queried then, and a graph's replays
       meet other conditions than its capture did). */
    a.sweeper = 0u;
    if (ctx->sweep_policy != SIFAR_SWEEP_NEVER && rl.early && a.e_host && !rl.programmatic_event &&
        kernel_mode != SIFAR_SPECULATIVE && ntiles >= (size_t)kSweepFromTilesPerSm * (size_t)ctx->sm_count) {
        if (ctx->sweep_policy == SIFAR_SWEEP_ALWAYS) a.sweeper = 1u;
        for (int r = 0; r < ctx->P && !a.sweeper; ++r) {
            /* a stream that is being captured may not be queried (the capture would be invalidated) */
            cudaStreamCaptureStatus cap = cudaStreamCaptureStatusActive;
            if (cudaStreamIsCapturing(ctx->prod_stream[r], &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) {
                cudaGetLastError();
                continue;
            }
            const cudaError_t q = cudaStreamQuery(ctx->prod_stream[r]);
            if (q == cudaErrorNotReady) a.sweeper = 1u;
            if (q != cudaSuccess) cudaGetLastError();          /* "not ready" is an answer, not an error */
        }
    }
    /* with the sweep kernel behind it the grid need not hold the machine for tiles that are not there yet */
    if (a.sweeper && a.spin_ns > kSweepSpinNs) a.spin_ns = kSweepSpinNs;
    g_programmatic_event = rl.programmatic_event;
    cudaError_t err = (ctx->dtype == SIFAR_BF16)
        ? launch_reduce_dt<SIFAR_BF16>(ctx->P, kernel_mode, (int)ntiles, stream, a)
        : launch_reduce_dt<SIFAR_F32>(ctx->P, kernel_mode, (int)ntiles, stream, a);
    if (err == cudaSuccess && a.sweeper) {
        const size_t groups = (ntiles + kSweepTiles - 1) / kSweepTiles;
        const int grid = (int)(groups < (size_t)ctx->sm_count ? groups : (size_t)ctx->sm_count);
        err = (ctx->dtype == SIFAR_BF16) ? launch_sweep_dt<SIFAR_BF16>(ctx->P, kernel_mode, grid, stream, a)
                                         : launch_sweep_dt<SIFAR_F32>(ctx->P, kernel_mode, grid, stream, a);
    }
    g_programmatic_event = nullptr;
    SIFAR_CUDA(err);
    return SIFAR_OK;
}

/*
 * With lazy module loading (the CUDA default) the first launch of a kernel loads its code, and that load
 * can wait for the device to become idle.  Producers are routinely launched for the first time while a
 * reducer is already polling for them, so such a launch would block on the host until the reducer gave
 * up.  Every kernel of a context's shape is therefore loaded when the context is created.
 */
template <typename K>
static cudaError_t preload(K kernel)
{
    cudaFuncAttributes at;
    return cudaFuncGetAttributes(&at, kernel);
}

template <int DT, int P>
static cudaError_t preload_reducers()
{
    cudaError_t e = preload(k_reduce_plain<DT, P, SIFAR_BARRIER_ONESHOT>);
    if (e == cudaSuccess) e = preload(k_reduce_plain<DT, P, SIFAR_DUALBUF>);
    if (e == cudaSuccess) e = preload(k_reduce_plain<DT, P, kModeTiles>);
    if (e == cudaSuccess) e = preload(k_reduce_spec<DT, P>);
    if (e == cudaSuccess) e = preload(k_sweep<DT, P, SIFAR_BARRIER_ONESHOT>);
    if (e == cudaSuccess) e = preload(k_sweep<DT, P, SIFAR_DUALBUF>);
    if (e == cudaSuccess) e = preload(k_sweep<DT, P, kModeTiles>);
    return e;
}

template <int DT>
static cudaError_t preload_dt(int P)
{
    cudaError_t e = cudaSuccess;
    switch (P) {
    case 1: e = preload_reducers<DT, 1>(); break;
    case 2: e = preload_reducers<DT, 2>(); break;
    case 3: e = preload_reducers<DT, 3>(); break;
    case 4: e = preload_reducers<DT, 4>(); break;
    case 5: e = preload_reducers<DT, 5>(); break;
    case 6: e = preload_reducers<DT, 6>(); break;
    case 7: e = preload_reducers<DT, 7>(); break;
    default: e = preload_reducers<DT, 8>(); break;
    }
    if (e == cudaSuccess) e = preload(k_pack<DT, SIFAR_BARRIER_ONESHOT>);
    if (e == cudaSuccess) e = preload(k_pack<DT, SIFAR_DUALBUF>);
    if (e == cudaSuccess) e = preload(k_pack<DT, SIFAR_SPECULATIVE>);
    if (e == cudaSuccess) e = preload(k_pack<DT, kModeTiles>);
    if (e == cudaSuccess) e = preload(k_pack_all<DT, SIFAR_BARRIER_ONESHOT>);
    if (e == cudaSuccess) e = preload(k_pack_all<DT, SIFAR_DUALBUF>);
    if (e == cudaSuccess) e = preload(k_pack_all<DT, SIFAR_SPECULATIVE>);
    if (e == cudaSuccess) e = preload(k_pack_all<DT, kModeTiles>);
    if (e == cudaSuccess) e = preload(k_arrive);
    if (e == cudaSuccess) e = preload(k_wait_writable);
    if (e == cudaSuccess) e = preload(k_empty_call);
    if (e == cudaSuccess) e = preload(k_set_epoch);
    return e;
}

cudaError_t preload_kernels(int dtype, int P)
{
    return dtype == SIFAR_BF16 ? preload_dt<SIFAR_BF16>(P) : preload_dt<SIFAR_F32>(P);
}

template <int DT>
static cudaError_t launch_pack_all_dt(int mode, dim3 grid, cudaStream_t s, const PackAllArgs &a)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: k_pack_all<DT, SIFAR_BARRIER_ONESHOT><<<grid, kThreads, 0, s>>>(a); break;
    case SIFAR_DUALBUF:         k_pack_all<DT, SIFAR_DUALBUF><<<grid, kThreads, 0, s>>>(a); break;
    case kModeTiles:            k_pack_all<DT, kModeTiles><<<grid, kThreads, 0, s>>>(a); break;
    default:                    k_pack_all<DT, SIFAR_SPECULATIVE><<<grid, kThreads, 0, s>>>(a); break;
    }
    return cudaGetLastError();
}

template <int DT>
static cudaError_t launch_pack_dt(int mode, int grid, cudaStream_t s, const PackArgs &a)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: k_pack<DT, SIFAR_BARRIER_ONESHOT><<<grid, kThreads, 0, s>>>(a); break;
    case SIFAR_DUALBUF:         k_pack<DT, SIFAR_DUALBUF><<<grid, kThreads, 0, s>>>(a); break;
    case kModeTiles:            k_pack<DT, kModeTiles><<<grid, kThreads, 0, s>>>(a); break;
    default:                    k_pack<DT, SIFAR_SPECULATIVE><<<grid, kThreads, 0, s>>>(a); break;
    }
    return cudaGetLastError();
}

}  /* namespace sifar */

using namespace sifar;

/* ------------------------------------------------------------------------ */
/* C ABI                                                                     */
/* ------------------------------------------------------------------------ */
static bool valid_mode(int m) { return m == SIFAR_BARRIER_ONESHOT || m == SIFAR_DUALBUF || m == SIFAR_SPECULATIVE; }
static bool valid_dtype(int d) { return d == SIFAR_BF16 || d == SIFAR_F32; }
static size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

extern "C" const char *sifar_last_error(void) { return g_error; }

extern "C" size_t sifar_slot_count(int dtype, size_t n)
{
    return valid_dtype(dtype) ? slots_for(dtype, n) : 0;
}

extern "C" size_t sifar_algorithmic_bytes(int P, int dtype, size_t n, int mode)
{
    if (!valid_dtype(dtype) || !valid_mode(mode) || P < 1) return 0;
    const size_t payload = n * elem_size(dtype);
    const bool slots = (mode == SIFAR_SPECULATIVE && spec_format(P, dtype, n) == SIFAR_FORMAT_SLOTS);
    const size_t per_rank = slots ? slots_for(dtype, n) * 16 : payload;
    size_t flags = 0;
    if (mode == SIFAR_SPECULATIVE && !slots) flags += (size_t)P * 4 * flag_blocks(dtype, n);   /* one flag per block */
    if (mode != SIFAR_SPECULATIVE) flags += (size_t)P * 4;          /* arrival flags */
    if (mode == SIFAR_BARRIER_ONESHOT) flags += (size_t)P * 4;      /* done flags    */
    return (size_t)P * per_rank + payload + flags;
}

extern "C" int sifar_spec_format(int P, int dtype, size_t n)
{
    if (P < 1 || P > kMaxRanks || !valid_dtype(dtype)) {
        set_error("sifar_spec_format: need 1 <= P <= %d and a known dtype", kMaxRanks);
        return SIFAR_ERR_INVALID;
    }
    return spec_format(P, dtype, n);
}

extern "C" sifar_ctx *sifar_create(int P, size_t max_elems, int dtype)
{
    g_error[0] = 0;
    if (P < 1 || P > kMaxRanks || max_elems == 0 || !valid_dtype(dtype)) {
        set_error("sifar_create: need 1 <= P <= %d, max_elems > 0, dtype in {0,1}", kMaxRanks);
        return nullptr;
    }
    if (max_elems > ((size_t)1 << 31)) {
        set_error("sifar_create: max_elems above 2^31 is not supported");
        return nullptr;
    }
    sifar_ctx *c = new (std::nothrow) sifar_ctx();
    if (!c) { set_error("sifar_create: out of host memory"); return nullptr; }
    memset(c, 0, sizeof *c);
    c->P = P; c->dtype = dtype; c->max_elems = max_elems;
    c->timeout_ns = 200000ull * 1000ull;
    c->poll_wide_max = 16384;
    c->spin_ns = 5000;
    c->sweep_policy = g_sweep ? SIFAR_SWEEP_AUTO : SIFAR_SWEEP_NEVER;
    if (const char *env = getenv("SIFAR_SPIN_NS")) c->spin_ns = strtoull(env, nullptr, 10);
    c->poll_pace_min = 16384;
    c->poll_sentinel_min = 16384;
    if (const char *env = getenv("SIFAR_POLL_SENTINEL_MIN")) c->poll_sentinel_min = (size_t)strtoull(env, nullptr, 10);
    c->poll_pace_ns = 0;
    if (const char *env = getenv("SIFAR_POLL_WIDE_MAX")) c->poll_wide_max = (size_t)strtoull(env, nullptr, 10);
    if (const char *env = getenv("SIFAR_POLL_PACE_MIN")) c->poll_pace_min = (size_t)strtoull(env, nullptr, 10);
    if (const char *env = getenv("SIFAR_POLL_PACE_NS")) c->poll_pace_ns = (uint32_t)strtoul(env, nullptr, 10);
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    /* kUnitPadBytes of slack: the persistent chain kernels work in whole warps of 16-byte units */
    c->plain_stride = round_up(max_elems * elem_size(dtype) + kUnitPadBytes, 256);
    c->slot_stride = round_up(slots_for(dtype, max_elems) * 16 + kUnitPadBytes, 256);
    const size_t plain_bytes = c->plain_stride * 2 * P, slot_bytes = c->slot_stride * 2 * P;
    if (e == cudaSuccess) e = cudaMalloc(&c->d_plain, plain_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_slots, slot_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_state, sizeof(DevState));
    const size_t defer_words = 2 + (slots_for(dtype, max_elems) + kThreads - 1) / kThreads;
    if (e == cudaSuccess) e = cudaMalloc(&c->d_defer, defer_words * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMemset(c->d_defer, 0, defer_words * sizeof(uint32_t));
    /* arrival flags of the flagged-tile format: one word per block, rank and parity; 0 = never valid */
    c->tflag_words = round_up((flag_blocks(dtype, max_elems) + 1) * kFlagStride, 32);
    const size_t tflag_bytes = c->tflag_words * 2 * sizeof(uint32_t);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_tflags, tflag_bytes);
    if (e == cudaSuccess) e = cudaMemset(c->d_tflags, 0, tflag_bytes);
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&c->h_status, sizeof(int), cudaHostAllocMapped);
    if (e == cudaSuccess) { *c->h_status = 0; e = cudaHostGetDevicePointer((void **)&c->d_status_alias, (void *)c->h_status, 0); }
    if (e == cudaSuccess) e = cudaMemset(c->d_plain, 0, plain_bytes);
    if (e == cudaSuccess) e = cudaMemset(c->d_slots, 0, slot_bytes);
    if (e == cudaSuccess) e = cudaMemset(c->d_state, 0, sizeof(DevState));
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->host_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = preload_kernels(dtype, P);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        set_error("sifar_create: %s", cudaGetErrorString(e));
        const bool nomem = (e == cudaErrorMemoryAllocation);
        cudaGetLastError();
        if (c->d_plain) cudaFree(c->d_plain);
        if (c->d_slots) cudaFree(c->d_slots);
        if (c->d_state) cudaFree(c->d_state);
        if (c->d_defer) cudaFree(c->d_defer);
        if (c->d_tflags) cudaFree(c->d_tflags);
        if (c->h_status) cudaFreeHost((void *)c->h_status);
        if (c->host_stream) cudaStreamDestroy(c->host_stream);
        delete c;
        (void)nomem;
        return nullptr;
    }
    return c;
}

extern "C" int sifar_destroy(sifar_ctx *c)
{
    if (!c) return SIFAR_OK;
    cudaSetDevice(c->device);
    cudaError_t e = cudaDeviceSynchronize();
    cudaFree(c->d_plain);
    cudaFree(c->d_slots);
    cudaFree(c->d_state);
    cudaFree(c->d_defer);
    cudaFree(c->d_tflags);
    if (c->d_stage_in) cudaFree(c->d_stage_in);
    if (c->d_stage_out) cudaFree(c->d_stage_out);
    cudaFreeHost((void *)c->h_status);
    cudaStreamDestroy(c->host_stream);
    delete c;
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
    return SIFAR_OK;
}

static int check_live(sifar_ctx *c, const char *fn)
{
    if (!c) { set_error("%s: NULL context", fn); return SIFAR_ERR_INVALID; }
    const int s = *c->h_status;
    if (s != 0) { set_error("%s: context carries device status %d; call sifar_reset", fn, s); return s; }
    return SIFAR_OK;
}

static int next_epoch(sifar_ctx *c, const char *fn, uint32_t *e)
{
    if (c->h_epoch >= kEpochLimit) {
        set_error("%s: call numbers exhausted; call sifar_reset", fn);
        return SIFAR_ERR_EPOCH;
    }
    *e = c->h_epoch + 1u;
    return SIFAR_OK;
}

static const void *ctx_buffer(const sifar_ctx *c, int mode, uint32_t e, int r)
{
    if (mode == SIFAR_BARRIER_ONESHOT) return c->plain_buf(0, r);
    if (mode == SIFAR_DUALBUF) return c->plain_buf((int)(e & 1u), r);
    return c->slot_buf((int)(e & 1u), r);
}

static size_t ctx_buffer_bytes(const sifar_ctx *c, int mode, size_t n)
{
    const bool slots = (mode == SIFAR_SPECULATIVE && spec_format(c->P, c->dtype, n) == SIFAR_FORMAT_SLOTS);
    return slots ? slots_for(c->dtype, n) * 16 : n * elem_size(c->dtype);
}

/* What sifar_pack / sifar_arrive remember about the producer of `rank` for call e. */
static void note_producer(sifar_ctx *c, int rank, uint32_t e, cudaStream_t stream, size_t n)
{
    c->prod_epoch[rank] = e;
    c->prod_stream[rank] = stream;
    c->prod_n[rank] = n;
}

static bool overlaps(const void *a, size_t na, const void *b, size_t nb)
{
    const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
    return x < y + nb && y < x + na;
}

extern "C" int sifar_allreduce(sifar_ctx *c, const void *const *rank_ptrs, void *out, size_t n, int mode,
                               void *stream)
{
    int rc = check_live(c, "sifar_allreduce");
    if (rc) return rc;
    if (!valid_mode(mode)) { set_error("sifar_allreduce: unknown mode %d", mode); return SIFAR_ERR_INVALID; }
    if (n > c->max_elems) { set_error("sifar_allreduce: n exceeds max_elems"); return SIFAR_ERR_INVALID; }
    if (n > 0 && (!out || ((uintptr_t)out & 15u))) {
        set_error("sifar_allreduce: out must be a 16-byte aligned device pointer");
        return SIFAR_ERR_INVALID;
    }
    uint32_t e;
    if ((rc = next_epoch(c, "sifar_allreduce", &e))) return rc;

    ReduceLaunch rl;
    memset(&rl, 0, sizeof rl);
    const size_t in_bytes = ctx_buffer_bytes(c, mode, n), out_bytes = n * elem_size(c->dtype);
    for (int r = 0; r < c->P; ++r) {
        const void *own = ctx_buffer(c, mode, e, r);
        const void *p = own;
        if (rank_ptrs) {
            p = rank_ptrs[r];
            if (mode != SIFAR_BARRIER_ONESHOT && p != own) {
                set_error("sifar_allreduce: rank_ptrs[%d] is not the context's buffer of this call", r);
                return SIFAR_ERR_INVALID;
            }
            if (!p || ((uintptr_t)p & 15u)) {
                set_error("sifar_allreduce: rank_ptrs[%d] must be a 16-byte aligned device pointer", r);
                return SIFAR_ERR_INVALID;
            }
        }
        if (n > 0 && overlaps(out, out_bytes, p, in_bytes)) {
            set_error("sifar_allreduce: out overlaps the buffer of rank %d", r);
            return SIFAR_ERR_INVALID;
        }
        rl.src[r] = p;
    }
    rl.out = out; rl.n = n; rl.mode = mode; rl.parity = e & 1u; rl.e_host = e;
    rl.format = (mode == SIFAR_SPECULATIVE) ? spec_format(c->P, c->dtype, n) : SIFAR_FORMAT_SLOTS;
    /* Where every rank's producer of this call is known to have been enqueued on another stream, nothing
       this reducer reads is produced by the kernel before it on its own stream, and its loads may start
       while that kernel drains (its writes still wait).  Unknown producers (partials stored by the
       caller's own kernels without sifar_arrive) or the same stream: the plain stream order. */
    rl.early = (stream != nullptr);
    for (int r = 0; r < c->P; ++r) {
        if (c->prod_epoch[r] != e) { rl.early = false; continue; }
        if (c->prod_stream[r] == (cudaStream_t)stream || c->prod_stream[r] == nullptr) rl.early = false;
        if (c->prod_n[r] != (size_t)-1 && c->prod_n[r] != n && mode == SIFAR_SPECULATIVE &&
            spec_format(c->P, c->dtype, c->prod_n[r]) != rl.format) {
            set_error("sifar_allreduce: rank %d was packed for %zu elements, whose speculative format differs "
                      "from that of n = %zu", r, c->prod_n[r], n);
            return SIFAR_ERR_INVALID;
        }
    }
    rl.tile_flags = c->tile_flags((int)(e & 1u));
    rc = launch_reduce(c, rl, (cudaStream_t)stream);
    if (rc) return rc;
    c->h_epoch = e;
    if (mode == SIFAR_BARRIER_ONESHOT) c->last_mode0_epoch = e;
    return SIFAR_OK;
}

extern "C" int sifar_rank_buffer(sifar_ctx *c, int rank, int mode, void **ptr, unsigned *epoch)
{
    if (!c) { set_error("sifar_rank_buffer: NULL context"); return SIFAR_ERR_INVALID; }
    if (rank < 0 || rank >= c->P || !valid_mode(mode)) {
        set_error("sifar_rank_buffer: bad rank or mode");
        return SIFAR_ERR_INVALID;
    }
    uint32_t e;
    int rc = next_epoch(c, "sifar_rank_buffer", &e);
    if (rc) return rc;
    if (ptr) *ptr = const_cast<void *>(ctx_buffer(c, mode, e, rank));
    if (epoch) *epoch = e;
    return SIFAR_OK;
}

extern "C" int sifar_tile_flags(sifar_ctx *c, int rank, void **flags, size_t *elems_per_flag, size_t *stride_words)
{
    if (!c || rank < 0 || rank >= c->P) { set_error("sifar_tile_flags: NULL context or bad rank"); return SIFAR_ERR_INVALID; }
    uint32_t e;
    int rc = next_epoch(c, "sifar_tile_flags", &e);
    if (rc) return rc;
    if (flags) *flags = c->tile_flags((int)(e & 1u)) + rank;
    if (elems_per_flag) *elems_per_flag = kFlagBlockVecs * 16 / elem_size(c->dtype);
    if (stride_words) *stride_words = kFlagStride;
    return SIFAR_OK;
}

extern "C" int sifar_pack(sifar_ctx *c, int rank, const void *src, size_t n, int mode, void *stream)
{
    int rc = check_live(c, "sifar_pack");
    if (rc) return rc;
    if (rank < 0 || rank >= c->P || !valid_mode(mode) || n > c->max_elems) {
        set_error("sifar_pack: bad rank, mode or n");
        return SIFAR_ERR_INVALID;
    }
    if (n > 0 && (!src || ((uintptr_t)src & 15u))) {
        set_error("sifar_pack: src must be a 16-byte aligned device pointer");
        return SIFAR_ERR_INVALID;
    }
    uint32_t e;
    if ((rc = next_epoch(c, "sifar_pack", &e))) return rc;
    PackArgs a;
    memset(&a, 0, sizeof a);
    a.src = src;
    a.dst = const_cast<void *>(ctx_buffer(c, mode, e, rank));
    a.n = n;
    a.st = c->d_state;
    a.host_status = c->d_status_alias;
    a.timeout_ns = c->timeout_ns;
    a.rank = (uint32_t)rank;
    a.parity = e & 1u;
    a.wait_delta = (mode == SIFAR_BARRIER_ONESHOT && c->last_mode0_epoch) ? e - c->last_mode0_epoch : 0u;
    a.tile_flags = c->tile_flags((int)(e & 1u));
    const int kernel_mode = (mode == SIFAR_SPECULATIVE && spec_format(c->P, c->dtype, n) == SIFAR_FORMAT_TILES)
                                ? kModeTiles : mode;
    const size_t units = (kernel_mode == SIFAR_SPECULATIVE) ? slots_for(c->dtype, n)
                                                            : (n * elem_size(c->dtype) + 15) / 16;
    size_t grid = (kernel_mode == kModeTiles) ? flag_blocks(c->dtype, n) : (units + kThreads - 1) / kThreads;
    /* two CTAs per SM: the P ranks pack at the same time on their own streams (measured: 5.4-5.5 TB/s for eight
       ranks together; four or eight CTAs per SM were slower together and little faster alone) */
    const size_t cap = (size_t)c->sm_count * 2;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    cudaError_t err = (c->dtype == SIFAR_BF16)
        ? launch_pack_dt<SIFAR_BF16>(kernel_mode, (int)grid, (cudaStream_t)stream, a)
        : launch_pack_dt<SIFAR_F32>(kernel_mode, (int)grid, (cudaStream_t)stream, a);
    SIFAR_CUDA(err);
    note_producer(c, rank, e, (cudaStream_t)stream, n);
    return SIFAR_OK;
}

extern "C" int sifar_arrive(sifar_ctx *c, int rank, int mode, void *stream)
{
    int rc = check_live(c, "sifar_arrive");
    if (rc) return rc;
    if (rank < 0 || rank >= c->P || (mode != SIFAR_BARRIER_ONESHOT && mode != SIFAR_DUALBUF)) {
        set_error("sifar_arrive: bad rank, or a mode without arrival flags");
        return SIFAR_ERR_INVALID;
    }
    uint32_t e;
    if ((rc = next_epoch(c, "sifar_arrive", &e))) return rc;
    k_arrive<<<1, 1, 0, (cudaStream_t)stream>>>(c->d_state, c->d_status_alias, (uint32_t)rank, e & 1u);
    SIFAR_CUDA(cudaGetLastError());
    note_producer(c, rank, e, (cudaStream_t)stream, (size_t)-1);
    return SIFAR_OK;
}

extern "C" int sifar_wait_writable(sifar_ctx *c, int rank, void *stream)
{
    int rc = check_live(c, "sifar_wait_writable");
    if (rc) return rc;
    if (rank < 0 || rank >= c->P) { set_error("sifar_wait_writable: bad rank"); return SIFAR_ERR_INVALID; }
    if (!c->last_mode0_epoch) return SIFAR_OK;      /* nothing has read the buffer yet */
    const uint32_t delta = c->h_epoch + 1u - c->last_mode0_epoch;
    k_wait_writable<<<1, 1, 0, (cudaStream_t)stream>>>(c->d_state, c->d_status_alias, (uint32_t)rank, delta,
                                                       (c->h_epoch + 1u) & 1u, c->timeout_ns);
    SIFAR_CUDA(cudaGetLastError());
    return SIFAR_OK;
}

extern "C" int sifar_status(sifar_ctx *c)
{
    if (!c) { set_error("sifar_status: NULL context"); return SIFAR_ERR_INVALID; }
    return *c->h_status;
}

extern "C" int sifar_get_stats(sifar_ctx *c, unsigned long long out[8])
{
    if (!c || !out) { set_error("sifar_get_stats: NULL argument"); return SIFAR_ERR_INVALID; }
    DevState h;
    SIFAR_CUDA(cudaDeviceSynchronize());
    SIFAR_CUDA(cudaMemcpy(&h, c->d_state, sizeof h, cudaMemcpyDeviceToHost));
    for (int i = 0; i < 5; ++i) out[i] = h.stats[i];
    out[5] = h.epoch; out[6] = 0; out[7] = 0;
    return SIFAR_OK;
}

extern "C" int sifar_set_timeout_us(sifar_ctx *c, unsigned us)
{
    if (!c || us == 0) { set_error("sifar_set_timeout_us: NULL context or zero"); return SIFAR_ERR_INVALID; }
    c->timeout_ns = (unsigned long long)us * 1000ull;
    return SIFAR_OK;
}

extern "C" int sifar_reset(sifar_ctx *c, void *stream)
{
    if (!c) { set_error("sifar_reset: NULL context"); return SIFAR_ERR_INVALID; }
    cudaStream_t s = (cudaStream_t)stream;
    SIFAR_CUDA(cudaDeviceSynchronize());
    SIFAR_CUDA(cudaMemsetAsync(c->d_slots, 0, c->slot_stride * 2 * c->P, s));
    SIFAR_CUDA(cudaMemsetAsync(c->d_state, 0, sizeof(DevState), s));
    SIFAR_CUDA(cudaMemsetAsync(c->d_defer, 0, sizeof(uint32_t), s));
    SIFAR_CUDA(cudaMemsetAsync(c->d_tflags, 0, c->tflag_words * 2 * sizeof(uint32_t), s));
    SIFAR_CUDA(cudaStreamSynchronize(s));
    *c->h_status = 0;
    c->h_epoch = 0;
    c->last_mode0_epoch = 0;
    memset(c->prod_epoch, 0, sizeof c->prod_epoch);
    return SIFAR_OK;
}

extern "C" int sifar_debug_set_epoch(sifar_ctx *c, unsigned calls_so_far)
{
    if (!c) { set_error("sifar_debug_set_epoch: NULL context"); return SIFAR_ERR_INVALID; }
    SIFAR_CUDA(cudaDeviceSynchronize());
    k_set_epoch<<<1, 1>>>(c->d_state, calls_so_far);
    SIFAR_CUDA(cudaGetLastError());
    SIFAR_CUDA(cudaDeviceSynchronize());
    c->h_epoch = calls_so_far;
    c->last_mode0_epoch = 0;
    memset(c->prod_epoch, 0, sizeof c->prod_epoch);
    return SIFAR_OK;
}

extern "C" int sifar_debug_sweep_policy(sifar_ctx *c, int policy)
{
    if (!c) { set_error("sifar_debug_sweep_policy: NULL context"); return SIFAR_ERR_INVALID; }
    if (policy < SIFAR_SWEEP_NEVER || policy > SIFAR_SWEEP_ALWAYS) {
        set_error("sifar_debug_sweep_policy: unknown policy %d", policy);
        return SIFAR_ERR_INVALID;
    }
    c->sweep_policy = policy;
    return SIFAR_OK;
}

extern "C" int sifar_debug_force_retries(sifar_ctx *c, unsigned rounds)
{
    if (!c) { set_error("sifar_debug_force_retries: NULL context"); return SIFAR_ERR_INVALID; }
    if (rounds > 64u) { set_error("sifar_debug_force_retries: at most 64 rounds"); return SIFAR_ERR_INVALID; }
    c->force_retries = rounds;
    return SIFAR_OK;
}

/* Device-usable address of a host pointer if it is pinned (or otherwise reachable from the GPU), else NULL. */
static void *device_view(const void *p)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeManaged || at.type == cudaMemoryTypeDevice)
        return at.devicePointer;
    return nullptr;
}

extern "C" int sifar_allreduce_host(sifar_ctx *c, const void *const *host_rank_ptrs, void *host_out, size_t n,
                                    int mode)
{
    int rc = check_live(c, "sifar_allreduce_host");
    if (rc) return rc;
    if (!valid_mode(mode) || n > c->max_elems || !host_rank_ptrs || (n > 0 && !host_out)) {
        set_error("sifar_allreduce_host: bad mode, n or pointer");
        return SIFAR_ERR_INVALID;
    }
    for (int r = 0; r < c->P; ++r)
        if (!host_rank_ptrs[r]) { set_error("sifar_allreduce_host: NULL rank pointer"); return SIFAR_ERR_INVALID; }
    cudaStream_t s = c->host_stream;
    const size_t bytes = n * elem_size(c->dtype);

    /* Fast path: every partial is pinned host memory the GPU can read in place.  One kernel packs all P
       ranks straight from host memory (the H2D transfer happens inside that kernel), one reduces. */
    PackAllArgs all;
    memset(&all, 0, sizeof all);
    bool direct = (n > 0);
    for (int r = 0; r < c->P && direct; ++r) {
        void *d = device_view(host_rank_ptrs[r]);
        direct = d && (((uintptr_t)d & 15u) == 0);
        all.src[r] = d;
    }
    if (direct) {
        uint32_t e;
        if ((rc = next_epoch(c, "sifar_allreduce_host", &e))) return rc;
        for (int r = 0; r < c->P; ++r) all.dst[r] = const_cast<void *>(ctx_buffer(c, mode, e, r));
        all.common.tile_flags = c->tile_flags((int)(e & 1u));
        const int kernel_mode = (mode == SIFAR_SPECULATIVE && spec_format(c->P, c->dtype, n) == SIFAR_FORMAT_TILES)
                                    ? kModeTiles : mode;
        all.common.n = n;
        all.common.st = c->d_state;
        all.common.host_status = c->d_status_alias;
        all.common.timeout_ns = c->timeout_ns;
        all.common.parity = e & 1u;
        all.common.wait_delta = (mode == SIFAR_BARRIER_ONESHOT && c->last_mode0_epoch) ? e - c->last_mode0_epoch : 0u;
        const size_t units = (kernel_mode == SIFAR_SPECULATIVE) ? slots_for(c->dtype, n) : (bytes + 15) / 16;
        size_t gx = (kernel_mode == kModeTiles) ? flag_blocks(c->dtype, n) : (units + kThreads - 1) / kThreads;
        const size_t cap = (size_t)c->sm_count * 2;
        if (gx > cap) gx = cap;
        cudaError_t err = (c->dtype == SIFAR_BF16)
            ? launch_pack_all_dt<SIFAR_BF16>(kernel_mode, dim3((unsigned)gx, (unsigned)c->P), s, all)
            : launch_pack_all_dt<SIFAR_F32>(kernel_mode, dim3((unsigned)gx, (unsigned)c->P), s, all);
        SIFAR_CUDA(err);
        for (int r = 0; r < c->P; ++r) note_producer(c, r, e, s, n);
        void *out_dev = device_view(host_out);
        if (out_dev && ((uintptr_t)out_dev & 15u) == 0) {
            if ((rc = sifar_allreduce(c, nullptr, out_dev, n, mode, s))) return rc;     /* result written in place */
        } else {
            if (!c->d_stage_out) {
                cudaError_t e2 = cudaMalloc(&c->d_stage_out, c->plain_stride);
                if (e2 != cudaSuccess) { cudaGetLastError(); set_error("sifar_allreduce_host: staging allocation failed"); return SIFAR_ERR_NOMEM; }
            }
            if ((rc = sifar_allreduce(c, nullptr, c->d_stage_out, n, mode, s))) return rc;
            SIFAR_CUDA(cudaMemcpyAsync(host_out, c->d_stage_out, bytes, cudaMemcpyDeviceToHost, s));
        }
        SIFAR_CUDA(cudaStreamSynchronize(s));
        rc = *c->h_status;
        if (rc) set_error("sifar_allreduce_host: device status %d", rc);
        return rc;
    }

    /* General path: pageable host memory goes through staging buffers allocated on first use. */
    const size_t stride = c->plain_stride;
    if (!c->d_stage_in) {
        cudaError_t e = cudaMalloc(&c->d_stage_in, stride * c->P);
        if (e == cudaSuccess && !c->d_stage_out) e = cudaMalloc(&c->d_stage_out, stride);
        if (e != cudaSuccess) {
            if (c->d_stage_in) { cudaFree(c->d_stage_in); c->d_stage_in = nullptr; }
            cudaGetLastError();
            set_error("sifar_allreduce_host: staging allocation failed: %s", cudaGetErrorString(e));
            return SIFAR_ERR_NOMEM;
        }
    }
    for (int r = 0; r < c->P; ++r) {
        if (bytes) SIFAR_CUDA(cudaMemcpyAsync(c->d_stage_in + r * stride, host_rank_ptrs[r], bytes, cudaMemcpyHostToDevice, s));
        if ((rc = sifar_pack(c, r, c->d_stage_in + r * stride, n, mode, s))) return rc;
    }
    if ((rc = sifar_allreduce(c, nullptr, c->d_stage_out, n, mode, s))) return rc;
    if (bytes) SIFAR_CUDA(cudaMemcpyAsync(host_out, c->d_stage_out, bytes, cudaMemcpyDeviceToHost, s));
    SIFAR_CUDA(cudaStreamSynchronize(s));
    rc = *c->h_status;
    if (rc) set_error("sifar_allreduce_host: device status %d", rc);
    return rc;
}
