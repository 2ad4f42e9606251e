/*
 * sifar_workload.cu - synthetic decode-step chains around the all-reduce:
 * seeded producer kernels, and the three ways a chain of dependent
 * {P producers -> all-reduce} steps runs on the device (streams + events, one
 * CUDA graph, one cooperative persistent kernel).
 *
 * The persistent kernel is the analogue of measuring all-reduces back to back
 * inside a fused forward-pass kernel (paper, Sections 4.2 "Megakernel
 * Integration" and 6.1): no launch or graph-edge latency separates the steps, so
 * what differs between the modes is exactly the synchronization they perform:
 *
 *   BARRIER_ONESHOT : take -> [done wait] produce -> arrival flag -> flag poll
 *                     -> load/sum -> hand over, the chunk's P done flags
 *   DUALBUF         : take -> produce -> arrival flag -> flag poll -> load/sum -> hand over
 *   SPECULATIVE     : take -> produce tagged slots -> load/validate/sum -> hand over
 *
 * where "hand over / take" is how a result reaches the next step's producers.  It
 * models ordinary same-GPU operator ordering and comes in two forms chosen by
 * size: tagged 16-byte stores polled by the thread that needs them (see
 * handoff_store), or, for grids whose polling threads would get in the way of the
 * stores they wait for, one result-ready flag per chunk.  With both barriers the
 * chunk's done flags (bottom barrier) hand the result over as well: they are
 * released after the result stores.  Every arrow is one dependent trip through the L2.
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

constexpr int kModeNoAllreduce = SIFAR_CHAIN_NO_ALLREDUCE;
constexpr unsigned kMaxDelayNs = 1000000u;       /* producer delays are capped at 1 ms */
constexpr size_t kConcurrentTiles = 48;          /* see sifar_chain::concurrent */

/* ------------------------------------------------------------------------ */
/* producer kernel of the stream / graph chains                              */
/* ------------------------------------------------------------------------ */
struct ProduceArgs {
    DevState *st;
    int *host_status;
    unsigned long long timeout_ns;
    sifar_workload w;
    uint32_t rank;
    unsigned long long n;
    const void *prev;          /* out^{t-1} (or the rank's own previous partial without all-reduce) */
    void *dst;                 /* the rank's buffer of this step                                    */
    uint32_t base_epoch;       /* step t = call number - base_epoch                                 */
    uint32_t parity;
    uint32_t t_fixed;          /* no-all-reduce chains: the step, since no call number advances     */
};

constexpr int kProdThreads = 128;

template <int DT, int MODE>
__global__ void __launch_bounds__(kProdThreads) k_produce(const ProduceArgs a)
{
    DevState *st = a.st;
    __shared__ uint32_t s_e, s_t, s_guess;
    constexpr int NW = (MODE == SIFAR_SPECULATIVE) ? 3 : 4;
    constexpr int EPU = NW * ((DT == SIFAR_BF16) ? 2 : 1);
    const size_t tid = (size_t)blockIdx.x * kProdThreads + threadIdx.x;
    const size_t nthreads = (size_t)gridDim.x * kProdThreads;
    /*
     * The kernel may be resident before the all-reduce it follows has finished (that all-reduce fires the step's
     * event as soon as its CTAs have started).  The step number is known even then: the call number read now is
     * the previous call's or the one before it, and the parity of this call is fixed at launch.  So the seeded
     * half of the thread's first unit is computed ahead of the dependency wait, as in the persistent kernel.
     */
    if (threadIdx.x == 0) {
        uint32_t tg = a.t_fixed;
        if (MODE != kModeNoAllreduce) {
            const uint32_t seen = ld_relaxed_u32(&st->epoch);
            tg = (((seen + 1u) & 1u) == a.parity ? seen + 1u : seen + 2u) - a.base_epoch;
        }
        s_guess = tg;
    }
    __syncthreads();
    const uint32_t t_ahead = s_guess;
    float z0[EPU];
    {
        const Gen g0 = make_gen(a.w, a.rank, t_ahead);
        if (tid * EPU < (size_t)a.n) {
            unit_noise<DT, NW>(g0, t_ahead == 1u, tid * EPU, (size_t)a.n, z0);
#pragma unroll
            for (int k = 0; k < EPU; ++k) asm volatile("" : "+f"(z0[k]));     /* keep it above the wait */
        }
    }
    /* if the all-reduce before this operation released its dependents early, wait here for its completion */
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0) {
        uint32_t e = 0, t = a.t_fixed;
        bool ok = true;
        if (MODE != kModeNoAllreduce) {
            const uint2 es = ld_relaxed_u32x2(&st->epoch);
            e = es.x + 1u;
            t = e - a.base_epoch;
            ok = (es.y == 0u);
            if (ok && MODE != SIFAR_BARRIER_ONESHOT && (e & 1u) != a.parity) {
                fail(st, a.host_status, SIFAR_ERR_EPOCH);
                ok = false;
            }
            /* bottom barrier, producer side: the single buffer may be overwritten once its last reader is done */
            if (ok && MODE == SIFAR_BARRIER_ONESHOT && t > 1u &&
                wait_flag_ge(&st->done[a.rank], e - 1u, a.timeout_ns) < 0) {
                fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
                ok = false;
            }
        }
        if (ok) spin_ns(gen_delay_ns(a.w, a.rank, t));
        s_e = ok ? (MODE == kModeNoAllreduce ? 1u : e) : 0u;
        s_t = t;
    }
    __syncthreads();
    const uint32_t e = s_e, t = s_t;
    if (e == 0u) return;

    const Gen g = make_gen(a.w, a.rank, t);
    const bool first = (t == 1u);
    const size_t n = (size_t)a.n;
    const bool ahead_ok = (t == t_ahead);              /* always, unless the context was used against its contract */
    if constexpr (MODE == SIFAR_SPECULATIVE) {
        constexpr int EPS = EPU;
        const size_t nslots = (n + EPS - 1) / EPS;
        for (size_t s = tid; s < nslots; s += nthreads) {
            uint32_t w[3];
            if (s == tid && ahead_ok) unit_combine<DT, 3>(g, first, a.prev, s * EPS, n, z0, w);
            else produce_words<DT, 3>(g, first, a.prev, s * EPS, n, w);
            store_slot(reinterpret_cast<uint4 *>(a.dst), s, w[0], w[1], w[2], e);
        }
    } else {
        constexpr int EPV = EPU;
        const size_t nvec = (n + EPV - 1) / EPV;       /* the last vector is zero-padded inside the context's buffer */
        for (size_t v = tid; v < nvec; v += nthreads) {
            uint32_t w[4];
            if (v == tid && ahead_ok) unit_combine<DT, 4>(g, first, a.prev, v * EPV, n, z0, w);
            else produce_words<DT, 4>(g, first, a.prev, v * EPV, n, w);
            st_slot(reinterpret_cast<uint4 *>(a.dst) + v, make_uint4(w[0], w[1], w[2], w[3]));
        }
        if (MODE != kModeNoAllreduce)
            signal_arrival(&st->pack_count[a.rank], gridDim.x, &st->arrive[e & 1u][a.rank], e);
    }
}

/* Generator probes: plain elements to dst, no protocol. */
template <int DT>
__global__ void k_probe(sifar_workload w, uint32_t rank, uint32_t t, const void *prev, void *dst, unsigned long long n)
{
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
    const Gen g = make_gen(w, rank, t);
    const size_t nvec = ((size_t)n + EPV - 1) / EPV;
    for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += (size_t)gridDim.x * blockDim.x) {
        uint32_t wds[4];
        produce_words<DT, 4>(g, t == 1u, prev, v * EPV, (size_t)n, wds);
        store_vec_result<DT>(dst, v, (size_t)n, make_uint4(wds[0], wds[1], wds[2], wds[3]));
    }
}

__global__ void k_delays(sifar_workload w, int P, uint32_t t, unsigned *out)
{
    if ((int)threadIdx.x < P) out[threadIdx.x] = gen_delay_ns(w, threadIdx.x, t);
}

__global__ void k_spin(unsigned ns) { spin_ns(ns); }

/*
 * Fused-producer stand-ins for tests: they store a part of a rank's partial the way a caller's own kernel
 * would, with the device helpers of sifar_device.cuh (store_slot; plain stores + signal_block).
 */
template <int DT>
__global__ void k_store_slots(const void *src, uint4 *slots, unsigned long long first, unsigned long long count,
                              unsigned long long n, uint32_t tag)
{
    constexpr int EPS = (DT == SIFAR_BF16) ? 6 : 3;
    for (size_t s = first + (size_t)blockIdx.x * blockDim.x + threadIdx.x; s < first + count;
         s += (size_t)gridDim.x * blockDim.x) {
        uint32_t w[3] = {0u, 0u, 0u};
        for (int k = 0; k < EPS && s * EPS + k < n; ++k) {
            if (DT == SIFAR_BF16)
                w[k >> 1] |= (uint32_t)reinterpret_cast<const uint16_t *>(src)[s * EPS + k] << ((k & 1) * 16);
            else
                w[k] = reinterpret_cast<const uint32_t *>(src)[s * EPS + k];
        }
        store_slot(slots, s, w[0], w[1], w[2], tag);
    }
}

/* One CTA per flag block: plain 16-byte stores of the block's elements, then the block's flag. */
template <int DT>
__global__ void k_store_blocks(const void *src, void *dst, uint32_t *flags, unsigned long long stride_words,
                               unsigned long long first, unsigned long long n, uint32_t tag)
{
    constexpr size_t EPV = (DT == SIFAR_BF16) ? 8 : 4;
    const size_t esz = 16 / EPV;
    const size_t b = first + blockIdx.x;
    const size_t nvec = (size_t)n / EPV;
    const size_t nblocks = nvec ? (nvec + kFlagBlockVecs - 1) / kFlagBlockVecs : 1;
    for (size_t v = b * kFlagBlockVecs + threadIdx.x; v < (b + 1) * kFlagBlockVecs && v < nvec; v += blockDim.x)
        st_slot(reinterpret_cast<uint4 *>(dst) + v, reinterpret_cast<const uint4 *>(src)[v]);
    if (b == nblocks - 1)                           /* the ragged tail travels with the last block */
        for (size_t i = nvec * EPV + threadIdx.x; i < (size_t)n; i += blockDim.x)
            memcpy(reinterpret_cast<char *>(dst) + i * esz, reinterpret_cast<const char *>(src) + i * esz, esz);
    signal_block(flags, (size_t)stride_words, b, tag);
}

/* ------------------------------------------------------------------------ */
/* persistent chain kernel                                                   */
/* ------------------------------------------------------------------------ */
struct __align__(128) ChunkFlags {
    uint32_t ready;                 /* call number whose result chunk is published (flag form of the hand-over) */
    uint32_t pad0[7];
    uint32_t arrive[2][8];          /* per parity, per rank: this chunk of the rank's partial stored */
    uint32_t done[8];               /* per rank: the chunk's reducer has finished reading call e (bottom barrier) */
};

struct __align__(128) ChainDev {
    uint32_t exit_count;            /* CTAs that left the kernel (monotonic)                        */
    uint32_t seen[3];               /* written by CTA 0 of the last run: role layout (1 = clustered), CTAs per
                                       cluster as the hardware reports them, form of the hand-over (1 = tagged) */
    uint32_t pad0[28];
};

struct PersistArgs {
    DevState *st;
    int *host_status;
    unsigned long long timeout_ns;
    sifar_workload w;
    unsigned long long n;
    char *plain;                    /* [parity][rank] plain buffers */
    unsigned long long plain_stride;
    char *slots;                    /* [parity][rank] slot buffers  */
    unsigned long long slot_stride;
    char *ring;
    unsigned long long ring_stride;
    uint32_t ring_len;
    uint32_t e0;                    /* calls completed before this run     */
    uint32_t base_epoch;
    uint32_t steps;
    uint32_t C;                     /* chunks = reducer CTAs               */
    uint32_t K;                     /* units per thread and step           */
    uint32_t exit_base;
    uint32_t clustered;             /* role layout, see k_chain */
    PollShape poll;
    ChainDev *cs;
    ChunkFlags *chunks;
    unsigned long long *stamps;     /* C x (steps + 1): per chunk, start of the run and every published result */
    unsigned long long *trace;      /* NULL, or steps x kTraceSlots phase stamps of chunk 0 (see sifar_workload.h) */
    uint32_t *retry_steps;          /* steps: 1 if any CTA re-loaded a slot in that step */
    uint4 *handoff;                 /* [parity][unit]: the result as the next producers take it over (see
                                       handoff_store), or NULL: one result-ready flag per chunk instead */
    unsigned long long handoff_stride;   /* 16-byte words per parity */
};

/*
 * Hand-over of a result unit from the chunk's reducer to the P producers of the next step.  The next operation
 * of a rank consumes the all-reduce result on the same GPU (Section 3.1: stream order there); in this one-reader
 * emulation reducer and producers are different CTAs, so the result has to cross.  It crosses the way the partials
 * do in the speculative mode: data and call number in one 16-byte store, validated by the reader, who polls the
 * unit it needs and nothing else - no CTA-wide barrier, no fence, no flag, no second round trip for the data.
 * The other form, one ready flag per chunk (barrier, release; acquire poll by thread 0, barrier, then the loads),
 * costs 0.3-1.0 us more per step at decode payloads in the two barrier-free modes; it is kept for large grids
 * (more than kHandoffMaxPairs polling threads), where eight times as many threads polling data lines as there
 * are units slowed the reducers' stores more than the flag costs (measured at P = 8: 256 KB per rank 7.8 against
 * 7.3 us, 512 KB per rank 14.2 against 11.7 us mean).  With both barriers neither form is needed: the done flags
 * of the bottom barrier follow the result stores.  The chain without all-reduce uses the words too: every rank
 * hands its partial to itself.
 * NW = 3 result words (a 12-byte unit: speculative mode, chain without all-reduce): {w0, w1, w2, tag}.  NW = 4
 * (a 16-byte vector of the dual-buffered mode): two stores {w0, tag, w1, tag}, {w2, tag, w3, tag}, each valid by
 * itself.
 */
template <int NW>
__device__ __forceinline__ void handoff_store(uint4 *base, size_t u, const uint4 &v, uint32_t tag)
{
    if (NW == 3) {
        st_slot(base + u, make_uint4(v.x, v.y, v.z, tag));
    } else {
        st_slot(base + 2 * u, make_uint4(v.x, tag, v.y, tag));
        st_slot(base + 2 * u + 1, make_uint4(v.z, tag, v.w, tag));
    }
}

/* Polls until unit u carries `tag` (bounded; also gives up when the context already carries an error). */
template <int NW>
__device__ __forceinline__ bool handoff_wait(const uint4 *base, size_t u, uint32_t tag, uint32_t (&w)[NW], DevState *st,
                                             int *host_status, unsigned long long timeout_ns)
{
    Deadline d;
    for (;;) {
        if (NW == 3) {
            const uint4 a = ld_slot(base + u);
            if (a.w == tag) { w[0] = a.x; w[1] = a.y; w[2] = a.z; return true; }
        } else {
            const uint4 a = ld_slot(base + 2 * u), b = ld_slot(base + 2 * u + 1);
            if (a.y == tag && a.w == tag && b.y == tag && b.w == tag) {
                w[0] = a.x; w[1] = a.z; w[2] = b.x; w[NW - 1] = b.z;
                return true;
            }
        }
        if (d.expired(timeout_ns)) { fail(st, host_status, SIFAR_ERR_TIMEOUT); return false; }
        if ((d.polls % 64u) == 0u && ld_relaxed_u32(&st->status) != 0u) return false;
    }
}

constexpr size_t kHandoffMaxPairs = 100000;
constexpr size_t kChainClusterMaxPairs = 50000;  /* one thread-block cluster per chunk up to here, see chain_setup_persistent */
constexpr size_t kChainWideMaxPairs = 50000;    /* speculative chain with tagged hand-over: wide polling up to here, sentinel above */      /* (unit, rank) pairs up to which the result is handed over in tagged words */
constexpr int kChainThreads = 128;
constexpr int kPreUnits = 4;            /* units per producer thread, beyond its first, whose seeded half is computed before the wait */
constexpr int kTraceSlots = 48;         /* 0-3 reducer, 4 + 3r .. 6 + 3r rank r's producer, 28 done flags */

template <int DT, int P, int MODE, bool TRACE, bool TAGGED>
__global__ void __launch_bounds__(kChainThreads, 6) k_chain(const PersistArgs a)
{
    DevState *st = a.st;
    const uint32_t C = a.C;
    const bool no_ar = (MODE == kModeNoAllreduce);
    /*
     * Roles.  Clustered layout: the CTAs that own one chunk (its reducer and its P producers) are consecutive
     * and launched as one thread-block cluster, which the hardware places inside one GPC, so their flag
     * and slot traffic stays on one die.  Nothing else of the cluster is used: all communication still
     * goes through global memory.  Flat layout: reducers first, then the producers rank by rank.
     */
    const uint32_t roles = no_ar ? (uint32_t)P : (uint32_t)P + 1u;
    bool is_reducer;
    uint32_t rank, chunk;
    if (a.clustered) {
        const uint32_t role = blockIdx.x % roles;
        chunk = blockIdx.x / roles;
        is_reducer = !no_ar && role == 0u;
        rank = no_ar ? role : (is_reducer ? 0u : role - 1u);
    } else {
        is_reducer = !no_ar && blockIdx.x < C;
        const uint32_t pidx = no_ar ? blockIdx.x : blockIdx.x - C;
        rank = is_reducer ? 0u : pidx / C;
        chunk = is_reducer ? blockIdx.x : pidx % C;
    }
    ChunkFlags *cf = a.chunks + chunk;
    const size_t n = (size_t)a.n;
    /* 12-byte units where the unit travels with a tag in one 16-byte word (speculative slots; the chain without
       all-reduce, whose ranks hand their partial over to themselves the same way), else 16-byte vectors */
    constexpr bool kSlotUnits = (MODE == SIFAR_SPECULATIVE || MODE == kModeNoAllreduce);
    constexpr int EPU = kSlotUnits ? ((DT == SIFAR_BF16) ? 6 : 3) : ((DT == SIFAR_BF16) ? 8 : 4);
    /* Whole warps of units: a warp of which only some lanes have a unit was measured up to 0.4 us per step slower
       (the ragged last chunk then set the pace of the whole result).  Units past the last element carry zeros;
       the rank buffers and the ring rows have room for them. */
    const size_t nunits = ((n + EPU - 1) / EPU + 31) / 32 * 32;
    const size_t n_io = nunits * EPU;         /* ring rows are padded: whole units are read and written */
    const size_t unit0 = (size_t)chunk * kChainThreads * a.K + threadIdx.x;
    __shared__ int s_ok;
    __shared__ int s_retried[2];
    __shared__ float s_z[kPreUnits][8][kChainThreads];   /* producers: seeded halves computed ahead of the wait */
    if (threadIdx.x < 2) s_retried[threadIdx.x] = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        /* what this launch really runs with, for sifar_chain_geometry */
        uint32_t cluster_ctas;
        asm volatile("mov.u32 %0, %%cluster_nctaid.x;" : "=r"(cluster_ctas));
        a.cs->seen[0] = a.clustered; a.cs->seen[1] = cluster_ctas; a.cs->seen[2] = TAGGED ? 1u : 0u;
    }
    __syncthreads();
    unsigned reloads = 0;
    bool alive = true;
    /* the CTA that publishes chunk results stamps them: the chunk's reducer (rank 0's producer without all-reduce) */
    const bool stamper = no_ar ? (rank == 0u) : is_reducer;
    unsigned long long *my_stamps = a.stamps + (size_t)chunk * (a.steps + 1u);
    if (stamper && threadIdx.x == 0) my_stamps[0] = globaltimer_ns();
    /* phase trace: thread 0 of the reducer of chunk 0 and of rank 0's producer of chunk 0 */
    const bool tracer = TRACE && a.trace != nullptr && threadIdx.x == 0 && chunk == 0;
#define SIFAR_TRACE(slot) do { if (TRACE && tracer) a.trace[(size_t)s * kTraceSlots + (slot)] = globaltimer_ns(); } while (0)

    for (uint32_t s = 0; s < a.steps && alive; ++s) {
        const uint32_t e = a.e0 + 1u + s;
        const uint32_t t = e - a.base_epoch;
        const uint32_t p = e & 1u;
        char *ring_row = a.ring + (size_t)((t - 1u) % a.ring_len) * a.ring_stride;

        constexpr bool tagged = TAGGED;          /* form of the hand-over, see handoff_store (the host's choice by size) */
        /* hand-over words [parity][unit]; without all-reduce [parity][rank][unit]: every rank hands its partial to itself */
        const size_t ho_sets = no_ar ? (size_t)P : 1u, ho_mine = no_ar ? (size_t)rank : 0u;
        uint4 *ho_cur = a.handoff + ((size_t)p * ho_sets + ho_mine) * a.handoff_stride;                 /* this step's result */
        const uint4 *ho_prev = a.handoff + ((size_t)(p ^ 1u) * ho_sets + ho_mine) * a.handoff_stride;   /* the step before */
        if (is_reducer) {
            /* ---------------- the pulling side ---------------- */
            SIFAR_TRACE(0);
            const uint4 *src[P];
#pragma unroll
            for (int r = 0; r < P; ++r) {
                if (MODE == SIFAR_SPECULATIVE)
                    src[r] = reinterpret_cast<const uint4 *>(a.slots + ((size_t)p * P + r) * a.slot_stride);
                else
                    src[r] = reinterpret_cast<const uint4 *>(
                        a.plain + ((size_t)(MODE == SIFAR_DUALBUF ? p : 0u) * P + r) * a.plain_stride);
            }
            if (MODE != SIFAR_SPECULATIVE) {
                /* top barrier: this chunk of every rank's partial has been stored */
                if (threadIdx.x < 32) {
                    bool ok = true;
                    if (threadIdx.x < P)
                        ok = wait_flag_or_fail<false>(&cf->arrive[p][threadIdx.x], e, st, a.host_status, a.timeout_ns);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (threadIdx.x == 0) s_ok = ok;
                }
                __syncthreads();
                if (!s_ok) { alive = false; break; }
                SIFAR_TRACE(1);
            }
            bool retried = false;
            for (uint32_t k = 0; k < a.K; ++k) {
                const size_t u = unit0 + (size_t)k * kChainThreads;
                if (MODE == SIFAR_SPECULATIVE && a.poll.sentinel) {
                    /* warp-uniform: the warp's first slot decides whether the warp has work at all */
                    const size_t w0 = u - (threadIdx.x & 31u);
                    if (w0 >= nunits) break;
                    if (k == 0 || a.K > 1u) {
                        const unsigned before = reloads;
                        if (!sentinel_wait<P>(src, w0, e, a.timeout_ns, reloads)) {
                            if (threadIdx.x == 0 || (threadIdx.x & 31u) == 0u) fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
                            alive = false;
                            break;
                        }
                        retried |= (reloads != before);
                    }
                }
                if (u >= nunits) break;
                uint4 x[P];
#pragma unroll
                for (int r = 0; r < P; ++r) x[r] = ld_slot(src[r] + u);
                if (MODE == SIFAR_SPECULATIVE) {
                    const unsigned before = reloads;
                    const bool valid = validate_slot<P>(x, src, u, e, a.timeout_ns, a.poll, reloads,
                                          (TRACE && tracer && k == 0) ? a.trace + (size_t)s * kTraceSlots + 30 : nullptr);
                    /* the whole warp leaves together (its lanes have the same k and all have a unit): a lane that
                       went on alone would meet the warp-wide vote of the next sentinel wait without its neighbours */
                    if (!__all_sync(0xFFFFFFFFu, valid)) {
                        if (!valid) fail(st, a.host_status, SIFAR_ERR_TIMEOUT);
                        alive = false;
                        break;
                    }
                    retried |= (reloads != before);
                    if (TRACE && a.trace != nullptr && chunk == 0 && k == 0 && (threadIdx.x & 31) == 0)
                        a.trace[(size_t)s * kTraceSlots + 38 + (threadIdx.x >> 5)] = globaltimer_ns();
                    if (k == 0) {
                        SIFAR_TRACE(1);
                        if (TRACE && tracer) a.trace[(size_t)s * kTraceSlots + 29] = reloads - before;
                    }
                    const uint4 v = sum_vec<DT, P>(x, false);
                    if (tagged) handoff_store<3>(ho_cur, u, v, e); /* to the next producers (on the chain's critical path) */
                    store_slot_result<DT>(ring_row, u, n_io, v);   /* and into the caller's ring */
                } else {
                    const uint4 v = sum_vec<DT, P>(x, true);
                    if (tagged) handoff_store<4>(ho_cur, u, v, e);
                    store_vec_result<DT>(ring_row, u, n_io, v);
                }
            }
            /* "somebody in this CTA re-loaded a slot": two alternating words, so that clearing one after the
               barrier of step s cannot race with the marks of step s + 1 */
            if (MODE == SIFAR_SPECULATIVE && retried) s_retried[s & 1u] = 1;
            if (!__syncthreads_and(alive)) { alive = false; break; }
            SIFAR_TRACE(2);
            if (threadIdx.x == 0) {
                if (!tagged && MODE != SIFAR_BARRIER_ONESHOT) st_release_u32(&cf->ready, e);    /* flag form: result chunk published */
                SIFAR_TRACE(3);                                /* every thread of the chunk has handed its units over */
                if (MODE == SIFAR_SPECULATIVE && s_retried[s & 1u]) {
                    s_retried[s & 1u] = 0;
                    st_relaxed_u32(&a.retry_steps[s], 1u);
                }
                if (stamper) my_stamps[s + 1u] = globaltimer_ns();
            }
            if (MODE == SIFAR_BARRIER_ONESHOT) {
                /* bottom barrier, reducer side, block by block as the top barrier: the chunk has been read, its
                   P done flags are released (one lane each; every thread has passed the barrier above) */
                if (threadIdx.x < P) st_release_u32(&cf->done[threadIdx.x], e);
                SIFAR_TRACE(28);
            }
        } else {
            /* ---------------- rank `rank`, chunk `chunk` of the next operation ---------------- */
            constexpr int NW = kSlotUnits ? 3 : 4;
            constexpr int NE = NW * ((DT == SIFAR_BF16) ? 2 : 1);
            const Gen g = make_gen(a.w, rank, t);
            const bool first = (t == 1u);
            /* the seeded half of a unit does not need the previous result: do it before waiting.  The first
               unit's stays in registers, those of the next kPreUnits units are parked in shared memory (grids
               that need more units per thread than that are far beyond the decode payloads) */
            float z0[NE];
            if (unit0 < nunits) {
                unit_noise<DT, NW>(g, first, unit0 * EPU, n, z0);
                /* pin the values here: without this the compiler sinks the arithmetic below the wait */
#pragma unroll
                for (int k = 0; k < NE; ++k) asm volatile("" : "+f"(z0[k]));
            }
#pragma unroll 1
            for (uint32_t k = 1; k < a.K && k <= (uint32_t)kPreUnits; ++k) {
                const size_t u = unit0 + (size_t)k * kChainThreads;
                if (u >= nunits) break;
                float z[NE];
                unit_noise<DT, NW>(g, first, u * EPU, n, z);
#pragma unroll
                for (int q = 0; q < NE; ++q) s_z[k - 1u][q][threadIdx.x] = z[q];
            }
            const uint32_t delay_ns = gen_delay_ns(a.w, rank, t);
            const bool by_flag = !no_ar && !tagged;      /* thread 0 waits for the chunk, then everybody loads */
            if (by_flag || MODE == SIFAR_BARRIER_ONESHOT) {
                if (threadIdx.x == 0) {
                    bool ok = true;
                    if (MODE == SIFAR_BARRIER_ONESHOT) {
                        /* bottom barrier, producer side: the chunk's reducer has finished reading the single
                           buffer.  It released the done flags after its result stores and a CTA barrier, so the
                           flag hands the result over as well. */
                        if (t > 1u) ok = wait_flag_or_fail<true>(&cf->done[rank], e - 1u, st, a.host_status, a.timeout_ns);
                    } else if (t > 1u) {
                        ok = wait_flag_or_fail<true>(&cf->ready, e - 1u, st, a.host_status, a.timeout_ns);
                    }
                    if (by_flag) { SIFAR_TRACE(4 + 3 * rank); if (ok) spin_ns(delay_ns); }   /* else: after the first unit is taken */
                    s_ok = ok;
                }
                __syncthreads();
                if (!s_ok) { alive = false; break; }
            }
            const char *prev = a.ring + (size_t)((t + a.ring_len - 2u) % a.ring_len) * a.ring_stride;   /* flag form */
            /* The previous result of unit u: polled where the reducer hands it over (first step: none).  The rank's
               seeded delay (skewed-arrival workload) follows the first unit's arrival, before anything is stored. */
            const auto take_prev = [&](size_t u, uint32_t (&pw)[NW], bool with_delay) -> bool {
#pragma unroll
                for (int q = 0; q < NW; ++q) pw[q] = 0u;
                bool ok = true;
                if (!first) ok = handoff_wait<NW>(ho_prev, u, e - 1u, pw, st, a.host_status, a.timeout_ns);
                if (with_delay) { SIFAR_TRACE(4 + 3 * rank); spin_ns(delay_ns); }
                return ok;
            };
            const auto store_unit = [&](size_t u, const uint32_t (&w)[NW]) {
                if (no_ar) {
                    handoff_store<3>(ho_cur, u, make_uint4(w[0], w[1], w[2], 0u), e);      /* to itself, next step */
                } else if (MODE == SIFAR_SPECULATIVE) {
                    store_slot(reinterpret_cast<uint4 *>(a.slots + ((size_t)p * P + rank) * a.slot_stride), u,
                               w[0], w[1], w[2], e);
                } else {
                    const uint32_t bp = (MODE == SIFAR_BARRIER_ONESHOT) ? 0u : p;
                    st_slot(reinterpret_cast<uint4 *>(a.plain + ((size_t)bp * P + rank) * a.plain_stride) + u,
                            make_uint4(w[0], w[1], w[2], w[NW - 1]));
                }
            };
            bool mine_ok = true;
            if (unit0 < nunits) {
                uint32_t w[NW];
                if (by_flag) {
                    unit_combine<DT, NW>(g, first, prev, unit0 * EPU, n, z0, w, n_io);
                } else {
                    uint32_t pw[NW];
                    mine_ok = take_prev(unit0, pw, true);
                    unit_apply<DT, NW>(g, first, pw, unit0 * EPU, n, z0, w);
                }
                if (mine_ok) store_unit(unit0, w);
            }
#pragma unroll 1
            for (uint32_t k = 1; k < a.K && mine_ok; ++k) {
                const size_t u = unit0 + (size_t)k * kChainThreads;
                if (u >= nunits) break;
                uint32_t w[NW];
                float z[NE];
                if (k <= (uint32_t)kPreUnits) {
#pragma unroll
                    for (int q = 0; q < NE; ++q) z[q] = s_z[k - 1u][q][threadIdx.x];
                } else {
                    unit_noise<DT, NW>(g, first, u * EPU, n, z);
                }
                if (by_flag) {
                    unit_combine<DT, NW>(g, first, prev, u * EPU, n, z, w, n_io);
                } else {
                    uint32_t pw[NW];
                    mine_ok = take_prev(u, pw, false);
                    unit_apply<DT, NW>(g, first, pw, u * EPU, n, z, w);
                }
                if (mine_ok) store_unit(u, w);
            }
            if (!mine_ok) alive = false;
            if (MODE == SIFAR_SPECULATIVE && !alive) break;        /* no barrier ahead of this thread in this mode */
            /* (by_flag never fails here: its waiting was done by thread 0 above) */
            if (TRACE && a.trace != nullptr && chunk == 0 && rank == 0 && (threadIdx.x & 31) == 0)
                a.trace[(size_t)s * kTraceSlots + 42 + (threadIdx.x >> 5)] = globaltimer_ns();
            SIFAR_TRACE(5 + 3 * rank);
            if (MODE == SIFAR_BARRIER_ONESHOT || MODE == SIFAR_DUALBUF) {
                /* the whole CTA leaves together if one of its threads gave up waiting */
                if (!__syncthreads_and(alive)) { alive = false; break; }
                if (threadIdx.x == 0) st_release_u32(&cf->arrive[p][rank], e);
                SIFAR_TRACE(6 + 3 * rank);
            } else if (no_ar) {
                if (!__syncthreads_and(alive)) { alive = false; break; }
                if (stamper && threadIdx.x == 0) my_stamps[s + 1u] = globaltimer_ns();
            }
        }
    }

#undef SIFAR_TRACE
    /* leave: mis-speculation counters, then the last CTA out publishes the call number */
    const unsigned warp_reloads = __reduce_add_sync(0xFFFFFFFFu, reloads);
    if (warp_reloads && (threadIdx.x & 31) == 0)
        atomicAdd(&st->stats[kStatSlotReloads], (unsigned long long)warp_reloads);
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t left = atom_add_acq_rel_u32(&a.cs->exit_count, 1u) + 1u;
        s_ok = (left == a.exit_base + gridDim.x && !no_ar && ld_relaxed_u32(&st->status) == 0u);
    }
    __syncthreads();
    if (s_ok) {
        /* last CTA out: the whole CTA sums and clears the per-step retry marks, then thread 0 books the run */
        if (MODE == SIFAR_SPECULATIVE) {
            unsigned long long part = 0;
            for (uint32_t s = threadIdx.x; s < a.steps; s += kChainThreads) {
                part += ld_relaxed_u32(&a.retry_steps[s]);
                st_relaxed_u32(&a.retry_steps[s], 0u);
            }
            if (part) atomicAdd(&st->stats[kStatCallsWithRetry], part);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            atomicAdd(&st->stats[kStatCalls], (unsigned long long)a.steps);
            st_release_u32(&st->epoch, a.e0 + a.steps);
        }
    }
}

/* ------------------------------------------------------------------------ */
/* 16-byte atomicity check                                                   */
/* ------------------------------------------------------------------------ */
__device__ __forceinline__ uint4 tear_pattern(uint32_t c)
{
    return make_uint4(c, ~c, c * 0x9E3779B9u, c ^ 0xA5A5A5A5u);
}

__global__ void __launch_bounds__(256) k_tear(uint4 *slots, unsigned nslots, unsigned rounds, unsigned writers,
                                              unsigned long long *torn, unsigned long long *reads)
{
    const bool writer = blockIdx.x < writers;
    unsigned long long my_torn = 0, my_reads = 0;
    if (writer) {
        const unsigned wid = blockIdx.x * blockDim.x + threadIdx.x, nw = writers * blockDim.x;
        for (unsigned round = 1; round <= rounds; ++round)
            for (unsigned s = wid; s < nslots; s += nw) st_slot(slots + s, tear_pattern(round * 2654435761u + s));
    } else {
        const unsigned rid = (blockIdx.x - writers) * blockDim.x + threadIdx.x;
        const unsigned nr = (gridDim.x - writers) * blockDim.x;
        for (unsigned round = 1; round <= rounds; ++round)
            for (unsigned s = rid; s < nslots; s += nr) {
                const uint4 v = ld_slot(slots + s);
                const uint4 want = tear_pattern(v.x);
                ++my_reads;
                if (!(v.x == 0u && v.y == 0u && v.z == 0u && v.w == 0u) &&
                    (v.y != want.y || v.z != want.z || v.w != want.w))
                    ++my_torn;
            }
    }
    if (my_torn) atomicAdd(torn, my_torn);
    if (my_reads) atomicAdd(reads, my_reads);
}

}  /* namespace sifar */

using namespace sifar;

/* ------------------------------------------------------------------------ */
/* host side                                                                 */
/* ------------------------------------------------------------------------ */
struct sifar_chain {
    sifar_ctx *ctx;
    sifar_workload w;
    size_t n;
    int mode, impl;
    char *ring;
    int ring_len;
    size_t ring_stride;
    int steps;
    uint32_t base_epoch;
    uint32_t runs;
    int launches_per_run;
    cudaStream_t prod[kMaxRanks];
    cudaStream_t red;
    cudaEvent_t ev_fork;
    cudaEvent_t ev_join[kMaxRanks + 1];
    cudaEvent_t ev_prod[kMaxRanks];
    /*
     * Stream / graph chains: may the reducer kernel of a step start without waiting for that step's
     * producers?  CUDA does not promise that independently launched kernels run at the same time, and on
     * B200 the producers of a graph step were measured to run only on SMs that hold no CTA of an
     * already polling speculative reducer (step time ~ 1 / free SMs, no progress at one CTA per SM).
     * Up to kConcurrentTiles reducer CTAs the step is left unordered, which is what the speculative and
     * barrier protocols are about at decode payloads; above it the reducer is ordered behind the
     * producers by events: there the transfer dominates and the early start buys nothing.
     */
    bool concurrent;
    std::vector<cudaEvent_t> ev_step;
    cudaGraph_t graph;
    cudaGraphExec_t exec;
    /* persistent */
    ChainDev *d_cs;
    ChunkFlags *d_chunks;
    unsigned long long *d_stamps;
    unsigned long long *d_trace;
    int trace_on;
    uint32_t *d_retry_steps;
    uint4 *d_handoff;
    size_t handoff_stride;
    bool tagged;                    /* form of the hand-over (see handoff_store) */
    uint32_t C, K;
    int grid;
    bool clustered;                 /* one thread-block cluster per chunk (placement only) */
};

/*
 * Kernels that are launched for the first time while another kernel already waits for them must not be
 * loaded by that launch: with lazy module loading a load can wait for the device to become idle.  The
 * helpers that tests and benchmarks use to script orderings are loaded on the first call of any of them,
 * the chain kernels when a chain is created.
 */
template <typename K>
static cudaError_t preload(K kernel)
{
    cudaFuncAttributes at;
    return cudaFuncGetAttributes(&at, kernel);
}

static cudaError_t preload_helpers()
{
    static cudaError_t done = [] {
        cudaError_t e = preload(k_spin);
        if (e == cudaSuccess) e = preload(k_store_slots<SIFAR_BF16>);
        if (e == cudaSuccess) e = preload(k_store_slots<SIFAR_F32>);
        if (e == cudaSuccess) e = preload(k_store_blocks<SIFAR_BF16>);
        if (e == cudaSuccess) e = preload(k_store_blocks<SIFAR_F32>);
        if (e == cudaSuccess) e = preload(k_probe<SIFAR_BF16>);
        if (e == cudaSuccess) e = preload(k_probe<SIFAR_F32>);
        if (e == cudaSuccess) e = preload(k_delays);
        return e;
    }();
    return done;
}

template <int DT>
static cudaError_t preload_produce()
{
    cudaError_t e = preload(k_produce<DT, SIFAR_BARRIER_ONESHOT>);
    if (e == cudaSuccess) e = preload(k_produce<DT, SIFAR_DUALBUF>);
    if (e == cudaSuccess) e = preload(k_produce<DT, SIFAR_SPECULATIVE>);
    if (e == cudaSuccess) e = preload(k_produce<DT, kModeNoAllreduce>);
    return e;
}

static bool valid_workload(const sifar_workload *w)
{
    return w && w->kind >= 0 && w->kind <= 2 && w->delay_max_ns <= kMaxDelayNs;
}

extern "C" size_t sifar_chain_ring_stride(int dtype, size_t n)
{
    if (dtype != SIFAR_BF16 && dtype != SIFAR_F32) return 0;
    /* room for a warp's worth of 16-byte units past the last element: the persistent chains read and write
       whole units in whole warps (sub-sector stores, the loads that follow them, and partly filled warps were
       all measured slow on the chain's critical path) */
    return (n * elem_size(dtype) + kUnitPadBytes + 255) / 256 * 256;
}

template <int DT>
static cudaError_t launch_produce_dt(int mode, int grid, cudaStream_t s, const ProduceArgs &a)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: k_produce<DT, SIFAR_BARRIER_ONESHOT><<<grid, kProdThreads, 0, s>>>(a); break;
    case SIFAR_DUALBUF:         k_produce<DT, SIFAR_DUALBUF><<<grid, kProdThreads, 0, s>>>(a); break;
    case SIFAR_SPECULATIVE:     k_produce<DT, SIFAR_SPECULATIVE><<<grid, kProdThreads, 0, s>>>(a); break;
    default:                    k_produce<DT, kModeNoAllreduce><<<grid, kProdThreads, 0, s>>>(a); break;
    }
    return cudaGetLastError();
}

static const void *chain_rank_buffer(const sifar_ctx *c, int mode, uint32_t e, int r)
{
    if (mode == SIFAR_BARRIER_ONESHOT) return c->plain_buf(0, r);
    if (mode == SIFAR_SPECULATIVE) return c->slot_buf((int)(e & 1u), r);
    return c->plain_buf((int)(e & 1u), r);          /* DUALBUF and the no-all-reduce floor */
}

/* Enqueue one run (steps steps starting at step first_t) as P producer streams + one reducer stream forked from `origin`. */
static int enqueue_run(sifar_chain *ch, cudaStream_t origin, uint32_t first_t)
{
    sifar_ctx *c = ch->ctx;
    const int P = c->P;
    const bool no_ar = (ch->mode == kModeNoAllreduce);
    SIFAR_CUDA(cudaEventRecord(ch->ev_fork, origin));
    for (int r = 0; r < P; ++r) SIFAR_CUDA(cudaStreamWaitEvent(ch->prod[r], ch->ev_fork, 0));
    if (!no_ar) SIFAR_CUDA(cudaStreamWaitEvent(ch->red, ch->ev_fork, 0));

    const size_t units = (ch->mode == SIFAR_SPECULATIVE) ? slots_for(c->dtype, ch->n)
                                                         : (ch->n * elem_size(c->dtype) + 15) / 16;
    size_t pgrid = (units + kProdThreads - 1) / kProdThreads;
    const size_t cap = (size_t)c->sm_count * 2;
    if (pgrid > cap) pgrid = cap;

    for (int s = 0; s < ch->steps; ++s) {
        const uint32_t t = first_t + (uint32_t)s;
        const uint32_t e = ch->base_epoch + t;
        for (int r = 0; r < P; ++r) {
            if (s > 0 && !no_ar) SIFAR_CUDA(cudaStreamWaitEvent(ch->prod[r], ch->ev_step[s - 1], 0));
            ProduceArgs a;
            memset(&a, 0, sizeof a);
            a.st = c->d_state; a.host_status = c->d_status_alias; a.timeout_ns = c->timeout_ns;
            a.w = ch->w; a.rank = (uint32_t)r; a.n = ch->n;
            a.dst = const_cast<void *>(chain_rank_buffer(c, ch->mode, e, r));
            a.prev = no_ar ? chain_rank_buffer(c, ch->mode, e - 1u, r)
                           : ch->ring + (size_t)((t + ch->ring_len - 2u) % ch->ring_len) * ch->ring_stride;
            a.base_epoch = ch->base_epoch; a.parity = e & 1u;
            a.t_fixed = no_ar ? t : 0u;
            cudaError_t err = (c->dtype == SIFAR_BF16)
                ? launch_produce_dt<SIFAR_BF16>(ch->mode, (int)pgrid, ch->prod[r], a)
                : launch_produce_dt<SIFAR_F32>(ch->mode, (int)pgrid, ch->prod[r], a);
            SIFAR_CUDA(err);
            if (!no_ar && !ch->concurrent) {
                /* large reducer grid: order it behind the producers (see sifar_chain::concurrent) */
                SIFAR_CUDA(cudaEventRecord(ch->ev_prod[r], ch->prod[r]));
                SIFAR_CUDA(cudaStreamWaitEvent(ch->red, ch->ev_prod[r], 0));
            }
        }
        if (!no_ar) {
            ReduceLaunch rl;
            memset(&rl, 0, sizeof rl);
            for (int r = 0; r < P; ++r) rl.src[r] = chain_rank_buffer(c, ch->mode, e, r);
            rl.out = ch->ring + (size_t)((t - 1u) % ch->ring_len) * ch->ring_stride;
            rl.n = ch->n; rl.mode = ch->mode; rl.parity = e & 1u;
            /* The step's event is fired programmatically, as soon as every CTA of the reducer has started: the
               next step's producers become resident while the reducer still runs and wait (griddepcontrol.wait)
               for its completion before they read anything.  This takes the launch latency of the producers
               out of every step (CUDA-graph chain at 8 KB, P = 8: 7.5 -> 4.9 us per step).  SIFAR_CHAIN_PDL=0
               records the event the plain way. */
            static const bool early = !(getenv("SIFAR_CHAIN_PDL") && atoi(getenv("SIFAR_CHAIN_PDL")) == 0);
            if (early) rl.programmatic_event = ch->ev_step[s];
            int rc = launch_reduce(c, rl, ch->red);
            if (rc) return rc;
            if (!early) SIFAR_CUDA(cudaEventRecord(ch->ev_step[s], ch->red));
        }
    }
    for (int r = 0; r < P; ++r) {
        SIFAR_CUDA(cudaEventRecord(ch->ev_join[r], ch->prod[r]));
        SIFAR_CUDA(cudaStreamWaitEvent(origin, ch->ev_join[r], 0));
    }
    if (!no_ar) {
        SIFAR_CUDA(cudaEventRecord(ch->ev_join[P], ch->red));
        SIFAR_CUDA(cudaStreamWaitEvent(origin, ch->ev_join[P], 0));
    }
    return SIFAR_OK;
}

template <int DT, int P, bool TRACE>
static const void *chain_kernel_p(int mode, bool tagged)
{
    switch (mode) {
    case SIFAR_BARRIER_ONESHOT: return (const void *)k_chain<DT, P, SIFAR_BARRIER_ONESHOT, TRACE, false>;
    case SIFAR_DUALBUF:         return tagged ? (const void *)k_chain<DT, P, SIFAR_DUALBUF, TRACE, true>
                                              : (const void *)k_chain<DT, P, SIFAR_DUALBUF, TRACE, false>;
    case SIFAR_SPECULATIVE:     return tagged ? (const void *)k_chain<DT, P, SIFAR_SPECULATIVE, TRACE, true>
                                              : (const void *)k_chain<DT, P, SIFAR_SPECULATIVE, TRACE, false>;
    default:                    return (const void *)k_chain<DT, P, kModeNoAllreduce, false, false>;
    }
}

template <int DT>
static const void *chain_kernel_dt(int P, int mode, bool trace, bool tagged)
{
    /* the traced build exists for the shapes of the workload list only */
    if (trace && P == 8) return chain_kernel_p<DT, 8, true>(mode, tagged);
    if (trace && P == 2) return chain_kernel_p<DT, 2, true>(mode, tagged);
    switch (P) {
    case 1: return chain_kernel_p<DT, 1, false>(mode, tagged);
    case 2: return chain_kernel_p<DT, 2, false>(mode, tagged);
    case 3: return chain_kernel_p<DT, 3, false>(mode, tagged);
    case 4: return chain_kernel_p<DT, 4, false>(mode, tagged);
    case 5: return chain_kernel_p<DT, 5, false>(mode, tagged);
    case 6: return chain_kernel_p<DT, 6, false>(mode, tagged);
    case 7: return chain_kernel_p<DT, 7, false>(mode, tagged);
    default: return chain_kernel_p<DT, 8, false>(mode, tagged);
    }
}

static const void *chain_kernel(const sifar_chain *ch, bool trace = false)
{
    return ch->ctx->dtype == SIFAR_BF16 ? chain_kernel_dt<SIFAR_BF16>(ch->ctx->P, ch->mode, trace, ch->tagged)
                                        : chain_kernel_dt<SIFAR_F32>(ch->ctx->P, ch->mode, trace, ch->tagged);
}

static void chain_free(sifar_chain *ch)
{
    if (!ch) return;
    for (int r = 0; r < kMaxRanks; ++r) if (ch->prod[r]) cudaStreamDestroy(ch->prod[r]);
    if (ch->red) cudaStreamDestroy(ch->red);
    if (ch->ev_fork) cudaEventDestroy(ch->ev_fork);
    for (int r = 0; r <= kMaxRanks; ++r) if (ch->ev_join[r]) cudaEventDestroy(ch->ev_join[r]);
    for (int r = 0; r < kMaxRanks; ++r) if (ch->ev_prod[r]) cudaEventDestroy(ch->ev_prod[r]);
    for (cudaEvent_t e : ch->ev_step) if (e) cudaEventDestroy(e);
    if (ch->exec) cudaGraphExecDestroy(ch->exec);
    if (ch->graph) cudaGraphDestroy(ch->graph);
    if (ch->d_cs) cudaFree(ch->d_cs);
    if (ch->d_chunks) cudaFree(ch->d_chunks);
    if (ch->d_stamps) cudaFree(ch->d_stamps);
    if (ch->d_trace) cudaFree(ch->d_trace);
    if (ch->d_retry_steps) cudaFree(ch->d_retry_steps);
    if (ch->d_handoff) cudaFree(ch->d_handoff);
    delete ch;
}

static int chain_setup_persistent(sifar_chain *ch)
{
    sifar_ctx *c = ch->ctx;
    const int roles = (ch->mode == kModeNoAllreduce) ? c->P : c->P + 1;
    const size_t units = (ch->mode == SIFAR_SPECULATIVE || ch->mode == kModeNoAllreduce)
                             ? slots_for(c->dtype, ch->n) : (ch->n * elem_size(c->dtype) + 15) / 16;
    /* how a result reaches the next step's producers: tagged words up to kHandoffMaxPairs polling threads, the
       chunks' ready flags above (see handoff_store); with both barriers the done flags do it */
    size_t max_pairs = kHandoffMaxPairs;
    if (const char *env = getenv("SIFAR_CHAIN_HANDOFF_MAX")) max_pairs = (size_t)strtoull(env, nullptr, 10);
    ch->tagged = (ch->mode == SIFAR_DUALBUF || ch->mode == SIFAR_SPECULATIVE) && units * (size_t)c->P <= max_pairs;
    int per_sm = 0;
    SIFAR_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, chain_kernel(ch), kChainThreads, 0));
    const size_t resident = (size_t)per_sm * c->sm_count;
    /* the whole machine if need be: every unit per thread beyond the first lengthens the step by its
       dependent load and store round trips */
    const size_t budget = resident > (size_t)roles ? resident : (size_t)roles;
    uint32_t K = 1;      /* units per thread and step: 1 whenever the grid fits (more only lengthens the step) */
    size_t C = (units + kChainThreads - 1) / kChainThreads;
    while (C * roles > budget) {
        ++K;
        C = (units + (size_t)kChainThreads * K - 1) / ((size_t)kChainThreads * K);
    }
    ch->K = K; ch->C = (uint32_t)C; ch->grid = (int)(C * roles);
    /* One cluster per chunk if the device can hold all of them at once, for grids up to kChainClusterMaxPairs
       (unit, rank) pairs: keeping a chunk's traffic inside one GPC takes 0.2-0.3 us off a step at decode payloads
       (P = 8, 8 KB: 1.79 against 1.98 us speculative, 3.58 against 3.87 us with both barriers); larger grids did
       better spread over the machine (128 KB: 3.81 against 3.34 us; 256 KB: 7.1 against 6.0 us dual-buffered mean).
       SIFAR_CHAIN_CLUSTER=0: never. */
    ch->clustered = false;
    const char *env_cluster = getenv("SIFAR_CHAIN_CLUSTER");
    if (!(env_cluster && atoi(env_cluster) == 0) && roles <= 16 && units * (size_t)c->P <= kChainClusterMaxPairs) {
        const void *fn = chain_kernel(ch);
        cudaError_t err = cudaSuccess;
        if (roles > 8) err = cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3((unsigned)ch->grid);
        cfg.blockDim = dim3(kChainThreads);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)roles;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int max_clusters = 0;
        if (err == cudaSuccess) err = cudaOccupancyMaxActiveClusters(&max_clusters, fn, &cfg);
        if (err == cudaSuccess && (size_t)max_clusters >= C) ch->clustered = true;
        else cudaGetLastError();
    }
    SIFAR_CUDA(cudaMalloc(&ch->d_cs, sizeof(ChainDev)));
    SIFAR_CUDA(cudaMalloc(&ch->d_chunks, sizeof(ChunkFlags) * C));
    SIFAR_CUDA(cudaMalloc(&ch->d_stamps, sizeof(unsigned long long) * (ch->steps + 1) * C));
    SIFAR_CUDA(cudaMalloc(&ch->d_trace, sizeof(unsigned long long) * ch->steps * kTraceSlots));
    SIFAR_CUDA(cudaMemset(ch->d_trace, 0, sizeof(unsigned long long) * ch->steps * kTraceSlots));
    SIFAR_CUDA(cudaMalloc(&ch->d_retry_steps, sizeof(uint32_t) * ch->steps));
    SIFAR_CUDA(cudaMemset(ch->d_cs, 0, sizeof(ChainDev)));
    SIFAR_CUDA(cudaMemset(ch->d_chunks, 0, sizeof(ChunkFlags) * C));
    SIFAR_CUDA(cudaMemset(ch->d_stamps, 0, sizeof(unsigned long long) * (ch->steps + 1) * C));
    SIFAR_CUDA(cudaMemset(ch->d_retry_steps, 0, sizeof(uint32_t) * ch->steps));
    /* the hand-over buffer (see handoff_store): one 16-byte word per 12-byte unit, two per 16-byte vector, whole
       warps of units, both parities; zero = tag 0 = never valid.  Large grids use the chunks' ready flags instead. */
    if (ch->tagged || ch->mode == kModeNoAllreduce) {
        /* without all-reduce every rank hands its partial over to itself in the same words: P sets per parity */
        const size_t padded = (units + 31) / 32 * 32;
        const size_t sets = (ch->mode == kModeNoAllreduce) ? (size_t)c->P : 1;
        ch->handoff_stride = padded * (ch->mode == SIFAR_DUALBUF ? 2 : 1);
        SIFAR_CUDA(cudaMalloc(&ch->d_handoff, 2 * sets * ch->handoff_stride * sizeof(uint4)));
        SIFAR_CUDA(cudaMemset(ch->d_handoff, 0, 2 * sets * ch->handoff_stride * sizeof(uint4)));
    }
    return SIFAR_OK;
}

extern "C" sifar_chain *sifar_chain_create(sifar_ctx *c, const sifar_workload *w, size_t n, int mode, int impl,
                                           void *out_ring, int ring_len, int steps_per_run)
{
    if (!c || !valid_workload(w) || n == 0 || n > c->max_elems || mode < 0 || mode > kModeNoAllreduce ||
        impl < 0 || impl > SIFAR_CHAIN_PERSISTENT || !out_ring || ((uintptr_t)out_ring & 15u) || ring_len < 2 ||
        steps_per_run < 2 || (steps_per_run & 1) || steps_per_run % ring_len != 0) {
        set_error("sifar_chain_create: bad argument (need 1 <= n <= max_elems, ring_len >= 2 dividing an even "
                  "steps_per_run, delay_max_ns <= %u)", kMaxDelayNs);
        return nullptr;
    }
    if (*c->h_status != 0) { set_error("sifar_chain_create: context carries a device error"); return nullptr; }
    if ((uint64_t)c->h_epoch + (uint64_t)steps_per_run >= kEpochLimit) {
        set_error("sifar_chain_create: call numbers exhausted");
        return nullptr;
    }
    sifar_chain *ch = new (std::nothrow) sifar_chain();
    if (!ch) { set_error("sifar_chain_create: out of host memory"); return nullptr; }
    ch->ctx = c; ch->w = *w; ch->n = n; ch->mode = mode; ch->impl = impl;
    ch->ring = (char *)out_ring; ch->ring_len = ring_len;
    ch->ring_stride = sifar_chain_ring_stride(c->dtype, n);
    ch->steps = steps_per_run; ch->base_epoch = c->h_epoch; ch->runs = 0;
    cudaSetDevice(c->device);
    int rc = SIFAR_OK;
    auto setup = [&]() -> int {
        SIFAR_CUDA(preload_helpers());
        SIFAR_CUDA(c->dtype == SIFAR_BF16 ? preload_produce<SIFAR_BF16>() : preload_produce<SIFAR_F32>());
        if (impl == SIFAR_CHAIN_PERSISTENT) {
            int coop = 0;
            SIFAR_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device));
            if (!coop) { set_error("sifar_chain_create: device lacks cooperative launch"); return SIFAR_ERR_CUDA; }
            ch->launches_per_run = 1;
            return chain_setup_persistent(ch);
        }
        for (int r = 0; r < c->P; ++r) SIFAR_CUDA(cudaStreamCreateWithFlags(&ch->prod[r], cudaStreamNonBlocking));
        SIFAR_CUDA(cudaStreamCreateWithFlags(&ch->red, cudaStreamNonBlocking));
        SIFAR_CUDA(cudaEventCreateWithFlags(&ch->ev_fork, cudaEventDisableTiming));
        for (int r = 0; r <= c->P; ++r) SIFAR_CUDA(cudaEventCreateWithFlags(&ch->ev_join[r], cudaEventDisableTiming));
        for (int r = 0; r < c->P; ++r) SIFAR_CUDA(cudaEventCreateWithFlags(&ch->ev_prod[r], cudaEventDisableTiming));
        ch->concurrent = reduce_tiles(c, n, mode == kModeNoAllreduce ? SIFAR_DUALBUF : mode) <= kConcurrentTiles;
        ch->ev_step.assign((size_t)ch->steps, nullptr);
        for (int s = 0; s < ch->steps; ++s) SIFAR_CUDA(cudaEventCreateWithFlags(&ch->ev_step[s], cudaEventDisableTiming));
        ch->launches_per_run = ch->steps * (c->P + (mode == kModeNoAllreduce ? 0 : 1));      /* one reducer kernel per all-reduce */
        if (impl == SIFAR_CHAIN_GRAPH) {
            /* capture one run; every later replay finds the same parities because steps_per_run is even */
            cudaStream_t cap;
            SIFAR_CUDA(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
            cudaError_t err = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
            int erc = SIFAR_OK;
            if (err == cudaSuccess) {
                erc = enqueue_run(ch, cap, 1u);
                err = cudaStreamEndCapture(cap, &ch->graph);
            }
            cudaStreamDestroy(cap);
            if (erc) return erc;
            SIFAR_CUDA(err);
            SIFAR_CUDA(cudaGraphInstantiate(&ch->exec, ch->graph, 0));
        }
        return SIFAR_OK;
    };
    rc = setup();
    if (rc) { cudaGetLastError(); chain_free(ch); return nullptr; }
    return ch;
}

extern "C" int sifar_chain_run(sifar_chain *ch, void *stream)
{
    if (!ch) { set_error("sifar_chain_run: NULL chain"); return SIFAR_ERR_INVALID; }
    sifar_ctx *c = ch->ctx;
    const int s0 = *c->h_status;
    if (s0) { set_error("sifar_chain_run: context carries device status %d", s0); return s0; }
    const bool no_ar = (ch->mode == kModeNoAllreduce);
    const uint32_t expect = ch->base_epoch + (no_ar ? 0u : ch->runs * (uint32_t)ch->steps);
    if (c->h_epoch != expect) {
        set_error("sifar_chain_run: the context was used outside the chain (call number %u, expected %u)",
                  c->h_epoch, expect);
        return SIFAR_ERR_EPOCH;
    }
    if ((uint64_t)c->h_epoch + (uint64_t)ch->steps >= kEpochLimit) {
        set_error("sifar_chain_run: call numbers exhausted");
        return SIFAR_ERR_EPOCH;
    }
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t first_t = ch->runs * (uint32_t)ch->steps + 1u;
    if (ch->impl == SIFAR_CHAIN_STREAMS) {
        int rc = enqueue_run(ch, s, first_t);
        if (rc) return rc;
    } else if (ch->impl == SIFAR_CHAIN_GRAPH) {
        SIFAR_CUDA(cudaGraphLaunch(ch->exec, s));
    } else {
        PersistArgs a;
        memset(&a, 0, sizeof a);
        a.st = c->d_state; a.host_status = c->d_status_alias; a.timeout_ns = c->timeout_ns;
        a.w = ch->w; a.n = ch->n;
        a.plain = c->d_plain; a.plain_stride = c->plain_stride;
        a.slots = c->d_slots; a.slot_stride = c->slot_stride;
        a.ring = ch->ring; a.ring_stride = ch->ring_stride; a.ring_len = (uint32_t)ch->ring_len;
        a.e0 = no_ar ? ch->base_epoch + ch->runs * (uint32_t)ch->steps : c->h_epoch;
        a.base_epoch = ch->base_epoch; a.steps = (uint32_t)ch->steps;
        a.C = ch->C; a.K = ch->K;
        a.poll = poll_shape_for(c, ch->n);
        if (ch->tagged && ch->mode == SIFAR_SPECULATIVE) {
            /* with the tagged hand-over the producers store sooner after the reducer's result, and the reducer does
               best polling all stale ranks of its own slots up to a larger grid than the discrete reducer's
               (measured at P = 8: 2.05 / 2.24 us at 32 / 64 KB per rank against 2.98 / 3.07 us with the sentinel) */
            size_t wide_max = kChainWideMaxPairs;
            if (const char *env = getenv("SIFAR_CHAIN_WIDE_MAX")) wide_max = (size_t)strtoull(env, nullptr, 10);
            const bool wide = slots_for(c->dtype, ch->n) * (size_t)c->P <= wide_max;
            a.poll.wide = wide ? 1u : 0u;
            a.poll.sentinel = wide ? 0u : 1u;
        }
        a.exit_base = ch->runs * (uint32_t)ch->grid;
        a.cs = ch->d_cs; a.chunks = ch->d_chunks; a.stamps = ch->d_stamps; a.retry_steps = ch->d_retry_steps;
        a.trace = ch->trace_on ? ch->d_trace : nullptr;
        a.handoff = ch->d_handoff; a.handoff_stride = ch->handoff_stride;
        a.clustered = ch->clustered ? 1u : 0u;
        void *params[] = {&a};
        const void *fn = chain_kernel(ch, ch->trace_on != 0);
        if (ch->clustered) {
            const unsigned roles = (unsigned)(no_ar ? c->P : c->P + 1);
            if (roles > 8) SIFAR_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof cfg);
            cfg.gridDim = dim3((unsigned)ch->grid);
            cfg.blockDim = dim3(kChainThreads);
            cfg.stream = s;
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeCooperative;
            attr[0].val.cooperative = 1;
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = roles;
            attr[1].val.clusterDim.y = 1;
            attr[1].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            SIFAR_CUDA(cudaLaunchKernelExC(&cfg, fn, params));
        } else {
            SIFAR_CUDA(cudaLaunchCooperativeKernel(fn, dim3((unsigned)ch->grid), dim3(kChainThreads), params, 0, s));
        }
    }
    ch->runs += 1;
    if (!no_ar) c->h_epoch += (uint32_t)ch->steps;
    /* The stream and graph chains end in a library reducer, whose done flags a later sifar_pack waits for.  The
       persistent kernel keeps done flags of its own, and once it has run nothing reads the rank buffers any more. */
    if (ch->mode == SIFAR_BARRIER_ONESHOT)
        c->last_mode0_epoch = (ch->impl == SIFAR_CHAIN_PERSISTENT) ? 0u : c->h_epoch;
    return SIFAR_OK;
}

extern "C" int sifar_chain_stamps(sifar_chain *ch, unsigned long long *stamps)
{
    if (!ch || !stamps || ch->impl != SIFAR_CHAIN_PERSISTENT) {
        set_error("sifar_chain_stamps: needs a persistent chain and a destination");
        return SIFAR_ERR_INVALID;
    }
    SIFAR_CUDA(cudaDeviceSynchronize());
    const size_t per = (size_t)ch->steps + 1;
    std::vector<unsigned long long> all(per * ch->C);
    SIFAR_CUDA(cudaMemcpy(all.data(), ch->d_stamps, sizeof(unsigned long long) * all.size(), cudaMemcpyDeviceToHost));
    /* a result is complete when its last chunk is: per step the latest stamp over the chunks; the run starts
       with the earliest CTA */
    for (size_t s = 0; s < per; ++s) {
        unsigned long long v = all[s];
        for (uint32_t c = 1; c < ch->C; ++c) {
            const unsigned long long x = all[(size_t)c * per + s];
            v = (s == 0) ? (x < v ? x : v) : (x > v ? x : v);
        }
        stamps[s] = v;
    }
    return SIFAR_OK;
}

extern "C" int sifar_chain_chunk_stamps(sifar_chain *ch, int chunk, unsigned long long *stamps)
{
    if (!ch || !stamps || ch->impl != SIFAR_CHAIN_PERSISTENT || chunk < 0 || (uint32_t)chunk >= ch->C) {
        set_error("sifar_chain_chunk_stamps: needs a persistent chain, a chunk below %u and a destination", ch ? ch->C : 0u);
        return SIFAR_ERR_INVALID;
    }
    SIFAR_CUDA(cudaDeviceSynchronize());
    const size_t per = (size_t)ch->steps + 1;
    SIFAR_CUDA(cudaMemcpy(stamps, ch->d_stamps + (size_t)chunk * per, sizeof(unsigned long long) * per,
                          cudaMemcpyDeviceToHost));
    return SIFAR_OK;
}

extern "C" int sifar_chain_chunks(sifar_chain *ch) { return ch && ch->impl == SIFAR_CHAIN_PERSISTENT ? (int)ch->C : 0; }

extern "C" int sifar_chain_geometry(sifar_chain *ch, unsigned out[8])
{
    if (!ch || ch->impl != SIFAR_CHAIN_PERSISTENT || !out) {
        set_error("sifar_chain_geometry: needs a persistent chain");
        return SIFAR_ERR_INVALID;
    }
    ChainDev h;
    SIFAR_CUDA(cudaDeviceSynchronize());
    SIFAR_CUDA(cudaMemcpy(&h, ch->d_cs, sizeof h, cudaMemcpyDeviceToHost));
    out[0] = ch->C; out[1] = ch->K; out[2] = (unsigned)ch->grid;
    out[3] = ch->clustered ? 1u : 0u; out[4] = ch->tagged ? 1u : 0u;
    out[5] = h.seen[0]; out[6] = h.seen[1]; out[7] = h.seen[2];
    return SIFAR_OK;
}

extern "C" int sifar_chain_trace(sifar_chain *ch, int enable, unsigned long long *phases)
{
    if (!ch || ch->impl != SIFAR_CHAIN_PERSISTENT) {
        set_error("sifar_chain_trace: needs a persistent chain");
        return SIFAR_ERR_INVALID;
    }
    if (enable && ch->ctx->P != 8 && ch->ctx->P != 2) {
        set_error("sifar_chain_trace: the traced kernel is built for P = 2 and P = 8 only");
        return SIFAR_ERR_INVALID;
    }
    ch->trace_on = enable ? 1 : 0;
    if (phases) {
        SIFAR_CUDA(cudaDeviceSynchronize());
        SIFAR_CUDA(cudaMemcpy(phases, ch->d_trace, sizeof(unsigned long long) * ch->steps * kTraceSlots,
                              cudaMemcpyDeviceToHost));
    }
    return SIFAR_OK;
}

extern "C" int sifar_chain_launches_per_run(sifar_chain *ch)
{
    return ch ? ch->launches_per_run : 0;
}

extern "C" int sifar_chain_destroy(sifar_chain *ch)
{
    if (!ch) return SIFAR_OK;
    cudaSetDevice(ch->ctx->device);
    cudaError_t e = cudaDeviceSynchronize();
    chain_free(ch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
    return SIFAR_OK;
}

static int probe_launch(const sifar_workload *w, int rank, unsigned t, int dtype, const void *prev, void *dst,
                        size_t n, void *stream)
{
    if (!valid_workload(w) || rank < 0 || (dtype != SIFAR_BF16 && dtype != SIFAR_F32) || !dst ||
        ((uintptr_t)dst & 15u) || (t > 1 && (!prev || ((uintptr_t)prev & 15u))) || t == 0) {
        set_error("sifar_workload probe: bad argument");
        return SIFAR_ERR_INVALID;
    }
    if (n == 0) return SIFAR_OK;
    size_t grid = (n / 8 + 255) / 256;
    if (grid < 1) grid = 1;
    if (grid > 1184) grid = 1184;
    if (dtype == SIFAR_BF16)
        k_probe<SIFAR_BF16><<<(int)grid, 256, 0, (cudaStream_t)stream>>>(*w, (uint32_t)rank, t, prev, dst, n);
    else
        k_probe<SIFAR_F32><<<(int)grid, 256, 0, (cudaStream_t)stream>>>(*w, (uint32_t)rank, t, prev, dst, n);
    SIFAR_CUDA(cudaGetLastError());
    return SIFAR_OK;
}

extern "C" int sifar_workload_first(const sifar_workload *w, int rank, int dtype, void *dst, size_t n, void *stream)
{
    return probe_launch(w, rank, 1u, dtype, nullptr, dst, n, stream);
}

extern "C" int sifar_workload_next(const sifar_workload *w, int rank, unsigned t, int dtype, const void *prev_out,
                                   void *dst, size_t n, void *stream)
{
    if (t < 2) { set_error("sifar_workload_next: t must be >= 2"); return SIFAR_ERR_INVALID; }
    return probe_launch(w, rank, t, dtype, prev_out, dst, n, stream);
}

extern "C" int sifar_workload_delays(const sifar_workload *w, int P, unsigned t, unsigned *host_out)
{
    if (!w || P < 1 || P > 32 || !host_out) { set_error("sifar_workload_delays: bad argument"); return SIFAR_ERR_INVALID; }
    unsigned *d = nullptr;
    SIFAR_CUDA(cudaMalloc(&d, sizeof(unsigned) * 32));
    k_delays<<<1, 32>>>(*w, P, t, d);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpy(host_out, d, sizeof(unsigned) * P, cudaMemcpyDeviceToHost);
    cudaFree(d);
    SIFAR_CUDA(e);
    return SIFAR_OK;
}

extern "C" int sifar_workload_preload(void)
{
    SIFAR_CUDA(preload_helpers());
    SIFAR_CUDA(preload_produce<SIFAR_BF16>());
    SIFAR_CUDA(preload_produce<SIFAR_F32>());
    return SIFAR_OK;
}

extern "C" int sifar_spin(unsigned ns, void *stream)
{
    if (ns > 50000000u) { set_error("sifar_spin: at most 50 ms"); return SIFAR_ERR_INVALID; }
    SIFAR_CUDA(preload_helpers());
    k_spin<<<1, 1, 0, (cudaStream_t)stream>>>(ns);
    SIFAR_CUDA(cudaGetLastError());
    return SIFAR_OK;
}

extern "C" int sifar_store_slots(const void *src, void *slots, size_t first_slot, size_t nslots, size_t n,
                                 int dtype, unsigned tag, void *stream)
{
    if (!src || !slots || ((uintptr_t)slots & 15u) || (dtype != SIFAR_BF16 && dtype != SIFAR_F32)) {
        set_error("sifar_store_slots: bad argument");
        return SIFAR_ERR_INVALID;
    }
    if (nslots == 0) return SIFAR_OK;
    SIFAR_CUDA(preload_helpers());
    const unsigned grid = (unsigned)((nslots + 255) / 256 < 592 ? (nslots + 255) / 256 : 592);
    if (dtype == SIFAR_BF16)
        k_store_slots<SIFAR_BF16><<<grid, 256, 0, (cudaStream_t)stream>>>(src, (uint4 *)slots, first_slot, nslots, n, tag);
    else
        k_store_slots<SIFAR_F32><<<grid, 256, 0, (cudaStream_t)stream>>>(src, (uint4 *)slots, first_slot, nslots, n, tag);
    SIFAR_CUDA(cudaGetLastError());
    return SIFAR_OK;
}

extern "C" int sifar_store_blocks(const void *src, void *dst, void *flags, size_t stride_words, size_t first_block,
                                  size_t nblocks, size_t n, int dtype, unsigned tag, void *stream)
{
    if (!src || !dst || !flags || ((uintptr_t)src & 15u) || ((uintptr_t)dst & 15u) ||
        (dtype != SIFAR_BF16 && dtype != SIFAR_F32) || nblocks > 0x7FFFFFFFu) {
        set_error("sifar_store_blocks: bad argument");
        return SIFAR_ERR_INVALID;
    }
    if (nblocks == 0) return SIFAR_OK;
    SIFAR_CUDA(preload_helpers());
    if (dtype == SIFAR_BF16)
        k_store_blocks<SIFAR_BF16><<<(unsigned)nblocks, 256, 0, (cudaStream_t)stream>>>(src, dst, (uint32_t *)flags,
                                                                                     stride_words, first_block, n, tag);
    else
        k_store_blocks<SIFAR_F32><<<(unsigned)nblocks, 256, 0, (cudaStream_t)stream>>>(src, dst, (uint32_t *)flags,
                                                                                    stride_words, first_block, n, tag);
    SIFAR_CUDA(cudaGetLastError());
    return SIFAR_OK;
}

extern "C" int sifar_tear_check(unsigned nslots, unsigned rounds, unsigned long long *host_torn,
                                unsigned long long *host_reads)
{
    if (nslots == 0 || rounds == 0 || rounds > 100000 || !host_torn || !host_reads) {
        set_error("sifar_tear_check: bad argument");
        return SIFAR_ERR_INVALID;
    }
    int dev = 0, sms = 0;
    SIFAR_CUDA(cudaGetDevice(&dev));
    SIFAR_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    uint4 *slots = nullptr;
    unsigned long long *counters = nullptr;
    SIFAR_CUDA(cudaMalloc(&slots, (size_t)nslots * 16));
    cudaError_t e = cudaMalloc(&counters, 16);
    if (e == cudaSuccess) e = cudaMemset(slots, 0, (size_t)nslots * 16);
    if (e == cudaSuccess) e = cudaMemset(counters, 0, 16);
    if (e == cudaSuccess) {
        /* writers and readers must overlap in time: launch them as one cooperative grid, one CTA per SM */
        unsigned writers = (unsigned)sms / 2;
        unsigned long long *torn = counters, *reads = counters + 1;
        void *params[] = {&slots, &nslots, &rounds, &writers, &torn, &reads};
        e = cudaLaunchCooperativeKernel((const void *)k_tear, dim3((unsigned)sms), dim3(256), params, 0, 0);
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    unsigned long long h[2] = {0, 0};
    if (e == cudaSuccess) e = cudaMemcpy(h, counters, 16, cudaMemcpyDeviceToHost);
    cudaFree(slots);
    if (counters) cudaFree(counters);
    SIFAR_CUDA(e);
    *host_torn = h[0];
    *host_reads = h[1];
    return SIFAR_OK;
}
