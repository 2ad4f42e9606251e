/*
 * Internal declarations shared by the translation units of libsifar.so:
 * the device-resident protocol state, the host context, launch helpers.
 */
#ifndef SIFAR_INTERNAL_CUH
#define SIFAR_INTERNAL_CUH

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "sifar.h"
#include "sifar_device.cuh"

namespace sifar {

constexpr int kMaxRanks = SIFAR_MAX_RANKS;
constexpr size_t kUnitPadBytes = 512;            /* 32 units of 16 bytes: room behind every rank buffer and ring row */
constexpr uint32_t kEpochLimit = 0xFFFFFFFEu;    /* last usable call number                  */
constexpr size_t kFlagBlockVecs = 1024;          /* flagged-tile format: 16-byte vectors covered by one arrival flag */
constexpr size_t kFlagStride = 8;                /* ... words between two blocks' flags: [block][rank], one 32-byte sector per block */

/*
 * Protocol state in device memory (one per context, zero-filled at creation).
 * Words that different actors poll sit in different 128-byte lines.
 */
struct __align__(128) DevState {
    /* line 0: call number and sticky status; read together by every kernel at entry */
    uint32_t epoch;                  /* number of completed calls                               */
    uint32_t status;                 /* 0, or a negative sifar_status_t stored as uint32         */
    uint32_t pad0[30];
    /* line 1: last-CTA detection of the reducer, retry marker and the statistics: everything the CTA that
       closes a call touches lies in the line the arriving CTAs keep hot */
    uint32_t cta_arrive[2];          /* arrived CTAs of the call, by parity of the call number; the top bit says
                                        that a tile was queued.  A call re-arms the OTHER parity's word when it
                                        closes, so nobody who still polls this call's word sees it change back */
    uint32_t retry_epoch;            /* call number of the last call that re-loaded a slot       */
    uint32_t janitor_done;           /* janitor CTAs that have finished their share              */
    uint32_t pad1[12];
    unsigned long long stats[8];
    /* lines 2-3: arrival flags, one 128-byte line per parity (top barrier) */
    uint32_t arrive[2][32];
    /* line 4: done flags (bottom barrier, BARRIER_ONESHOT) */
    uint32_t done[32];
    /* line 5: per-rank CTA counters of the pack kernels */
    uint32_t pack_count[32];
};

enum StatIndex { kStatCalls = 0, kStatCallsWithRetry = 1, kStatSlotReloads = 2, kStatFlagPolls = 3,
                 kStatTimeouts = 4 };

/* Record a failed wait: sticky status on the device and in the host-mapped word. */
__device__ __forceinline__ void fail(DevState *st, volatile int *host_status, int code)
{
    if (atomicCAS(&st->status, 0u, (uint32_t)code) == 0u) {
        atomicAdd(&st->stats[kStatTimeouts], 1ull);
        *host_status = code;
        __threadfence_system();
    }
}

/* Element geometry */
__host__ __device__ inline size_t elem_size(int dtype) { return dtype == SIFAR_BF16 ? 2 : 4; }
__host__ __device__ inline size_t elems_per_slot(int dtype) { return (size_t)kSlotDataWords * (dtype == SIFAR_BF16 ? 2 : 1); }
__host__ __device__ inline size_t slots_for(int dtype, size_t n)
{
    size_t k = elems_per_slot(dtype);
    return (n + k - 1) / k;
}

}  /* namespace sifar */

/* Host context. */
struct sifar_ctx {
    int P;
    int dtype;
    int device;
    int sm_count;
    size_t max_elems;
    size_t plain_stride;             /* bytes between two rank buffers (multiple of 256) */
    size_t slot_stride;
    char *d_plain;                   /* [parity][rank] plain buffers                     */
    char *d_slots;                   /* [parity][rank] slot buffers                      */
    sifar::DevState *d_state;
    uint32_t *d_defer;               /* queued tiles of the deferring reducer: count, then tile indices */
    uint32_t *d_tflags;              /* [parity][block][kFlagStride] arrival flags of the flagged-tile format   */
    size_t tflag_words;              /* words per parity (a multiple of 32)                                    */
    volatile int *h_status;          /* pinned, mapped                                   */
    int *d_status_alias;             /* device alias of h_status                         */
    uint32_t h_epoch;                /* calls enqueued so far                            */
    uint32_t last_mode0_epoch;       /* last BARRIER_ONESHOT call (0: none): whose done flags a producer waits for */
    unsigned long long timeout_ns;
    unsigned long long spin_ns;      /* deferring reducer: how long a CTA waits before it queues its tile     */
    size_t poll_wide_max;            /* speculative: wide polling up to this many (slot, rank) pairs per call */
    size_t poll_pace_min;            /* ... paced polling above this many pairs                              */
    uint32_t poll_pace_ns;
    size_t poll_sentinel_min;        /* ... sentinel wait per warp above this many pairs (persistent chain) */
    int sweep_policy;                /* SIFAR_SWEEP_*: when a large call gets a sweep kernel of its own        */
    uint32_t force_retries;          /* measurement knob: forced re-load rounds per slot (0 in normal use)    */
    /* what the host knows about the producers of the next call (sifar_pack / sifar_arrive record it) */
    uint32_t prod_epoch[SIFAR_MAX_RANKS];   /* call number the rank's producer was enqueued for (0: none)      */
    cudaStream_t prod_stream[SIFAR_MAX_RANKS];
    size_t prod_n[SIFAR_MAX_RANKS];         /* elements it packs (sifar_pack only, else SIZE_MAX)              */
    /* staging for sifar_allreduce_host, allocated on first use */
    char *d_stage_in;
    char *d_stage_out;
    cudaStream_t host_stream;

    char *plain_buf(int parity, int r) const { return d_plain + ((size_t)parity * P + r) * plain_stride; }
    char *slot_buf(int parity, int r) const { return d_slots + ((size_t)parity * P + r) * slot_stride; }
    /* rank r's flag of block b of that parity: tile_flags(parity)[b * kFlagStride + r] */
    uint32_t *tile_flags(int parity) const { return d_tflags + (size_t)parity * tflag_words; }
};

namespace sifar {

/* Error text of the calling thread. */
void set_error(const char *fmt, ...);
int cuda_fail(cudaError_t e, const char *what);

#define SIFAR_CUDA(call)                                                   \
    do {                                                                   \
        cudaError_t e__ = (call);                                          \
        if (e__ != cudaSuccess) return ::sifar::cuda_fail(e__, #call);     \
    } while (0)

/* Internal launchers, implemented in sifar_core.cu, used by the chains too. */
struct ReduceLaunch {
    const void *src[kMaxRanks];      /* parity-resolved rank buffers (plain or slots)   */
    void *out;
    size_t n;
    int mode;
    uint32_t parity;                 /* parity the host expects the call number to have */
    uint32_t e_host;                 /* the call number the host expects, or 0 (chains: taken from device memory) */
    cudaEvent_t programmatic_event;  /* NULL, or an event the kernel fires as soon as all its CTAs have started */
    int format;                      /* SPECULATIVE: SIFAR_FORMAT_SLOTS or SIFAR_FORMAT_TILES                   */
    const uint32_t *tile_flags;      /* SIFAR_FORMAT_TILES: the flag array of this call's parity                */
    bool early;                      /* the producers are known to run on other streams: reads need not wait for
                                        the kernel before this one on the stream (see the reducer kernels)       */
};

int launch_reduce(sifar_ctx *ctx, const ReduceLaunch &rl, cudaStream_t stream);
struct PollShape;
PollShape poll_shape_for(const sifar_ctx *ctx, size_t n);
size_t reduce_tiles(const sifar_ctx *ctx, size_t n, int mode);     /* CTAs of the reducer kernel for n elements */

}  /* namespace sifar */
#endif
