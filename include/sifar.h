/*
 * sifar.h - C ABI of the emulated synchronization-free all-reduce (one GPU).
 *
 * The operation (paper, Section 3.1 "Oneshot"): each of P tensor-parallel ranks
 * holds a partial of n elements; every rank needs the element-wise sum.  Oneshot
 * pulls all P partials and reduces locally, guarded by a TOP barrier (all
 * partials produced before any pull: read-after-write) and a BOTTOM barrier (all
 * pulls finished before a partial is overwritten: write-after-write).  The paper
 * removes the bottom barrier by alternating two input buffers (Section 3.3,
 * "dual buffering") and the cost of the top barrier by reading at once and
 * validating afterwards (Sections 3.5 and 4.2, "speculative reduction").
 *
 * Here the P ranks are P equally laid out buffers in ONE GPU's memory, written by
 * per-rank producer kernels on their own streams; one reducer kernel plays the
 * pulling side.  There is no second GPU, no NVLink and no collective library.
 * The paper's in-switch reduction ("redundant pull", Section 3.4) and multicast
 * push are not part of this library.
 *
 * Result of every mode, exactly:  acc = widen(x_0[i]);  acc = acc + widen(x_r[i])
 * for r = 1..P-1 in binary32, round-to-nearest-even;  out[i] = narrow(acc) with
 * one RNE to the element type.
 *
 * Tuning knobs, read from the environment by sifar_create / sifar_chain_create
 * (defaults are what measurement on B200 settled on):
 *   SIFAR_SPIN_NS           how long a CTA of a large reducer grid waits before it queues its tile (5000)
 *   SIFAR_POLL_WIDE_MAX     re-poll all stale ranks per round up to this many (slot, rank) pairs (16384)
 *   SIFAR_POLL_PACE_NS/_MIN sleep between polling rounds above _MIN pairs (0 = unpaced)
 *   SIFAR_POLL_SENTINEL_MIN persistent chain: above this many pairs a warp first waits on one slot per rank (16384)
 *   SIFAR_CHAIN_CLUSTER     0 = persistent chain without thread-block clusters (by default the CTAs of a chunk are
 *                           one cluster, for placement, on grids of up to 50000 (unit, rank) pairs)
 *   SIFAR_CHAIN_HANDOFF_MAX persistent chain: up to this many (unit, rank) pairs a result reaches the next step's
 *                           producers in tagged 16-byte words that each thread polls for itself, above it through one
 *                           ready flag per chunk (100000)
 *   SIFAR_CHAIN_WIDE_MAX    persistent speculative chain with tagged hand-over: re-poll all stale ranks per round up to
 *                           this many (slot, rank) pairs, wait on a sentinel slot above (50000)
 *   SIFAR_CHAIN_PDL         0 = stream / graph chains record the step events the plain way (by default the
 *                           all-reduce of a step fires its event as soon as all its CTAs have started, and the
 *                           next step's producers wait inside the kernel for its completion)
 *   SIFAR_PDL               0 = reducers are launched without programmatic dependent launch (read when the
 *                           library is loaded).  By default a reducer with more CTAs than the GPU has SMs,
 *                           or one whose producers were all enqueued on other streams, may become resident
 *                           while the kernel before it on its stream drains.  In the two barrier-free modes
 *                           its loads then start at once (they are ordered by flags or tags, not by the
 *                           stream); everything it writes waits until that kernel is complete.
 *   SIFAR_BARRIER_EARLY     1 = the loads of a BARRIER_ONESHOT reducer may start early as well (they are ordered by
 *                           its arrival flags); off by default, the baseline keeps the conventional stream order
 *                           (read when the library is loaded)
 *   SIFAR_SWEEP             0 = contexts start with SIFAR_SWEEP_NEVER (see sifar_debug_sweep_policy; read when
 *                           the library is loaded)
 *
 * All pointers named "device" are CUDA device pointers valid on the context's
 * device; "stream" arguments are cudaStream_t passed as void* (NULL = the legacy
 * default stream).  Functions return a sifar_status_t unless stated otherwise;
 * no function throws, none synchronizes the device unless stated.
 */
#ifndef SIFAR_H
#define SIFAR_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sifar_ctx sifar_ctx;   /* opaque, owned by the library */

typedef enum { SIFAR_BF16 = 0, SIFAR_F32 = 1 } sifar_dtype;

/*
 * SIFAR_BARRIER_ONESHOT  baseline of Section 3.1: top barrier on P arrival flags,
 *                        plain partials in ONE buffer per rank, bottom barrier
 *                        (reducer CTAs all arrive, then P done flags are released;
 *                        the rank's next producer waits on its done flag).
 * SIFAR_DUALBUF          Section 3.3: two buffers per rank selected by the parity
 *                        of the call number; top barrier kept, bottom barrier gone.
 * SIFAR_SPECULATIVE      Sections 3.5 / 4.2 re-expressed for one GPU: the partial
 *                        travels in 16-byte slots of 12 data bytes + a 4-byte tag
 *                        equal to the call number; the reducer loads at once,
 *                        accepts a slot iff its tag matches, and re-loads only the
 *                        stale (rank, slot) pairs.  No flag, no barrier.
 */
typedef enum { SIFAR_BARRIER_ONESHOT = 0, SIFAR_DUALBUF = 1, SIFAR_SPECULATIVE = 2 } sifar_mode;

typedef enum {
    SIFAR_OK          =  0,
    SIFAR_ERR_INVALID = -1,   /* bad argument; nothing was launched, call number unchanged */
    SIFAR_ERR_NOMEM   = -2,
    SIFAR_ERR_CUDA    = -3,   /* a CUDA call failed; sifar_last_error() has its text       */
    SIFAR_ERR_TIMEOUT = -4,   /* a device-side wait ran out (sticky until sifar_reset)     */
    SIFAR_ERR_EPOCH   = -5    /* call numbers exhausted, or a parity mismatch on the device */
} sifar_status_t;

enum { SIFAR_MAX_RANKS = 8 };

/*
 * ORDERING CONTRACT (what the caller's streams must guarantee; it is the co-design
 * the paper asks of the inference engine, Sections 3.3 and 4.2 "Dual Buffering":
 * the input of an all-reduce is the output of the operation before it).
 *   - The producer of call e + 1 for any rank (sifar_pack, sifar_arrive,
 *     sifar_wait_writable, or a caller's own kernel writing into the buffer that
 *     sifar_rank_buffer returned) must be ORDERED AFTER the reducer kernel of call
 *     e: same stream, an event, or a graph edge.  In a decode step it is anyway,
 *     because it consumes `out` of call e.  The producer kernels take the call
 *     number from device memory when they run (so that a replayed CUDA graph needs
 *     no new arguments), and the reducer advances it when its last CTA is done.  A
 *     producer that runs before that finds the number one short; it is detected by
 *     the number's parity and the context turns SIFAR_ERR_EPOCH (sticky), in every
 *     mode, instead of overwriting a buffer under a running reducer.
 *   - The producer of call e must NOT be ordered before the reducer of call e by
 *     anything but the mode's own flags or tags: that wait is the thing measured.
 *   - sifar_allreduce calls on one context are enqueued on one stream (or otherwise
 *     serialized).  A reducer's reads are ordered by the protocol alone, its writes
 *     (`out`, the call number) by the stream: a large reducer whose producers were
 *     enqueued on other streams starts polling and loading while the kernel before
 *     it on its stream still drains, and stores only when that kernel is complete.
 *   - BARRIER_ONESHOT: the device-side bottom barrier (done flags, and the wait for
 *     them in sifar_pack / sifar_wait_writable) protects the single buffer against
 *     a producer that is ordered after the reducer's START only, as a fused
 *     forward-pass kernel would be.  With whole kernels in stream order the wait is
 *     already satisfied when the producer runs; the baseline then pays the
 *     reducer-side half only (all CTAs counted, P flag stores).
 */

/*
 * Create a context for P ranks (1..8) of at most max_elems elements of `dtype`
 * on the CURRENT device.  The operation is the oneshot all-reduce of Section 3.1;
 * the two parity sets of rank buffers it allocates are the buffer-ownership side
 * of dual buffering (Section 4.2, "Dual Buffering": the previous input buffer must
 * stay alive until the next all-reduce has run).  Allocates (cudaMalloc), once, per rank: two plain
 * buffers, two slot buffers, and the shared flag / call-number / status words;
 * everything zero-filled, so every tag starts as 0 = "never valid".
 * Synchronizes the device.  Returns NULL on failure (see sifar_last_error()).
 */
sifar_ctx *sifar_create(int P, size_t max_elems, int dtype);

/* Waits for the context's outstanding work, frees everything (the buffers of Section 4.2, "Dual Buffering",
   live exactly as long as the context).  NULL is a no-op. */
int sifar_destroy(sifar_ctx *ctx);

/*
 * The all-reduce (Section 3.1 "Oneshot": pull all P partials, reduce locally; with
 * the barriers of `mode`, Sections 3.3, 3.5 and 4.2).
 * Enqueue call number e = (calls so far) + 1 on `stream`: one reducer kernel, no
 * allocation, no host synchronization.
 *
 *   rank_ptrs  host array of P device pointers, or NULL.
 *              NULL: read the context's own rank buffers of this call (the buffers
 *              sifar_rank_buffer() / sifar_pack() hand out).
 *              non-NULL, mode BARRIER_ONESHOT: arbitrary caller buffers of n plain
 *              elements each, 16-byte aligned, reusable every call; each rank's
 *              stream must still announce them with sifar_arrive().
 *              non-NULL, other modes: every pointer must equal the context's
 *              buffer of this call, else SIFAR_ERR_INVALID.
 *   out        device, n plain elements, 16-byte aligned, caller-owned, must not
 *              overlap any rank buffer.  Valid once the kernel has finished
 *              (stream order).
 *   n          0 <= n <= max_elems.  n = 0 still consumes a call number.
 *
 * The reducer waits (barrier modes: for the arrival flags; speculative: per slot)
 * until every rank's partial of THIS call number has been stored.  Producers may
 * be enqueued on other streams before or after this call's kernel starts, but the
 * host must have issued sifar_pack()/sifar_rank_buffer() for this call number
 * before calling sifar_allreduce().  A wait that exceeds the time-out makes the
 * kernel give up: the sticky status becomes SIFAR_ERR_TIMEOUT, `out` is undefined
 * and later calls fail until sifar_reset().  Calls on one context must be
 * enqueued on one stream (or otherwise serialized).
 *
 * The early start pays only if the producers can actually run while the reducer
 * waits.  CUDA does not promise that for independently launched kernels: with
 * separate streams it held in every measurement here, but inside a captured graph
 * a waiting reducer of more than about 64 CTAs (n > 98 304 bf16 at P = 8) kept the
 * producers off the SMs it occupied.  For payloads of that size enqueue the
 * reducer behind its producers (an event or a graph edge); nothing is lost there.
 * Outside a graph, a call of at least 8 reducer tiles per SM (4.6 MiB per rank at
 * P = 8) in plain format whose producers still have work pending on their own
 * streams when this function is called is enqueued as two kernels, the reducer
 * grid and a sweep kernel for the tiles that grid had to leave
 * (sifar_debug_sweep_policy).
 */
int sifar_allreduce(sifar_ctx *ctx, const void *const *rank_ptrs, void *out, size_t n,
                    int mode, void *stream);

/*
 * Same operation from HOST memory, synchronous: moves the P host partials
 * (n plain elements each) to the device, packs them, reduces, delivers the result
 * in host_out and waits.  Pinned (page-locked), 16-byte aligned buffers are read
 * and written in place by the kernels: one launch packs all ranks, one reduces.
 * Pageable buffers go through staging buffers that the context allocates on the
 * first such call (one copy per rank).  For end-to-end measurements and simple
 * clients.
 */
int sifar_allreduce_host(sifar_ctx *ctx, const void *const *host_rank_ptrs, void *host_out,
                         size_t n, int mode);

/*
 * Where, and with which tag, `rank` must store its partial for the NEXT call in
 * `mode`.  *ptr: device buffer (plain elements for the barrier modes; 16-byte
 * slots {12 data bytes, 4-byte little-endian tag} for SPECULATIVE, slot i holding
 * elements [i*k, i*k+k), k = 6 for bf16 and 3 for fp32, a short last slot padded
 * with zeros; plain elements in the large-payload format, see sifar_spec_format).
 * *epoch: the call number, i.e. the tag value.  Either may be NULL.  The kernel that
 * writes there follows the ordering contract above.
 */
int sifar_rank_buffer(sifar_ctx *ctx, int rank, int mode, void **ptr, unsigned *epoch);

/*
 * Library producer-side store path: enqueue on `stream` a kernel that moves n
 * plain elements from `src` (device, 16-byte aligned) into the context's buffer
 * of `rank` for the NEXT call: a copy followed by a release of the rank's arrival
 * flag (barrier modes; BARRIER_ONESHOT first waits for the rank's done flag of
 * the previous call), or tagged 16-byte slot stores and nothing else (SPECULATIVE;
 * plain stores and one flag per 16 KiB block in its large-payload format, see
 * sifar_spec_format).  Must be ordered after the previous call's reducer (ordering
 * contract above); a kernel that was not turns the context SIFAR_ERR_EPOCH.
 */
int sifar_pack(sifar_ctx *ctx, int rank, const void *src, size_t n, int mode, void *stream);

/*
 * Barrier modes with partials written by the caller's own kernels: enqueue on
 * `stream` (after those kernels) the release of `rank`'s arrival flag for the
 * NEXT call.  Same ordering contract as sifar_pack.
 */
int sifar_arrive(sifar_ctx *ctx, int rank, int mode, void *stream);

/*
 * BARRIER_ONESHOT only: enqueue on `stream` the producer-side half of the bottom
 * barrier, a bounded wait until the reducer of the previous call has released
 * `rank`'s done flag.  Enqueue it before the kernel that overwrites the buffer,
 * and after the previous call's reducer in stream or event order (ordering contract).
 */
int sifar_wait_writable(sifar_ctx *ctx, int rank, void *stream);

/* Sticky device status (SIFAR_OK, SIFAR_ERR_TIMEOUT, SIFAR_ERR_EPOCH); reads a host-mapped word, no synchronization. */
int sifar_status(sifar_ctx *ctx);

/*
 * Copies eight counters (synchronizes the device):
 *   [0] calls completed        [1] calls in which at least one slot was re-loaded
 *   [2] slot re-loads          [3] arrival-flag polls that found the flag not yet set
 *   [4] waits that timed out   [5] current call number on the device   [6],[7] reserved
 */
int sifar_get_stats(sifar_ctx *ctx, unsigned long long out[8]);

/* Limit of every device-side wait, in microseconds (default 200000). */
int sifar_set_timeout_us(sifar_ctx *ctx, unsigned us);

/* Waits for outstanding work on `stream`, zeroes tags, flags, counters and status; call number back to 0. */
int sifar_reset(sifar_ctx *ctx, void *stream);

/*
 * Test hook: set the number of calls made so far (host and device).  Requires an
 * idle context.  Call numbers are 32-bit; 0 is reserved, and the library refuses
 * call number 2^32-1 and beyond with SIFAR_ERR_EPOCH until sifar_reset().
 */
int sifar_debug_set_epoch(sifar_ctx *ctx, unsigned calls_so_far);

/*
 * The two layouts in which a partial travels in SIFAR_SPECULATIVE, chosen by size.
 * The paper has no counterpart: it targets decode payloads of 8-32 KB (Section 5),
 * where the tags of the slots cost nothing that matters.  For large payloads the
 * tagged slots move a third more bytes than plain data, which is what bounds the
 * reducer there, so from 8 MiB for all P partials together the speculative mode
 * keeps the early start (Section 3.5) but validates per block instead of per slot:
 *
 * SIFAR_FORMAT_SLOTS   16-byte slots {12 data bytes, 4-byte tag}; no flag at all.  (A library built with
 *                      -DSIFAR_SLOT_S8X2, libsifar_s8x2.so, uses two halves {4 data bytes, tag} per slot
 *                      instead, each valid on its own: it needs only 64-bit atomicity and is the fallback
 *                      should a 16-byte access ever be seen torn; sifar_slot_count() tells the geometry.)
 * SIFAR_FORMAT_TILES   plain elements at the start of the same rank buffer, plus one
 *                      arrival flag per block of 16 KiB (8192 bf16 / 4096 fp32
 *                      elements; the last block may be short), set to the call number
 *                      with release semantics once the block is stored.  A reducer CTA
 *                      acquires only the P flags of the block its tile lies in, so
 *                      tiles are reduced as they land; there is no call-wide barrier
 *                      and no tag traffic.
 *
 * sifar_spec_format() is a pure function (no device access): the format that
 * sifar_pack() and sifar_allreduce() use for n elements per rank; SIFAR_ERR_INVALID
 * for a bad P or dtype.  sifar_tile_flags(): where `rank`'s block flags of the NEXT
 * call lie, for producers that store their partial themselves (device helper
 * sifar::signal_block in sifar_device.cuh): *flags = device address of the rank's
 * flag of block 0, a 32-bit word; the flag of block b is stride_words words further
 * per block (the P ranks' flags of one block share a 32-byte sector, so a reducer
 * CTA fetches them with one access); block b = elements [b * elems_per_flag,
 * (b + 1) * elems_per_flag).  Any of the three results may be NULL.
 */
typedef enum { SIFAR_FORMAT_SLOTS = 0, SIFAR_FORMAT_TILES = 1 } sifar_format;
int sifar_spec_format(int P, int dtype, size_t n);
int sifar_tile_flags(sifar_ctx *ctx, int rank, void **flags, size_t *elems_per_flag, size_t *stride_words);

/*
 * Measurement hook for the retry-latency experiment (Section 6.3, "Retry Overhead":
 * latency of the no-retry case and what each further retry adds, obtained by
 * forcing a fixed number of retries).  With rounds = k > 0 the speculative reducer
 * treats the attempt that found all P copies of a slot valid as mis-speculated,
 * k times: it loads all P copies again, one round after another, and validates
 * the last copies as usual.  Results are unchanged; the statistics count the extra
 * loads as re-loads and every such call as a call with retry.  rounds <= 64.
 * Takes effect for sifar_allreduce calls enqueued afterwards, for the next run of
 * a persistent chain, and for stream / graph chains created afterwards.
 */
int sifar_debug_force_retries(sifar_ctx *ctx, unsigned rounds);

/*
 * Measurement hook: who reduces the tiles that a large reducer grid had to queue because its producers
 * were late (one-GPU emulation only: Section 3.5's early start, with the reducer and its producers
 * sharing one machine; the paper's ranks each have a GPU of their own and no counterpart for this).
 *   SIFAR_SWEEP_AUTO (default; SIFAR_SWEEP=0 in the environment makes NEVER the default): a call in plain
 *     format (barrier modes, flagged tiles) of at least 8 tiles per SM whose P producers were all enqueued
 *     with sifar_pack / sifar_arrive on streams other than the reducer's gets a sweep kernel of its own,
 *     behind the reducer grid on the same stream, if at least one of those streams still has work pending
 *     when sifar_allreduce is called (cudaStreamQuery); the grid then keeps no janitors.  Not while the
 *     stream is being captured (a producer stream that is being captured is not asked and counts as idle).  A stream handed to sifar_pack / sifar_arrive must therefore stay alive until
 *     the sifar_allreduce of the same call number has returned.
 *   SIFAR_SWEEP_NEVER: queued tiles are always swept by the grid's own last CTAs (one per SM).
 *   SIFAR_SWEEP_ALWAYS: as AUTO without asking the streams (what the extra kernel costs on ready data).
 * Results do not depend on it.  Takes effect for sifar_allreduce calls enqueued afterwards.
 */
enum sifar_sweep_policy { SIFAR_SWEEP_NEVER = 0, SIFAR_SWEEP_AUTO = 1, SIFAR_SWEEP_ALWAYS = 2 };
int sifar_debug_sweep_policy(sifar_ctx *ctx, int policy);

/*
 * All-reduce without any allocation.  The paper has no counterpart for this call.
 *
 * For callers that must not allocate device memory: an engine that gave the whole
 * device to its own arena at start-up and may not call cudaMalloc afterwards, or
 * a latency-critical loop that cannot afford the device-wide synchronization an
 * allocation implies.  It reduces P caller-owned plain partials that are already
 * complete in the order of `stream` (no flags, no tags, no context) into `out`:
 * same arithmetic as sifar_allreduce().
 *
 *   rank_ptrs  host array of P device pointers (1 <= P <= 8), n plain elements each,
 *              16-byte aligned, read only.
 *   out        device, n plain elements, 16-byte aligned, must not overlap an input.
 *   n          at most sifar_noalloc_max_elems() = 2^20 elements per rank; larger n
 *              is refused with SIFAR_ERR_INVALID (use a context instead).  n = 0 is
 *              a no-op.
 *
 * The kernel's bookkeeping (the count of finished CTAs by which the last CTA
 * knows it is last, and two call counters; 256 bytes) lives in a fixed array in
 * the library's device image: every GPU that loads the library holds it until
 * the process exits.  The first call on a device looks up the array's device
 * address (cudaGetSymbolAddress, with that device current) and caches it; make
 * that first call before any stream capture begins.  The call itself enqueues a
 * 4-byte clear of the CTA count and one kernel on `stream`; it calls no
 * cudaMalloc, cudaFree or other allocating routine and does not synchronize.
 * All calls on a device share the array, which keeps the previous call's
 * counters: calls that overlap in time on the GPU (different streams without an
 * ordering between them) race on it and are not supported.
 */
int sifar_allreduce_noalloc(const void *const *rank_ptrs, int P, void *out, size_t n, int dtype, void *stream);
size_t sifar_noalloc_max_elems(void);
/*
 * The bookkeeping words of the current device's array, for tests and diagnosis (waits for the device, copies
 * to the caller's array, allocates nothing): out[0] = count of finished CTAs (0 between calls: the last CTA of
 * a call re-arms it), out[1] = calls completed on this device since the library was loaded, out[2] = n of the
 * last completed call.
 */
int sifar_noalloc_counters(unsigned long long out[3]);

/* Geometry helpers (no device work). */
size_t sifar_slot_count(int dtype, size_t n);          /* slots needed for n elements  */
size_t sifar_algorithmic_bytes(int P, int dtype, size_t n, int mode);  /* bytes the method must move per call:
                                                          P reads of the partial (plain or slots) + one write of
                                                          out + the flag words of the mode */

/* Text of the last error on the calling thread ("" if none). */
const char *sifar_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SIFAR_H */
