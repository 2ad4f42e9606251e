/*
 * sifar_workload.h - synthetic decode-step workloads that drive the all-reduce:
 * the chain of dependent {P producers -> all-reduce} steps of one token.
 *
 * The paper's setting (Sections 2.3, 3.5, 6.1): a decode step issues two
 * all-reduces per transformer layer, each fed by an operation on the previous
 * result, all inside one CUDA graph or one fused "megakernel" with no host
 * involvement, and all-reduce latency is measured back to back inside that
 * kernel.  Model weights are not available here, so "the next operation" of rank
 * r is a seeded elementwise update of the previous result (rules below); what is
 * kept is the dependency structure and the per-call traffic.
 *
 * Step t = 1, 2, ... of a chain (t = call number - call number at creation):
 *   every rank r produces its partial x_r^t   (t = 1: from the generator;
 *                                              t > 1: from out^{t-1});
 *   out^t = all-reduce(x_0^t .. x_{P-1}^t)  in the chain's mode.
 * Producers of step t are ordered after the all-reduce of step t-1 (they consume
 * its result: stream event, graph edge, or, inside the persistent kernel, result
 * words that carry the call number and are polled by the thread that needs them
 * (one ready flag per chunk for large grids; the done flags of the bottom barrier
 * with both barriers)) and are NOT ordered before the all-reduce of step t by anything but
 * the arrival flags / slot tags of the mode under test.
 *
 * Update rules (each product and the sum rounded separately, no fused
 * multiply-add; z = noise of (seed, rank, step, element)):
 *   kind 0 (gauss, z ~ N(0,1) as a sum of twelve 16-bit uniforms) and
 *   kind 2 (uniform, z ~ U[-1,1)):
 *       x_r^1[i]   = narrow( z * (outlier(r,i) ? 100 : 1) )
 *       x_r^t[i]   = narrow( widen(out^{t-1}[i]) * scale + z * sigma )
 *   kind 1 (integers in [-64,64], k uniform on 0..128):
 *       x_r^1[i]   = k - 64
 *       x_r^t[i]   = ((int(out^{t-1}[i]) + k) mod 129, taken in [0,128]) - 64
 * delay_max_ns > 0: before storing, rank r at step t busy-waits a seeded time
 * uniform on [0, delay_max_ns] (skewed arrival); values are unaffected.
 *
 * Two families of chains run these steps:
 *   sifar_chain_*     one reader: P producers feed one all-reduce whose single result
 *                     feeds all P producers again (streams, CUDA graph, or one
 *                     persistent kernel), which is what sifar_allreduce computes;
 *   sifar_symchain_*  P readers: every rank runs its operation and its own
 *                     pull-and-reduce and keeps its own copy of the result, as every
 *                     GPU of the paper's system does; also carries the twoshot baseline.
 */
#ifndef SIFAR_WORKLOAD_H
#define SIFAR_WORKLOAD_H

#include "sifar.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int      kind;            /* 0 gauss, 1 integers, 2 uniform */
    unsigned seed;
    float    scale;
    float    sigma;
    unsigned outlier_mod;     /* 0: none; m: one first partial in m is multiplied by 100 */
    unsigned delay_max_ns;
} sifar_workload;

typedef struct sifar_chain sifar_chain;   /* opaque */

/* How the chain runs on the device. */
typedef enum {
    SIFAR_CHAIN_STREAMS    = 0,  /* P producer streams + one reducer stream, events for the result dependency   */
    SIFAR_CHAIN_GRAPH      = 1,  /* the same topology captured once into a CUDA graph and replayed              */
    SIFAR_CHAIN_PERSISTENT = 2   /* one cooperative kernel: reducer CTAs and P groups of producer CTAs that talk
                                    only through flags / tags in memory, for all steps of a run                 */
} sifar_chain_impl;

/* Fourth "mode", chains only: no all-reduce at all; each rank's next operation consumes its own
   partial (the paper's "feed the input of the all-reduce to the next operation" experiment, Section 2.4).
   The producers' own cost (in the persistent kernel a rank hands its partial to itself the way an all-reduce
   result reaches the next step's producers); its results are not a sum. */
enum { SIFAR_CHAIN_NO_ALLREDUCE = 3 };

/* Fifth "mode", sifar_symchain_create only: the twoshot baseline (reduce-scatter, barrier, all-gather;
   Section 3.1), which needs the P readers of that chain to mean anything. */
enum { SIFAR_SYMCHAIN_TWOSHOT = 4 };

/* Sixth and seventh "mode", sifar_symchain_create only: the paper's own validation scheme (Section 4.2,
   "Speculative Reduction" and "Verification Logic Correctness"; overheads in Section 6.3): plain payload in
   two alternating buffers, one validation flag per threadblock written after the payload (the flags alternate
   too), one extra warp per threadblock that pulls the P flags while the other warps pull the payload, success
   iff the flags add up to P x flag, otherwise the whole threadblock pulls again.
   FLAGVAL issues payload and flag loads together, as the paper does; a stale payload read followed by a
   fresh flag read would pass the check, which is what the paper's monotonicity assumption (Section 8.1)
   excludes.  FLAGVAL_ORDERED pulls the payload only after all P flags were seen with acquire semantics:
   sound without that assumption, at the price of the flag round trip. */
enum { SIFAR_SYMCHAIN_FLAGVAL = 5, SIFAR_SYMCHAIN_FLAGVAL_ORDERED = 6 };

/* Eighth "mode", sifar_symchain_create only, TIMING ONLY: the pull of FLAGVAL with no flag and no check at all
   (the paper's idealized "no barriers" configuration of Section 6.3).  Its results are whatever the buffers
   held; it exists so that verification overhead = (a validated mode) - (this) can be measured. */
enum { SIFAR_SYMCHAIN_UNCHECKED = 7 };

/* Bytes between two rows of an output ring for n elements (a multiple of 256, at least 512 bytes more than the
   row: the persistent kernels work in whole warps of 16-byte units and write zeros behind the last element). */
size_t sifar_chain_ring_stride(int dtype, size_t n);

/*
 * Create a chain on `ctx` (which it then owns exclusively until destroyed: no other
 * sifar_allreduce / sifar_pack on that context in between).
 *   n              elements per rank, 1 <= n <= max_elems of the context
 *   mode           a sifar_mode, or SIFAR_CHAIN_NO_ALLREDUCE
 *   impl           a sifar_chain_impl
 *   out_ring       device, ring_len rows of sifar_chain_ring_stride() bytes, caller-owned;
 *                  out^t lands in row (t-1) mod ring_len (bytes of a row past n elements
 *                  are unspecified)
 *   ring_len       >= 2 and a divisor of steps_per_run
 *   steps_per_run  even, >= 2
 * Returns NULL on failure (sifar_last_error()).
 */
sifar_chain *sifar_chain_create(sifar_ctx *ctx, const sifar_workload *w, size_t n, int mode, int impl,
                                void *out_ring, int ring_len, int steps_per_run);

/* Enqueue the next steps_per_run steps on `stream`; consecutive runs continue the same chain. */
int sifar_chain_run(sifar_chain *chain, void *stream);

/*
 * Device timestamps (nanoseconds, %globaltimer) of the last run, after it has
 * finished: stamps[0] = start of the run (earliest CTA), stamps[s] = result of
 * step s of the run complete, i.e. its last chunk published, s = 1..steps_per_run
 * (the chunks of a result are reduced by different CTAs, which may run ahead of
 * one another).  PERSISTENT only (else SIFAR_ERR_INVALID).  Synchronizes the device.
 */
int sifar_chain_stamps(sifar_chain *chain, unsigned long long *stamps);

/* The same stamps for one chunk alone (its reducer CTA), and the number of chunks of a PERSISTENT chain. */
int sifar_chain_chunk_stamps(sifar_chain *chain, int chunk, unsigned long long *stamps);
int sifar_chain_chunks(sifar_chain *chain);

/*
 * How a PERSISTENT chain is laid out, as the host chose it and as the kernel of the last run saw it (synchronizes
 * the device): out[0] chunks, [1] units per thread and step, [2] CTAs, [3] 1 = the CTAs of a chunk are launched as
 * one thread-block cluster, [4] 1 = results reach the next step's producers in tagged words (0 = ready flag per
 * chunk, or done flags with both barriers); from the kernel: [5] the role layout it used (1 = clustered), [6] CTAs
 * per cluster as the hardware reported them (1 without clusters), [7] the form of the hand-over it was built for.
 * Before the first run [5..7] are 0.
 */
int sifar_chain_geometry(sifar_chain *chain, unsigned out[8]);

/*
 * Phase timeline of the persistent chain (the latency breakdown that stands in for
 * a bandwidth figure at decode payloads).  enable != 0 makes later runs record,
 * for every step s of a run, 48 words (0 = not taken; %globaltimer nanoseconds
 * unless stated) written by the CTAs that own chunk 0:
 *   reducer, thread 0:  [0] enters the step      [1] arrival flags seen (speculative: its warp's slots valid)
 *                       [2] whole chunk reduced  [3] result handed over (every thread has stored its units;
 *                                                    large grids: ready flag released)
 *                       [28] done flags released (BARRIER_ONESHOT)
 *                       [29] number of slot re-loads of thread 0 in this step (a count)
 *                       [30..37] end of its first eight re-poll rounds (speculative)
 *   reducer, lane 0 of warp w:   [38+w] the warp's slots validated (speculative)
 *   producer of rank r, thread 0: [4+3r] previous result taken (its first unit's word valid, or the chunk's
 *                                          ready / done flag seen)             [5+3r] stores issued
 *                                 [6+3r] arrival flag released (barrier modes)
 *   producer of rank 0, lane 0 of warp w: [42+w] the warp's stores issued
 * If `phases` is not NULL the words of the last run (steps_per_run x 48) are copied
 * to it (synchronizes the device).  PERSISTENT chains with P = 2 or P = 8 only; the
 * traced kernel is a separate build, so an untraced run pays nothing for it.
 */
int sifar_chain_trace(sifar_chain *chain, int enable, unsigned long long *phases);

/* Kernels launched per run by this chain (graph replays count their kernel nodes). */
int sifar_chain_launches_per_run(sifar_chain *chain);

int sifar_chain_destroy(sifar_chain *chain);

/*
 * The same decode step with P readers: every emulated rank runs its own next
 * operation AND its own pull-and-reduce, as every GPU does in the paper's system
 * (Section 3.1; the oneshot pseudocode of Section 4.2), and keeps its own copy of
 * every result.  One cooperative kernel of P x C CTAs; CTA (r, c) computes chunk c
 * of rank r's partial from chunk c of rank r's copy of the previous result, stores
 * it, pulls chunk c of all P partials (its own included) and reduces it.  Ranks
 * are ordered against each other by the mode's protocol alone (P x P arrival and
 * done flags, or slot tags), so they drift as real GPUs do and a rank
 * mis-speculates exactly when a peer is behind it.  Results are those of the
 * one-reader chains, P times.
 *   out_rings      device, P x ring_len rows of sifar_chain_ring_stride() bytes, caller-owned;
 *                  rank r's copy of out^t lands in row r * ring_len + (t-1) mod ring_len
 *   other arguments as for sifar_chain_create (mode may also be SIFAR_CHAIN_NO_ALLREDUCE: every rank's
 *   operation feeds on its own partial, the timing floor; or SIFAR_SYMCHAIN_TWOSHOT: every rank reduces
 *   1/P of each chunk for all, a second barrier, then every rank reads the reduced chunk; or one of the
 *   two SIFAR_SYMCHAIN_FLAGVAL modes above)
 * The chain owns the context exclusively until it is destroyed.
 */
typedef struct sifar_symchain sifar_symchain;   /* opaque */

sifar_symchain *sifar_symchain_create(sifar_ctx *ctx, const sifar_workload *w, size_t n, int mode,
                                      void *out_rings, int ring_len, int steps_per_run);
/* Enqueue the next steps_per_run steps on `stream`. */
int sifar_symchain_run(sifar_symchain *chain, void *stream);
/*
 * Device timestamps of the last run (synchronizes): stamps[0] = start of the run,
 * stamps[s] = result s complete on every rank (latest chunk of the latest rank),
 * s = 1..steps_per_run; sifar_symchain_rank_stamps: the same for one rank's copy.
 */
int sifar_symchain_stamps(sifar_symchain *chain, unsigned long long *stamps);
int sifar_symchain_rank_stamps(sifar_symchain *chain, int rank, unsigned long long *stamps);
/*
 * Mis-speculation per rank (Section 6.3, "Mis-Speculation and Verification Overhead": the
 * fraction of all-reduces that retried):
 * host_per_rank[r] = number of steps so far in which rank r had to load a slot
 * again, r = 0..P-1 (speculative mode; zeros otherwise).  Synchronizes.  The
 * context's statistics count a step as a call with retry if any rank retried.
 */
int sifar_symchain_retries(sifar_symchain *chain, unsigned long long *host_per_rank);
int sifar_symchain_destroy(sifar_symchain *chain);

/*
 * Generator probes (for tests and for building inputs on the device): write the
 * first partial of `rank`, or its partial of step t >= 2 from prev_out, as n plain
 * elements of `dtype` to dst (device, 16-byte aligned).
 */
int sifar_workload_first(const sifar_workload *w, int rank, int dtype, void *dst, size_t n, void *stream);
int sifar_workload_next(const sifar_workload *w, int rank, unsigned t, int dtype, const void *prev_out,
                        void *dst, size_t n, void *stream);
/* The seeded producer delays of ranks 0..P-1 at step t, computed on the device, copied to host_out[P]. Synchronizes. */
int sifar_workload_delays(const sifar_workload *w, int P, unsigned t, unsigned *host_out);

/*
 * Loads the code of the helper and producer kernels of this library on the current
 * device.  With lazy module loading (the CUDA default) the first launch of a kernel
 * loads it, and that load can wait until the device is idle: a helper launched for
 * the first time while a reducer already polls for its data would block the host
 * until that reducer gave up.  Call once before scripting such orderings (the
 * Python binding does when it loads the library on a machine with a GPU; chain
 * creation does for what a chain launches).  Kernels of sifar.h are loaded by
 * sifar_create.
 */
int sifar_workload_preload(void);

/*
 * Enqueue a kernel that busy-waits `ns` nanoseconds (at most 50 ms) on `stream`:
 * used to force producer / reducer orderings in tests and benchmarks.
 */
int sifar_spin(unsigned ns, void *stream);

/*
 * Stand-ins for a caller's own fused producer (tests): store a part of a rank's
 * partial for call number `tag` with the device helpers of sifar_device.cuh, on
 * `stream`.  src: n plain elements (device, 16-byte aligned).
 * sifar_store_slots:  slots [first_slot, first_slot + nslots) of the tagged-slot
 *                     format into `slots` (the pointer sifar_rank_buffer() returned).
 * sifar_store_blocks: blocks [first_block, first_block + nblocks) of the flagged-tile
 *                     format as plain elements into `dst` (the same pointer), each
 *                     followed by the release of its flag; flags / stride_words as
 *                     returned by sifar_tile_flags().
 */
int sifar_store_slots(const void *src, void *slots, size_t first_slot, size_t nslots, size_t n, int dtype,
                      unsigned tag, void *stream);
int sifar_store_blocks(const void *src, void *dst, void *flags, size_t stride_words, size_t first_block,
                       size_t nblocks, size_t n, int dtype, unsigned tag, void *stream);

/*
 * 16-byte access atomicity check (the speculative slots rely on it): `writers`
 * CTAs keep overwriting `nslots` slots with patterns whose four words all derive
 * from one counter, while reader CTAs load them with the slot load and count
 * slots whose words disagree.  Runs `rounds` rounds, all co-resident (cooperative
 * launch), bounded.  *host_torn receives the number of torn observations,
 * *host_reads the number of slot reads.  Synchronizes.
 */
int sifar_tear_check(unsigned nslots, unsigned rounds, unsigned long long *host_torn,
                     unsigned long long *host_reads);

#ifdef __cplusplus
}
#endif
#endif /* SIFAR_WORKLOAD_H */
