/*
 * attn.h -- C ABI of the B200 (sm_100a) fused attention forward library.
 *
 * The operation is the one the paper states in Section 2.2 ("Attention computation"):
 *
 *     O = softmax(Q K^T * scale [+ causal mask]) V
 *
 * evaluated tile by tile with a running row maximum and row sum (the FlashAttention
 * scheme the same section describes), for multi-head attention (Section 4.2) and
 * grouped-query attention (Section 4.3), BF16 inputs, head dimension 128
 * (Section 4.1, "Benchmark Configurations").  In addition the library returns the
 * per-row log-sum-exp of the scaled visible scores, which the paper does not mention.
 *
 * Everything is `extern "C"`, plain pointers and integers.  No entry point throws,
 * aborts or prints; each returns an attn_status_t.
 */
#ifndef ATTN_B200_ATTN_H_
#define ATTN_B200_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ATTN_OK = 0,
  ATTN_ERR_NULL = 1,        /* a required pointer is NULL */
  ATTN_ERR_SHAPE = 2,       /* a dimension is <= 0, or Hq is not a multiple of Hkv */
  ATTN_ERR_UNSUPPORTED = 3, /* D != 128; scale not finite or <= 0; sizes beyond the index range */
  ATTN_ERR_ALIGN = 4,       /* q, k, v or o not 16-byte aligned; lse not 4-byte aligned */
  ATTN_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed (descriptor, launch, copy) */
  ATTN_ERR_ARCH = 6,        /* the current device is not compute capability 10.x */
  ATTN_ERR_TIMEOUT = 7,     /* a bounded wait inside a kernel expired (see attn_last_device_status) */
  ATTN_ERR_TOO_LARGE = 8    /* attn_fwd_noalloc: the problem exceeds ATTN_NOALLOC_MAX_Q_TILES;
                               attn_fwd_splitkv: the workspace is too small */
} attn_status_t;

/*
 * attn_fwd -- fused attention forward (Section 2.2; GQA head mapping per Section 4.3:
 * consecutive query heads share a key/value head, hkv = hq / (Hq / Hkv)).
 *
 * All pointers are DEVICE pointers on the current device, owned by the caller; the
 * library neither frees nor retains them.  The call is asynchronous: work is enqueued
 * on `stream` and the function returns without synchronising.
 *
 *   q    BF16 [B, Sq, Hq,  D]  contiguous, D innermost            (read)
 *   k    BF16 [B, Sk, Hkv, D]                                     (read)
 *   v    BF16 [B, Sk, Hkv, D]                                     (read)
 *   o    BF16 [B, Sq, Hq,  D]  rounded to nearest even from fp32  (written)
 *   lse  FP32 [B, Hq, Sq]      natural-log sum of exp(scale * q.k_j) over the visible
 *                              keys of each row; may be NULL to skip   (written)
 *   B, Hq, Hkv, Sq, Sk  any positive sizes (lengths need not be multiples of the
 *                       128-row tile); Hq % Hkv == 0
 *   D        must be 128
 *   causal   0: every key is visible.  non-zero: key j is visible to query i iff
 *            j <= i + (Sk - Sq)  (lower-triangular when Sq == Sk).  With Sq > Sk the
 *            first Sq - Sk rows see no key: their o is 0 and their lse is -infinity
 *   scale    multiplies Q K^T; finite and > 0 (callers normally pass 1/sqrt(D))
 *   stream   cudaStream_t (NULL = default stream)
 *
 * o must not alias q, k or v.  Distinct streams may call concurrently.  The first
 * call on a device allocates a few KB of library-owned device state (tile-scheduler
 * counters and a status word); tensors are never allocated.  After that first call,
 * attn_fwd issues only a 4-byte cudaMemsetAsync and one kernel launch on `stream`, so it
 * can be captured into a CUDA graph; replays of one captured call share a work counter
 * and must not overlap each other.
 * Work counters: the library owns a pool of 1024 four-byte counters per device and gives each
 * call the next one, round-robin; the call's memset clears it on `stream` just before its
 * kernel.  Two launches that use the same counter must not be resident on the GPU together.
 * That cannot happen while fewer than 1024 calls (all entry points that launch the forward
 * kernel counted, attn_fwd_host and attn_fwd_splitkv one per chunk or key range) are queued
 * or running across all streams of the device.  It can happen when more are, and when a
 * captured graph -- which keeps the counter its call was given at capture -- is replayed on
 * one stream while the 1024th later call runs on another: serialise such a replay against the
 * other streams, or re-capture.
 * Arithmetic: S and O accumulate in fp32 on the tensor cores; P = exp2 of the scaled,
 * max-subtracted scores is rounded to BF16 before P V; the row sum is taken in fp32
 * before that rounding.
 */
attn_status_t attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                       int B, int Hq, int Hkv, int Sq, int Sk, int D,
                       int causal, float scale, void* stream);

/*
 * attn_fwd_strided -- attn_fwd on strided views (the paper states no memory layout; this
 * entry point takes any layout whose head dimension is contiguous).
 *
 * Same operation, arithmetic, result and rules as attn_fwd.  q, k, v, o are indexed as
 *   x[b, s, h, d] = base[b * strides[0] + s * strides[1] + h * strides[2] + d]
 * with x_strides = {batch, sequence, head} strides in ELEMENTS (host arrays of 3, read
 * during the call only).  Examples: a [B, H, S, D] buffer is {H*S*D, D, S*D}; the q slice of
 * a packed [B, S, 3, H, D] projection is {3*S*H*D, 3*H*D, D} with base + 0; the keys
 * s0 .. s0+n of a longer sequence are the same strides with base + s0 * strides[1] and
 * Sk = n (attn_merge combines the partial results of disjoint key ranges).  lse is always
 * contiguous [B, Hq, Sq].
 *
 * Every stride must be positive and a multiple of 8 elements (16 bytes: the tiles move by
 * TMA), the sequence and head strides at least 128, all below 2^39 elements; an axis of
 * extent 1 still needs a legal value.  Errors: ATTN_ERR_NULL for a missing stride array,
 * ATTN_ERR_SHAPE for a stride <= 0 or < 128 where rows would overlap, ATTN_ERR_ALIGN for a
 * stride that is not a multiple of 8, ATTN_ERR_UNSUPPORTED beyond the range, and
 * ATTN_ERR_CUDA if the driver rejects the resulting descriptor.  Rows addressed by
 * different (b, s, h) of o must not overlap; the inputs may overlap each other freely.
 */
attn_status_t attn_fwd_strided(const void* q, const void* k, const void* v, void* o, float* lse,
                               int B, int Hq, int Hkv, int Sq, int Sk, int D,
                               const long long* q_strides, const long long* k_strides,
                               const long long* v_strides, const long long* o_strides,
                               int causal, float scale, void* stream);

/*
 * attn_fwd_host -- the same operation on HOST buffers (same layouts).  Copies q, k, v
 * to library-owned device staging buffers (grown on demand, kept for later calls),
 * runs the forward, copies o and lse (if not NULL) back and synchronises `stream` before
 * returning; the work starts after whatever is already queued on `stream`.
 * Query rows are independent, so by default the call is pipelined: chunks of whole
 * 256-row work items (about one wave of CTAs each) are uploaded, computed (one strided
 * launch per chunk) and downloaded on three library-owned streams, so that host-to-device
 * copies, kernels and device-to-host copies overlap; under the causal mask a chunk waits
 * only for the keys its rows can see.  Results are bit-identical to attn_fwd on the same
 * data.  Option "host_pipeline" = 0 selects the plain copy / launch / copy sequence (also
 * used for causal problems with Sq > Sk).  The overlap needs pinned host memory; pageable
 * memory works, serialised by the driver.  Not re-entrant: one call at a time per process.
 */
attn_status_t attn_fwd_host(const void* q, const void* k, const void* v, void* o, float* lse,
                            int B, int Hq, int Hkv, int Sq, int Sk, int D,
                            int causal, float scale, void* stream);

/*
 * attn_fwd_noalloc -- attn_fwd for callers that must not allocate device memory.
 * (The paper has no counterpart; this is a convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a memory budget that
 * was handed out in full at start-up (an inference server that pre-reserves all of HBM for
 * its own pools), on a latency-critical thread that may not take the driver's allocation
 * lock, or in an embedding runtime that forbids library-side allocations altogether.
 * attn_fwd allocates a few KB of scheduler state with cudaMalloc on its first call per
 * device; this entry point never calls cudaMalloc, cudaFree or any allocating routine.
 *
 * Same arguments, layouts, arithmetic and results as attn_fwd (device pointers, asynchronous
 * on `stream`).  The kernel's scratch -- the tile scheduler's work counter and the status
 * words of its bounded waits -- lives in a 256-byte array that is part of the library image,
 * so every GPU that loads the library carries those 256 bytes until the process exits.
 *
 * Limits and rules:
 *   - B * Hq * ceil(Sq / 128) must not exceed ATTN_NOALLOC_MAX_Q_TILES, else
 *     ATTN_ERR_TOO_LARGE is returned and nothing is launched.
 *   - All calls on a device share the one scratch array.  Each call clears the words that
 *     must start at zero (on `stream`, before its kernel), so back-to-back calls on one
 *     stream are fine; two calls whose kernels can overlap on the GPU (different streams,
 *     no dependency) race on the work counter and give wrong results.  Use attn_fwd there.
 *   - The first call on each device looks up the array's device address and sets the
 *     kernel's shared-memory attribute; make that first call outside any stream capture.
 *   - Expired bounded waits are recorded in the scratch array only; no API reads them back.
 */
#define ATTN_NOALLOC_MAX_Q_TILES (1 << 20)
attn_status_t attn_fwd_noalloc(const void* q, const void* k, const void* v, void* o, float* lse,
                               int B, int Hq, int Hkv, int Sq, int Sk, int D,
                               int causal, float scale, void* stream);

/* Releases the staging buffers attn_fwd_host holds on the current device. */
attn_status_t attn_release_host_staging(void);

/*
 * attn_set_option -- tuning / A-B switches; returns ATTN_ERR_UNSUPPORTED for an
 * unknown name or value.  (The paper's Section 5 analyses such design choices one at a time;
 * these switches exist to measure them.)  Options are PROCESS-WIDE: one set of values for every
 * device, stream and thread, read by each entry point when it is called.  Setting an option is
 * atomic, but it is not synchronised with launches: a call that another thread makes while an
 * option changes may see the old or the new value, and two threads that want different values
 * cannot both have them.  Set options once, before the threads that launch are started, or keep
 * all calls on one thread.  attn_get_option reads a value back.  Defaults: scheduler 2,
 * max_ctas 0, rescale_threshold 8, split_p 1, overlap_epilogue 1, gqa_pack 1, host_pipeline 1,
 * kernel 0.
 *   "scheduler"   0 = one CTA per work item (hardware block scheduler)
 *                 1 = persistent CTAs, static round-robin over work items
 *                 2 = persistent CTAs, dynamic work counter (default)
 *   "max_ctas"    0 = one per SM (default), else an upper bound on persistent CTAs
 *   "rescale_threshold"  0..64 (default 8): log2 units by which a row's reference maximum may
 *                 lag its true running maximum before the O accumulator is rescaled; 0 rescales
 *                 whenever the maximum moves (the paper's Section 5.1 discusses this step)
 *   "split_p"     1 (default) = P is handed to the MMA warp in two halves of 64 keys, so the
 *                 first half of P V overlaps the second half of the exponentials; 0 = in one piece
 *                 ("kernel" = 0 only)
 *   "overlap_epilogue"  1 (default) = a query stage is normalised and stored as soon as its own
 *                 last P V has completed, overlapping the other stage's (Section 5.2);
 *                 0 = only after both stages' last P V ("kernel" = 0 only)
 *   "gqa_pack"    1 (default) = when a GQA group's query rows all fit two tiles
 *                 (Sq <= 2 * 128 / group, group a power of two <= 16, "kernel" = 0), the heads of
 *                 a KV group share the rows of a tile, so its K/V is streamed once for the whole
 *                 group (decoding, short chunks); results are bit-identical; 0 = never
 *   "host_pipeline"  1 (default) = attn_fwd_host overlaps upload, compute and download in row
 *                 chunks; 0 = one upload, one launch, one download
 *   "kernel"      0 = dual query stage: a CTA runs two 128-row query tiles against one stream
 *                     of K/V tiles, one score buffer each (default)
 *                 1 = triple score buffer: a CTA runs one query tile with three score tiles
 *                     in flight and two softmax groups that alternate K/V blocks
 *                 2 = dual query stage on CTA pairs: two CTAs (a cluster) share every
 *                     tcgen05.mma (M = 256), so a work item is four query tiles and each CTA
 *                     loads and keeps only half of every K/V tile; same arithmetic per row as
 *                     "kernel" = 0.  Problems that "gqa_pack" packs run "kernel" = 0.
 *                 3 = two softmax threads per query row: the default kernel with sixteen softmax
 *                     warps (each thread exponentiates 64 of a block's 128 keys; partial row
 *                     maxima are exchanged once per block, partial row sums once per work item)
 *                     and no separate epilogue warps; the row sum is added up in another order,
 *                     so results differ from "kernel" = 0 by rounding.  Packed problems run
 *                     "kernel" = 0.
 */
attn_status_t attn_set_option(const char* name, int value);
/* *value = the current setting of option `name` (host only); ATTN_ERR_UNSUPPORTED for an unknown name. */
attn_status_t attn_get_option(const char* name, int* value);

/*
 * attn_plan / attn_plan_item -- host-only introspection of the tile scheduler (Section 2.2's
 * "processes key blocks sequentially" per query tile, and the causal case where some key
 * blocks are fully masked and skipped).  No device is touched.
 *
 * attn_plan fills plan[0..5] = { n_work, pair_heads, items_per_group, n_q_tiles,
 * n_kv_blocks, ctas } for a problem, where `ctas` is the grid a launch on a device with
 * `sm_count` SMs would use under the current options.  A work item is two 128-row query
 * tiles ("stages") that share one stream of K/V tiles: two consecutive row tiles of one
 * query head (pair_heads = 0), or the same row tile of two query heads that share a KV
 * head (pair_heads = 1, used when Hq / Hkv is even).
 *
 * attn_plan_item fills item[0..7] = { b, hkv, hq0, hq1, row0_0, row0_1, n_blocks_0,
 * n_blocks_1 } for work item `w` in launch order (causal: longest items first inside each
 * head).  n_blocks_s = 0 marks an unused stage (its rows lie beyond Sq; with "kernel" = 1
 * every item has one tile and stage 1 is always unused).
 * Both return ATTN_ERR_SHAPE / ATTN_ERR_UNSUPPORTED like attn_fwd, ATTN_ERR_SHAPE for w
 * out of range.
 *
 * With "kernel" = 2 a work item belongs to a pair of CTAs and holds four tiles: `ctas` is
 * twice the number of pairs, and attn_plan_item_pair gives the item as CTA `rank` (0 = the
 * leader, 1 = its peer) of the pair sees it, in the layout of attn_plan_item: with
 * pair_heads = 0 stage s of CTA c holds row tile 4 r + 2 s + c of one head, with
 * pair_heads = 1 the stages hold two query heads and CTA c row tile 2 r + c.  Both CTAs
 * report the same n_blocks_s (the two tiles of a stage are multiplied by the same
 * instructions); a tile whose row0 lies beyond Sq is computed and discarded.
 * attn_plan_item returns the leader's view.  attn_plan_item_pair returns
 * ATTN_ERR_UNSUPPORTED when the plan in force is not the pair kernel's.
 */
attn_status_t attn_plan(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, int sm_count, int* plan);
attn_status_t attn_plan_item(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, int w, int* item);
attn_status_t attn_plan_item_pair(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, int w, int rank,
                                  int* item);

/* Human-readable name of a status code (static storage). */
const char* attn_status_str(attn_status_t status);

/* Library version: major * 10000 + minor * 100 + patch. */
int attn_version(void);

/*
 * attn_last_device_status -- synchronises the current device and reads the status word
 * kernels write when one of their bounded waits expires.  *code is 0 when nothing
 * expired, else identifies the waiting role; *detail identifies the barrier.  Returns
 * ATTN_ERR_TIMEOUT when *code != 0 (the word is then cleared), ATTN_OK otherwise.
 */
attn_status_t attn_last_device_status(int* code, int* detail);

/*
 * attn_last_launch_clock -- the SM clock the most recent launch of a forward kernel ("kernel" =
 * 0, 2 or 3, through attn_fwd, attn_fwd_strided, attn_fwd_host or attn_fwd_splitkv) actually
 * ran at on the current device: its first CTA, which lives as long as the launch, reads the SM
 * cycle counter and the nanosecond timer when it starts and when it ends.  *sm_mhz = cycles /
 * time, *kernel_ms = that CTA's lifetime.  A measurement aid for benchmarks (the paper reports
 * throughput on a part whose clock moves under its power limit; Section 4.1): NVML's clock reading
 * lags a launch of a few milliseconds.  Synchronises the device.  ATTN_ERR_UNSUPPORTED when no such
 * launch has finished yet.
 */
attn_status_t attn_last_launch_clock(double* sm_mhz, double* kernel_ms);

/*
 * attn_launch_clocks -- the same measurement for the most recent launches, newest first: the
 * library keeps the stamps of the last 64 launches of a stamping kernel per device (a ring indexed
 * by a launch counter).  Fills sm_mhz[0 .. *n - 1] (HOST array of max_n doubles) with the SM clock
 * each of them ran at, *n <= min(max_n, 64).  A benchmark reads it once after its timed region and
 * gets the clock of EVERY timed launch (the paper's Section 4.1 reports means over repeated runs on
 * a part whose clock drifts under its power limit), so that time x clock -- cycles per unit of work
 * -- can be compared between runs at different clocks.  Synchronises the device.  *kernel_ms of
 * attn_last_launch_clock is the first CTA's lifetime, which can be one work item shorter than the
 * launch; time launches with events.
 */
attn_status_t attn_launch_clocks(double* sm_mhz, int max_n, int* n);

/*
 * attn_merge -- combines two partial attention results that were computed over DISJOINT sets of
 * keys for the same queries (e.g. two attn_fwd calls on the two halves of K and V, non-causal):
 *
 *     LSE = log(exp(LSE1) + exp(LSE2)),   O = exp(LSE1 - LSE) * O1 + exp(LSE2 - LSE) * O2
 *
 * which is the attention over the union of the keys -- a direct consequence of the softmax
 * definition of Section 2.2 and the reason attn_fwd returns LSE.  It is what a caller needs to
 * split a long key sequence over several launches or devices.
 *
 *   o1, o2   BF16 [B, Sq, Hq, D] device pointers (read), 16-byte aligned
 *   lse1/2   FP32 [B, Hq, Sq] (read); -inf marks a part that saw no key (weight 0)
 *   o        BF16 [B, Sq, Hq, D] (written; may be the same buffer as o1 or o2)
 *   lse      FP32 [B, Hq, Sq]    (written; must not alias lse1 or lse2)
 *   D        must be 128
 * Asynchronous on `stream`.  Arithmetic in fp32, O rounded to nearest-even BF16.  If both parts
 * are empty the row is O = 0, LSE = -inf.
 */
attn_status_t attn_merge(const void* o1, const float* lse1, const void* o2, const float* lse2,
                         void* o, float* lse, int B, int Hq, int Sq, int D, void* stream);

/*
 * attn_merge_n -- the same identity for n parts at once (1 <= n <= 64), stored back to back:
 *
 *     LSE = log(sum_i exp(LSE_i)),   O = sum_i exp(LSE_i - LSE) * O_i
 *
 *   o_parts    BF16 [n][B, Sq, Hq, D] device pointer (read), 16-byte aligned
 *   lse_parts  FP32 [n][B, Hq, Sq] (read); -inf marks an empty part, whose O_i is not read
 *   o          BF16 [B, Sq, Hq, D] (written; must not overlap o_parts)
 *   lse        FP32 [B, Hq, Sq] (written; may be NULL to skip)
 * Asynchronous on `stream`; fp32 accumulation, one rounding of O to BF16.  Rows whose parts are
 * all empty get O = 0, LSE = -inf.  ATTN_ERR_UNSUPPORTED for D != 128 or n > 64.
 */
attn_status_t attn_merge_n(const void* o_parts, const float* lse_parts, int n, void* o, float* lse,
                           int B, int Hq, int Sq, int D, void* stream);

/*
 * attn_fwd_splitkv -- attn_fwd for few query rows against many keys (decoding, short chunks of a
 * long context), where one launch has too few 256-row work items to fill the GPU.  The key
 * sequence is cut into up to n_splits ranges of whole 128-key tiles; each range is one launch
 * of the forward kernel on views of k and v (under the causal mask with the offset that keeps
 * the global key indices; a range no key of which a row may see leaves that row empty), the
 * launches run concurrently on library-owned streams, and attn_merge_n combines the partial
 * results.  The paper's workloads (Sq = Sk) never need this; it is the use the returned LSE
 * makes possible.
 *
 * Arguments as attn_fwd (contiguous layouts), plus:
 *   n_splits         1..64; fewer ranges are used when Sk is short (one 128-key tile per range
 *                    at least); with a single range this is attn_fwd
 *   workspace        device buffer for the partial results, 16-byte aligned, owned by the caller,
 *                    at least attn_splitkv_workspace_bytes(B, Hq, Sq, D, n_splits) bytes
 *                    (n_splits * B * Sq * Hq * (2 * D + 4)); may be NULL when n_splits == 1
 * Result: the same attention; each partial O is rounded to BF16 before the merge, so O carries
 * up to two more BF16 roundings than attn_fwd's.  Work on `stream` queued before the call is
 * waited for, and `stream` continues after the merge.  One call at a time per device (the
 * library's streams and events are shared).  ATTN_ERR_TOO_LARGE if the workspace is too small.
 */
size_t attn_splitkv_workspace_bytes(int B, int Hq, int Sq, int D, int n_splits);
attn_status_t attn_fwd_splitkv(const void* q, const void* k, const void* v, void* o, float* lse,
                               int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale,
                               int n_splits, void* workspace, size_t workspace_bytes, void* stream);

/*
 * attn_selftest_wait_timeout -- exercises the bounded waits every kernel of this library uses
 * between its warp roles (the paper's kernels hand work between MMA, softmax, correction and
 * load warps "with barrier-based signaling", Section 2.2; here every such wait has a time limit).
 * Launches one warp that waits on a barrier nobody signals; after `limit_ms` (1..1000) the wait
 * gives up, the kernel returns normally and attn_last_device_status() reports ATTN_ERR_TIMEOUT
 * with *code = 0x905.  Nothing faults or hangs; later calls on the device work as usual.
 * Asynchronous on `stream`.
 */
attn_status_t attn_selftest_wait_timeout(int limit_ms, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_B200_ATTN_H_ */
