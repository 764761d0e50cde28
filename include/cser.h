/*
 * cser.h - C ABI of the B200 (sm_100a) CSER / M-CSER optimizer-step library.
 *
 * What it computes.  n simulated workers each hold a local model x_i, a local
 * error e_i and (with momentum) a local momentum m_i, all vectors of d fp32
 * elements, stored as row-major [n, d] arrays in one GPU's memory.  One call of
 * cser_step() performs one iteration t of "CSER" (Algorithm 2) or, when beta != 0,
 * of "M-CSER, implementation I" (Algorithm 4) of arXiv 2007.13221 for all workers:
 *
 *   1. Get_p (Appendix A.4):    m_i <- beta*m_i + g_i ;  p_i <- eta*(beta*m_i + g_i)
 *                               (beta == 0:  p_i <- eta*g_i)
 *   2. PSync(p, C) (Algorithm 3) with the GRBS compressor of Definition 2:
 *        selected blocks:    x_i <- x_i - mean_k p_k        (e_i unchanged)
 *        unselected blocks:  x_i <- x_i - p_i ;  e_i <- e_i - p_i
 *   3. if t mod H == 0, error reset (Algorithm 2 lines 11-12) with a second,
 *      independently drawn GRBS mask, on its selected blocks only:
 *        x_i <- (x_i - e_i) + mean_k e_k ;  e_i <- 0
 *
 * The mean over the worker axis is what a deployment would do with an allreduce.
 *
 * Naming.  R1 is the compression ratio of the compressor applied to the update
 * every step (the paper's Algorithm 2 calls it C_2); R2 is the ratio of the
 * compressor applied to the error every H steps (the paper's C_1).
 *
 * GRBS mask (Definition 2).  The vector is cut into B = ceil(d / block_size)
 * contiguous blocks.  Block b is selected at step t for compressor s (0 = update,
 * 1 = reset) iff  word0 * R < 2^32, where word0 is the first output word of
 * Philox4x32-10 with key = (seed & 0xffffffff, seed >> 32) and counter =
 * (b, t & 0xffffffff, t >> 32, s).  R = 1 selects every block; for any R each
 * block is selected independently with probability ceil(2^32/R)/2^32 (= 1/R for
 * powers of two), so the compressor is 1/R-approximate in expectation.
 *
 * Arithmetic.  fp32, round-to-nearest, no fused multiply-add, no flush-to-zero.
 * Order: t1 = beta*m; m' = t1+g; t2 = beta*m'; t3 = t2+g; p = eta*t3.  Sums over
 * workers run in ascending worker order starting from worker 0's value; the mean
 * is sum / (float)n.  The reset computes (x - e) first, then adds the mean.
 *
 * Conventions.  t is 0 after cser_create / cser_set_x0; the first cser_step is
 * t = 1; resets happen at t = H, 2H, ...  All pointers named "device" must be
 * device memory of the GPU that was current when the handle was created.  A
 * `stream` argument is a cudaStream_t passed as void* (NULL = the legacy default
 * stream).  Every call that takes a stream only enqueues work on it and returns;
 * the caller synchronizes.  Calls on one handle must not run concurrently.
 *
 * Errors.  Functions returning int give 0 on success or a negative code below;
 * cser_last_error() returns a thread-local message for the last failure.  No call
 * aborts, throws, or traps on the device.  The only device-side waits are those of the
 * opt-in kernel of CSER_FLAG_STAGED_SELECTED (a kernel waiting for its own asynchronous
 * copies into shared memory); they are bounded to about a second, and one that ran out
 * raises a host-visible word in the handle: every later cser_step / cser_read_state on
 * that handle then returns CSER_ERR_CUDA, the step it happened in being incomplete.
 */
#ifndef CSER_H_
#define CSER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CSER_OK             0
#define CSER_ERR_INVALID   -1   /* bad argument (NULL, non-positive size, bad ratio, misuse)   */
#define CSER_ERR_NOMEM     -2   /* device or host allocation failed                            */
#define CSER_ERR_CUDA      -3   /* a CUDA runtime call or a kernel launch failed               */
#define CSER_ERR_TOO_SMALL -4   /* destination / source buffer smaller than the state it holds */

/* `which` of cser_read_state / cser_write_state */
#define CSER_STATE_X       0    /* fp32 [n, d]  local models                                   */
#define CSER_STATE_E       1    /* fp32 [n, d]  local errors                                   */
#define CSER_STATE_M       2    /* fp32 [n, d]  local momenta (only when beta != 0)            */
#define CSER_STATE_MASK_G  3    /* uint8 [B]    update mask of the last step                   */
#define CSER_STATE_MASK_R  4    /* uint8 [B]    reset mask of the last reset step              */
#define CSER_STATE_T       5    /* uint64       step counter t (host value, copied immediately) */

typedef struct cser_ctx *cser_handle;

/*
 * Create an optimizer state for n_workers x d on the current device (Algorithm 2
 * line 2 / Algorithm 4 line 2: x = 0 until cser_set_x0, e = 0, m = 0, t = 0).
 *   d           > 0, elements per worker
 *   n_workers   > 0
 *   block_size  > 0, elements per GRBS block (last block may be short)
 *   R1          compression ratio of the update compressor; R1 = 1 keeps everything,
 *               R1 = 0 keeps nothing (C = 0: the special cases CSER-PL and, with H = 1,
 *               CSEA of Appendix A.1, where nothing is exchanged between resets)
 *   R2          >= 1, compression ratio of the reset compressor
 *   H           > 0, error-reset interval
 *   eta         finite learning rate;  beta in [0, 1): 0 = no momentum (m is not
 *               allocated, read or written)
 *   seed        shared GRBS seed
 * The library owns x, e, m and the masks (about (2 or 3)*n*d*4 bytes of device
 * memory) until cser_destroy.  Returns NULL on failure.
 */
cser_handle cser_create(int64_t d, int32_t n_workers, int32_t block_size,
                        uint32_t R1, uint32_t R2, int32_t H,
                        float eta, float beta, uint64_t seed);

/*
 * Same, for one column slab of a longer vector that several GPUs share by
 * columns: this handle holds blocks block_begin .. block_begin + ceil(d/block_size) - 1
 * of the global vector, and draws its masks with those global block ids, so that
 * every slab sees the mask the whole vector would see (Section 3.3: all workers
 * pick the same blocks from the synchronized seed).  No data is exchanged.
 */
cser_handle cser_create_slab(int64_t d, int32_t n_workers, int32_t block_size,
                             uint32_t R1, uint32_t R2, int32_t H,
                             float eta, float beta, uint64_t seed, int64_t block_begin);

/*
 * General form.  flags:
 *   CSER_FLAG_NO_ERROR_ARRAY  "implementation II" of Appendix A.4: with GRBS a block's
 *       residual is either already part of the local model or reset to zero, so no error
 *       array is kept; on a reset step the reset-selected blocks of x are replaced by
 *       their mean over workers (PSync applied to x itself).  State is x (and m) only;
 *       CSER_STATE_E cannot be read or written.  The models equal implementation I's up
 *       to rounding.
 */
#define CSER_FLAG_NO_ERROR_ARRAY 1u
/*
 *   CSER_FLAG_EXACT_COUNT  Definition 2 read literally ("picks B/R random blocks"): every
 *       mask selects exactly k = round(B / R) blocks (halves up; R = 0 gives 0), namely the
 *       k blocks with the smallest keys (word0, block id), word0 being the same Philox draw
 *       the default mode thresholds.  Each block is still selected with probability k / B
 *       and the bytes moved per step no longer fluctuate.  Needs block_begin = 0 and at most
 *       2^22 blocks.
 */
#define CSER_FLAG_EXACT_COUNT 2u
/*
 *   CSER_FLAG_L2_RESIDENT  if x, e and m together fit the part of the GPU's L2 cache that can
 *       be set aside for persisting lines (about 79 MB on B200), keep them there: the step
 *       kernels are launched with an access-policy window over the state, so only the
 *       gradients stream from HBM.  The set-aside is a limit of the whole CUDA context: it
 *       takes that much L2 away from every other kernel of the process until the handle is
 *       destroyed, which is why it is opt-in.  Ignored when the state does not fit.
 */
#define CSER_FLAG_L2_RESIDENT 4u
/*
 *   CSER_FLAG_STAGED_SELECTED  the blocks selected by a mask (Algorithm 3 line 7: the mean over
 *       workers) are normally handled by a kernel in which a thread walks the worker axis of its
 *       column with a few loads held in registers.  With this flag they go through an alternative
 *       kernel instead, which brings all workers' segments of a block into shared memory with
 *       asynchronous bulk copies (a producer warp, a ring of stages, shared-memory barriers with
 *       bounded waits) and reduces from there.  Results are bit-identical.  On B200 the alternative is
 *       slower at every ratio that was measured, which is why it is opt-in; it is kept so that the
 *       comparison can be repeated.  It needs d and block_size to be multiples of 4, blocks of at
 *       least 64 elements and few enough workers for one stage of shared memory; otherwise the flag
 *       has no effect.
 */
#define CSER_FLAG_STAGED_SELECTED 8u
/*
 *   CSER_FLAG_THREE_KERNELS  an iteration of a large problem is three kernels (block select, streaming
 *       kernel for the unselected blocks, selected-block kernel beside it).  cser_step runs an iteration
 *       as ONE kernel instead, which draws the masks itself and walks every column over the workers
 *       (same Philox draws, same arithmetic, bit-identical results), in two cases: when the iteration
 *       moves at most 256 MB (n_workers * d * 28 bytes with momentum and an error array), because it
 *       would take a few tens of microseconds and the kernel boundaries would cost as much as the
 *       traffic; and when a large share of the blocks is selected in that iteration (with up to 8
 *       workers: 1/R1 >= 1/4 on an ordinary step, 1/R1 + 1/R2 >= 1/10 on a reset step; with 9 to 16
 *       workers: R1 = 1, or 1/R1 + 1/R2 >= 1/5 on a reset step), because walking all columns in their
 *       natural order then beats sending scattered blocks through the selected-block kernel.  This flag keeps the three kernels for every iteration.  Steps with injected masks,
 *       exact-count masks, replayable steps, cser_step_host and vectors whose d or block_size is not a
 *       multiple of 4 use the three kernels in any case.
 */
#define CSER_FLAG_THREE_KERNELS 16u
cser_handle cser_create_ex(int64_t d, int32_t n_workers, int32_t block_size,
                           uint32_t R1, uint32_t R2, int32_t H,
                           float eta, float beta, uint64_t seed, int64_t block_begin,
                           uint32_t flags);

/*
 * Free everything the handle owns (no passage of the paper: lifecycle).  The caller must have
 * synchronized its streams; the library waits for its own auxiliary stream.  NULL is ignored.
 */
void cser_destroy(cser_handle h);

/*
 * x_i <- x0 for every worker, e <- 0, m <- 0, t <- 0 (Algorithm 2 line 2).
 * x0: d fp32 values, host or device memory.
 */
int cser_set_x0(cser_handle h, const float *x0, void *stream);

/*
 * One iteration (Algorithm 2 lines 5-13 / Algorithm 4 lines 5-15) for all workers.
 * grad: device, fp32 [n, d] row-major with leading dimension d; borrowed, read-only,
 * must stay valid and unchanged until the work enqueued on `stream` has finished.
 * Increments t, then enqueues the step kernels (and, beside them, the GRBS select kernel of
 * the following iteration, whose masks depend only on seed and t; the first step, and a step
 * after cser_set_x0, cser_write_state(T) or cser_debug_set_masks, runs its own first).
 * The iteration number is passed to the kernels by value, so the launches of one call
 * belong to that iteration only: a stream capture of cser_step must not be replayed.
 */
int cser_step(cser_handle h, const float *grad, void *stream);

/*
 * Replayable steps, for callers that capture their training iteration in a CUDA graph.
 * Between cser_replay_begin and cser_replay_end the step counter lives in device memory and
 * is advanced by the step itself, so the launches enqueued by one call of
 * cser_step_replayable perform "the next iteration", whichever that is: they may be captured
 * once (stream capture of the call on `stream`) and replayed any number of times; every
 * replay is one more iteration of Algorithm 2 / 4 on whatever the gradient buffer then holds.
 * The call may also be used without capture.  Results are the same as cser_step's.
 * cser_replay_begin copies the host step counter to the device (and synchronizes `stream`);
 * cser_replay_end synchronizes `stream` and reads it back.  In between, cser_step,
 * cser_step_host, cser_set_x0, cser_write_state and cser_debug_set_masks are refused;
 * cser_read_state works (the step counter is read from the device).  Not available with
 * exact-count masks or worker-sharded handles.  grad must be the same pointer at replay time
 * as at capture time (a captured launch carries its arguments).  A handle whose iterations move
 * at most 256 MB replays as ONE kernel per step (see CSER_FLAG_THREE_KERNELS); it then needs a
 * 16-byte aligned grad.
 */
int cser_replay_begin(cser_handle h, void *stream);
int cser_step_replayable(cser_handle h, const float *grad, void *stream);
int cser_replay_end(cser_handle h, void *stream);

/*
 * The same iteration with the gradients in HOST memory (pinned memory gives
 * asynchronous copies): the library copies them, slab by slab, into a device
 * staging buffer it owns (allocated on the first such call, n*d*4 bytes) and runs
 * the step kernel on each slab as it lands, so copy and compute overlap.
 * Uses two internal streams that are ordered after `stream` at entry and joined
 * back into `stream` before returning.
 */
int cser_step_host(cser_handle h, const float *grad_host, void *stream);

/*
 * Copy one piece of state to dst (host or device), enqueued on `stream` (no passage of the paper:
 * inspection and checkpointing of the state of Algorithm 2 / 4: x_i, e_i, m_i, the masks, t).
 * dst_bytes must be at least the size of the piece: n*d*4 for x/e/m, B for a mask,
 * 8 for t.  CSER_STATE_M with beta == 0 is CSER_ERR_INVALID.
 */
int cser_read_state(cser_handle h, int which, void *dst, size_t dst_bytes, void *stream);

/*
 * Copy columns [col_begin, col_begin + col_count) of x, e or m, for all workers, into dst
 * (host or device) as a dense fp32 [n, col_count] array; enqueued on `stream`.  For looking
 * at part of a state that is too large to copy whole.
 */
int cser_read_columns(cser_handle h, int which, int64_t col_begin, int64_t col_count,
                      float *dst, size_t dst_elems, void *stream);

/*
 * Learning rate eta for the following steps (the schedules of Section 5.1 change it between
 * steps; Algorithms 2 and 4 take it as given).  Takes effect with the next cser_step.  A step
 * captured in a CUDA graph carries the eta of capture time: replays do not see a later change.
 */
int cser_set_lr(cser_handle h, float eta);

/*
 * Restore one piece of state from src (host or device) - the inverse of
 * cser_read_state, for checkpoint/resume (no passage of the paper: lifecycle).  `bytes` must be exactly the piece's size.
 * Masks cannot be written (use cser_debug_set_masks).
 */
int cser_write_state(cser_handle h, int which, const void *src, size_t bytes, void *stream);

/*
 * Test hook (no passage of the paper): the NEXT cser_step uses these block masks (uint8 [B] each, host or
 * device, non-zero = selected) instead of drawing them.  r_mask may be NULL if
 * that step is not a reset step.  The copy is enqueued on `stream`.
 */
int cser_debug_set_masks(cser_handle h, const uint8_t *g_mask, const uint8_t *r_mask, void *stream);

/*
 * Test hook for the bounded waits of the CSER_FLAG_STAGED_SELECTED kernel (no passage of the paper).
 * In the NEXT cser_step one CTA of that kernel is told to expect 16 bytes that no copy delivers, and every
 * wait is limited to wait_mcycles million SM clock cycles (1 .. 2000; the normal limit is 2000, about a
 * second).  The wait runs out, the CTA leaves, the kernel ends, and every later cser_step /
 * cser_read_state on the handle returns CSER_ERR_CUDA.  The state is then incomplete: destroy the handle.
 * Nothing traps and the CUDA context stays usable.
 */
int cser_debug_stall_next_staged_step(cser_handle h, unsigned wait_mcycles);

/*
 * Stand-alone GRBS block-select kernel (Definition 2): writes uint8 flags of blocks
 * block_begin .. block_begin + n_blocks - 1 at step t for compressor `which`
 * (0 = update, 1 = reset) with ratio R (0 = nothing selected) into device memory `mask_out`.
 */
int cser_grbs_mask(uint64_t seed, uint64_t t, uint32_t which, int64_t block_begin,
                   int64_t n_blocks, uint32_t R, uint8_t *mask_out, void *stream);

/*
 * Worker-sharded deployment (the paper's own setting, Section 3.3: GRBS is compatible with
 * all-reduce because every worker picks the same blocks).  This GPU holds n_local of the
 * n_total workers, all d columns.  Masks are exact-count GRBS, so the message length is
 * known on the host.  One iteration is
 *     cser_wshard_pack(h, grad, msg, ...)   select, update the unselected blocks, and write
 *                                           into msg the sum over the LOCAL workers of p on the
 *                                           update-selected blocks (ascending block order)
 *                                           followed, on a reset step, by the sum of
 *                                           e_{t-1/2} on the reset-selected blocks;
 *     sum msg over all ranks                (the caller's all-reduce, e.g. NCCL);
 *     cser_wshard_apply(h, msg, ...)        divide by n_total and finish the iteration.
 * Both PSyncs of a reset step (Algorithm 2 lines 6 and 11) share that one all-reduce.
 * cser_wshard_pack returns with msg complete in stream order on `stream`, while the update of the
 * unselected blocks still runs on a stream of the library's own: an all-reduce enqueued on
 * `stream` right after the call overlaps it.  cser_wshard_apply (and cser_read_state) wait for it.
 * msg: device, fp32, at least cser_wshard_message_elems(h, reset_step) elements
 * (reset_step = whether the NEXT iteration t+1 is a multiple of H); a short last block is
 * padded with zeros.  grad: device fp32 [n_local, d].  With one rank holding all workers the
 * result equals cser_step's (exact-count masks) bit for bit; across ranks the sum over
 * workers is associated rank by rank, so results agree to rounding.
 */
cser_handle cser_create_wshard(int64_t d, int32_t n_local, int32_t n_total, int32_t block_size,
                               uint32_t R1, uint32_t R2, int32_t H,
                               float eta, float beta, uint64_t seed);
int64_t cser_wshard_message_elems(cser_handle h, int reset_step);   /* -1 if h is not worker-sharded */
int cser_wshard_pack(cser_handle h, const float *grad, float *msg, size_t msg_elems, void *stream);
int cser_wshard_apply(cser_handle h, const float *msg, void *stream);

/*
 * Per-kernel timing (no passage of the paper: measurement).  With on != 0, cser_step brackets its
 * mask kernel and its step kernels with CUDA events on the launching stream.
 * cser_last_kernel_ms waits for the last step's events and returns both durations
 * in milliseconds (either pointer may be NULL).
 */
int cser_set_timing(cser_handle h, int on);
int cser_last_kernel_ms(cser_handle h, float *mask_ms, float *step_ms);

/* Number of kernels this library has launched on behalf of the handle. */
int64_t cser_launch_count(cser_handle h);

/*
 * One iteration without any allocation (the paper has no counterpart: this is a
 * calling convenience of this library, not a part of the algorithm).
 *
 * Who it is for: code that may not call cudaMalloc at the point where it steps the
 * optimizer - a host framework that owns all device memory through its own pool and
 * forbids driver allocations once training runs (cudaMalloc can stall every stream of
 * the device), a real-time loop that must not take the allocator's locks, or a plug-in
 * that is handed its buffers and has no right to create state of its own.  Such a
 * caller owns x, e and m itself (device, fp32 [n, d] row-major, updated in place) and
 * keeps the step counter; cser_create is never called and nothing has to be destroyed.
 *
 * It performs exactly the iteration `t` (1-based; resets when t mod H == 0) that
 * cser_step performs on a handle whose counter stands at t - 1, with the same kernels
 * and the same arithmetic.  m is ignored (may be NULL) when beta == 0.
 *
 * Scratch: the two GRBS masks and the list of selected blocks are kept in a fixed array
 * inside the library, in the device memory of every GPU that loads it, for the life of
 * the process (6 * CSER_NOALLOC_MAX_BLOCKS + 256 bytes = 1.5 MiB per GPU).  A vector with more than
 * CSER_NOALLOC_MAX_BLOCKS blocks (ceil(d / block_size)) is refused with
 * CSER_ERR_INVALID; choose a larger block_size or use the handle API.
 *
 * The first call on each device looks up the array's device address (no allocation,
 * but a runtime query); make that first call outside any stream capture.  As with
 * cser_step, t and the rotation of the list counters are launch arguments, so a stream
 * capture of the call must not be replayed.
 * All calls on a device share the one array: the masks and list of a call are
 * overwritten by the next.  Each call rewrites every entry it later reads and clears the
 * list counter the following call will use, so no clearing is needed between calls, but
 * two calls whose kernels may overlap on the GPU (different streams, or different host
 * threads) race on the array - serialize them on one stream and one host thread.  (Such
 * a race gives wrong masks, hence a wrong step; it cannot write outside the array or
 * outside the caller's arrays: list appends and list reads are bounded by the number of
 * blocks.)
 * No cudaMalloc, cudaFree or other allocating routine is called.
 */
#define CSER_NOALLOC_MAX_BLOCKS 262144
int cser_step_noalloc(int64_t d, int32_t n_workers, int32_t block_size,
                      uint32_t R1, uint32_t R2, int32_t H,
                      float eta, float beta, uint64_t seed, uint64_t t,
                      const float *grad, float *x, float *e, float *m, void *stream);

/* Thread-local description of the last error in this thread ("" if none).  No passage of the paper: error reporting. */
const char *cser_last_error(void);

/*
 * Identifier the build stamped into this binary (no passage of the paper: provenance): 16 hex digits
 * over the library's sources and compiler flags, "unstamped" if it was built by other means.
 */
const char *cser_build_id(void);

#ifdef __cplusplus
}
#endif
#endif /* CSER_H_ */
