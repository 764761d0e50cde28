// CSER / M-CSER optimizer step for B200 (sm_100a): host side of the C ABI declared in
// include/cser.h.  The kernels live in grbs_kernels.cuh (block selection),
// step_kernels.cuh (streaming and selected-block kernels) and wshard_kernels.cuh
// (worker-sharded pack / apply).
//
// Layout: g, x, e, m are fp32 [n, d] row-major (worker-major).  The step is bound
// by HBM traffic (about 28 bytes per element and worker against 7 flops), so the
// step is organised around how DRAM likes to be walked: the streaming kernel's grid
// is (workers x column tiles), dispatched tile-fastest, so the unselected blocks
// (all but 1/R of the data, purely elementwise) are streamed row after row as four
// long contiguous read streams and three write streams, every byte touched once.
// Blocks selected by a mask (1/R of the data) need the mean over workers: the
// select kernel compacts their ids into a list and a second kernel, with its own
// register budget, walks the worker axis for exactly those columns.  There is no
// contraction here and tensor cores are not used.
//
// Compiled with -fmad=false: every multiply and add rounds separately, in the
// order stated in include/cser.h.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdarg.h>
#include <string.h>
#include <math.h>
#include <new>

#include "cser.h"

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

#define CU_TRY(expr)                                                                      \
    do {                                                                                  \
        cudaError_t _e = (expr);                                                          \
        if (_e != cudaSuccess)                                                            \
            return fail(_e == cudaErrorMemoryAllocation ? CSER_ERR_NOMEM : CSER_ERR_CUDA, \
                        "%s: %s", #expr, cudaGetErrorString(_e));                         \
    } while (0)

#include "grbs_kernels.cuh"
#include "step_kernels.cuh"
#include "staged_kernel.cuh"
#include "wshard_kernels.cuh"

}  // namespace

// ------------------------------------------------------------------ handle
struct cser_ctx {
    long long d = 0, B = 0, block_begin = 0;
    long long Bpad = 0;                              // B rounded up to 16: distance between the two buffer sets
    int n = 0, bs = 0, H = 0, device = 0;
    uint32_t R1 = 1, R2 = 1;
    float eta = 0.f, beta = 0.f;
    uint64_t seed = 0, t = 0;
    float *x = nullptr, *e = nullptr, *m = nullptr;   // carved out of one allocation, state_base
    void *state_base = nullptr;
    size_t state_bytes = 0;
    // A state that fits the part of L2 that can be set aside for persisting lines is kept there:
    // the step kernels are launched with an access-policy window over the state.
    bool l2_persist = false;
    size_t l2_limit_before = 0;
    // Masks and list of the current step (aliases of one of the two buffer sets below).
    uint8_t *mask_g = nullptr, *mask_r = nullptr;
    uint32_t *sel_list = nullptr;                    // [B] blocks selected this step
    const uint32_t *cur_count = nullptr;             // how many
    uint8_t *last_mask_r = nullptr;                  // reset mask of the last reset step
    // The reset mask of reset number q = t / H lives in half q & 1 of the reset-mask allocation, so the
    // select kernel that prepares the next reset step never overwrites the last reset step's mask.
    uint8_t *mask_r_half[2] = {nullptr, nullptr};
    // The masks of an iteration depend only on (seed, t), so the select kernel of iteration
    // t + 1 runs during iteration t, beside the step kernels, into the other buffer set.
    struct SelBuf {
        uint8_t *mask_g = nullptr, *mask_r = nullptr;
        uint32_t *list = nullptr;
    } sb[2];
    int n_buf = 2, cur = 0;
    uint32_t *sel_count = nullptr;                   // [3] counters, used in rotation
    unsigned kseq = 0;                               // select-kernel launches so far
    bool pre_valid = false;                          // sb[cur ^ 1] holds iteration pre_t
    uint64_t pre_t = 0;
    const uint32_t *pre_count = nullptr;
    bool walk_all = false;                           // masks were injected: no estimate of the selected count
    // replayable steps (cser_replay_begin .. cser_replay_end): the iteration lives on the device
    ReplayCtl *ctl = nullptr;
    bool replay = false;
    bool replay_fused = false;                       // replayable steps go through the single-launch kernel
    // worker-sharded mode (cser_create_wshard): n = local workers, n_total = all ranks' workers
    int n_total = 0;
    // ordered lists of the selected blocks, one set per mask buffer set (allocations of 2 B entries)
    uint32_t *pos_g = nullptr, *pos_r = nullptr, *olist_g = nullptr, *olist_r = nullptr;
    bool lists_ready[2] = {false, false};            // set k holds the lists of the masks in buffer set k
    // Worker-sharded step: the streaming kernel runs on a side stream of its own and is joined only in
    // cser_wshard_apply, so that the caller's all-reduce, enqueued on its stream right behind the pack
    // kernel, overlaps the streaming of the unselected blocks.
    cudaStream_t ws_side = nullptr;
    cudaEvent_t ev_side = nullptr;
    bool side_pending = false;
    bool wshard_open = false;                        // pack done, apply pending
    bool wshard_reset = false;
    // exact-count GRBS (CSER_FLAG_EXACT_COUNT)
    bool exact = false;
    ExactScratch *exact_scratch = nullptr;
    uint32_t *exact_words = nullptr;                 // [2][B] the step's draws
    // The selected-block kernel and the streaming kernel touch disjoint columns; with an
    // auxiliary stream they run side by side (fork after the select kernel, join after both).
    cudaStream_t aux = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // The prefetched select kernel runs on aux behind the join, off the caller's stream; whoever next
    // touches the buffer sets waits for ev_pre first.
    cudaEvent_t ev_pre = nullptr;
    bool pre_pending = false;
    // Shared-memory staged selected-block kernel (CSER_FLAG_STAGED_SELECTED), 128-bit path only.
    // Its bounded waits report through err_host, one word of mapped pinned host memory that the host
    // looks at on every call without synchronizing.
    bool staging = false;
    bool fused_small = true;                         // small problems as one launch (off with CSER_FLAG_THREE_KERNELS)
    int sm_count = 0;
    unsigned *err_host = nullptr, *err_dev = nullptr;
    unsigned wait_mcycles = 2000;                    // about a second at 2 GHz
    bool test_stall = false;                         // cser_debug_stall_next_staged_step
    float *x0_stage = nullptr;                       // [d] staging for a host x0
    bool masks_injected = false;
    bool vec4 = false;                               // 128-bit path usable for the state arrays
    // timing
    bool timing = false;
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
    bool ev_valid = false;
    long long launches = 0;
    // host-gradient path
    float *g_stage = nullptr;
    cudaStream_t hs[2] = {nullptr, nullptr};
    cudaEvent_t h_ev[4] = {nullptr, nullptr, nullptr, nullptr};
};

namespace {

size_t state_elems(const cser_ctx *h) { return (size_t)h->n * (size_t)h->d; }

// k of exact-count GRBS: round(B / R), halves up; R = 0 keeps nothing.
uint32_t exact_k(long long B, uint32_t R) {
    if (R == 0) return 0;
    const long long k = (2 * B + R) / (2 * (long long)R);
    return (uint32_t)(k > B ? B : k);
}

// Where the reset mask of iteration t is kept (t a reset step).
uint8_t *reset_mask_of(const cser_ctx *h, uint64_t t) {
    if (h->n_buf != 2 || !h->mask_r_half[0]) return h->sb[0].mask_r;
    return h->mask_r_half[(t / (uint64_t)h->H) & 1u];
}

// Order stream s behind a select kernel that is still running ahead on the auxiliary stream.
int join_prefetch(cser_ctx *h, cudaStream_t s) {
    if (h->pre_pending) {
        CU_TRY(cudaStreamWaitEvent(s, h->ev_pre, 0));
        h->pre_pending = false;
    }
    return CSER_OK;
}

// Select kernel(s) of iteration `t` into buffer set `buf`, on stream s.  Counter k % 3 is
// used by the k-th launch, which also clears counter (k + 1) % 3; the counter of the launch
// before (still read by a step kernel that may be running) is left alone.
int launch_select(cser_ctx *h, int buf, uint64_t t, bool is_reset, bool draw, cudaStream_t s,
                  const uint32_t **count_out) {
    const unsigned grid = (unsigned)((h->B + 255) / 256);
    const uint32_t k0 = (uint32_t)(h->seed & 0xffffffffu), k1 = (uint32_t)(h->seed >> 32);
    const uint32_t t_lo = (uint32_t)(t & 0xffffffffu), t_hi = (uint32_t)(t >> 32);
    uint32_t *count = h->sel_count + h->kseq % 3, *count_next = h->sel_count + (h->kseq + 1) % 3;
    uint32_t R_g = h->R1, R_r = h->R2;
    int exact_g = 0, exact_r = 0;
    if (h->exact && draw) {
        // k = 0 and k = B need no threshold: they are "nothing" (R = 0) and "everything" (R = 1).
        const uint32_t kg = exact_k(h->B, h->R1), kr = exact_k(h->B, h->R2);
        if (kg == 0) R_g = 0; else if (kg >= h->B) R_g = 1; else exact_g = 1;
        if (is_reset) {
            if (kr == 0) R_r = 0; else if (kr >= h->B) R_r = 1; else exact_r = 1;
        }
        const int n_masks = (exact_g ? 1 : 0) + (exact_r ? 1 : 0);
        if (n_masks) {
            const uint32_t first = exact_g ? 0u : 1u;
            const unsigned g2 = (unsigned)((h->B * n_masks + 255) / 256);
            grbs_exact_hist_kernel<<<g2, 256, 0, s>>>(h->exact_scratch, h->exact_words, h->B, k0, k1, t_lo,
                                                      t_hi, kg, kr, n_masks, first);
            grbs_exact_threshold_kernel<<<g2, 256, 0, s>>>(h->exact_scratch, h->exact_words, h->B, n_masks,
                                                           first);
            h->launches += 2;
            CU_TRY(cudaGetLastError());
        }
    }
    grbs_select_kernel<<<grid, 256, 0, s>>>(h->sb[buf].mask_g, reset_mask_of(h, t), h->sb[buf].list, count,
                                            count_next, h->B, h->block_begin, k0, k1, t_lo, t_hi, R_g, R_r,
                                            is_reset ? 1 : 0, draw ? 1 : 0,
                                            h->exact_scratch ? h->exact_scratch->thr : nullptr, exact_g, exact_r);
    h->launches++;
    CU_TRY(cudaGetLastError());
    h->kseq++;
    *count_out = count;
    return CSER_OK;
}

// Make buffer set `buf` (with its list counter) the current step's.
void activate_selection(cser_ctx *h, int buf, const uint32_t *count, bool is_reset, uint64_t t) {
    h->cur = buf;
    h->mask_g = h->sb[buf].mask_g, h->sel_list = h->sb[buf].list;
    h->cur_count = count;
    if (is_reset) h->mask_r = h->last_mask_r = reset_mask_of(h, t);
}

// Masks and list for iteration h->t: take the prefetched ones if they are for this iteration,
// else run the select kernel now on stream s.
int select_for_iteration(cser_ctx *h, bool is_reset, cudaStream_t s) {
    if (int rc = join_prefetch(h, s)) return rc;
    if (h->pre_valid && h->pre_t == h->t && !h->masks_injected) {
        activate_selection(h, h->cur ^ 1, h->pre_count, is_reset, h->t);
        h->pre_valid = false;
        h->walk_all = false;
        return CSER_OK;
    }
    const int nb = h->n_buf == 2 ? (h->cur ^ 1) : 0;
    const uint32_t *count = nullptr;
    if (int rc = launch_select(h, nb, h->t, is_reset, !h->masks_injected, s, &count)) return rc;
    activate_selection(h, nb, count, is_reset, h->t);
    h->pre_valid = false;
    h->walk_all = h->masks_injected;
    h->masks_injected = false;
    return CSER_OK;
}

// Iterations that move at most this many bytes go through the single-launch kernel: below it the
// kernel boundaries, events and stream waits of the three-kernel step cost more than its better use
// of DRAM gains (about 10 us against 8 % of the traffic time; the two designs were measured to break
// even at 235 to 300 MB per step).
#ifndef CSER_FUSED_MAX_BYTES
#define CSER_FUSED_MAX_BYTES (1ll << 28)
#endif
constexpr long long kFusedMaxBytes = CSER_FUSED_MAX_BYTES;
long long step_bytes_bound(const cser_ctx *h) {
    return (long long)h->n * h->d * (12 + (h->m ? 8 : 0) + (h->e ? 8 : 0));
}
// The same kernel also wins on large problems when a large share of the blocks is selected: there the
// three-kernel step sends that share through the selected-block kernel as scattered pieces of one block
// per worker, while the single-launch kernel walks all columns in their natural order.  Measured on the
// WRN-40-8-sized vector (n = 8; ordinary / reset steps in ms, three kernels against one launch): R = 2
// 1.113 / 1.526 against 1.077 / 1.179; R = 4 1.165 / 1.449 against 1.164 / 1.196; R = 8 1.179 / 1.338
// against 1.206 / 1.219; R = 16 1.177 / 1.256 against 1.226 / 1.233; R = 32 1.178 / 1.226 against
// 1.237 / 1.242.  Hence, for up to 8 workers, one launch from a selected share of 1/4 on ordinary steps
// and of 1/10 on reset steps (update mask and reset mask together).  With 16 workers (ResNet-50-sized
// vector, block 1024) the walk over all columns pays later: ordinary steps only when everything is
// selected (R = 2: 1.554 against 1.566 ms, R = 4: 1.628 against 1.716), reset steps from a share of 1/5
// (R = 8: 1.832 against 1.806, R = 4: 1.941 against 1.771, R = 2: 2.015 against 1.732).  Beyond 16
// workers nothing was measured and the three kernels are kept.
struct FusedShare { double plain, reset; };
FusedShare fused_share_thresholds(int n) {
    if (n <= 8) return {0.25, 0.10};
    if (n <= 16) return {1.0, 0.20};
    return {2.0, 2.0};      // never
}
// Whether iteration number t of handle h goes through the single-launch kernel (given a gradient
// pointer that allows 128-bit loads).
bool fused_for_iteration(const cser_ctx *h, uint64_t t) {
    if (!(h->fused_small && h->vec4 && !h->exact && !h->replay && h->n_total == 0 && h->n_buf == 2)) return false;
    if (step_bytes_bound(h) <= kFusedMaxBytes) return true;
    if (h->d / 4 > 0xffffffffll) return false;
    const bool is_reset = (t % (uint64_t)h->H) == 0;
    const double share = (h->R1 ? 1.0 / h->R1 : 0.0) + (is_reset ? 1.0 / h->R2 : 0.0);
    const FusedShare th = fused_share_thresholds(h->n);
    return share >= (is_reset ? th.reset : th.plain);
}

// Work-unit geometry of the staged selected-block kernel: C vector columns per unit so that all n
// workers' segments of every array fit one stage, blocks cut into equal chunks, as many stages as fit
// the CTA's shared-memory budget.
struct StagedGeom {
    unsigned C = 0, n_chunks = 0, stages = 0;
    size_t smem = 0;
    bool ok = false;
};

StagedGeom staged_geometry(int n, unsigned bsv, bool mom, bool reset_err) {
    StagedGeom G;
    const unsigned long long per_col = (2ull + (mom ? 1 : 0) + (reset_err ? 1 : 0)) * (unsigned long long)n * 16ull;
    unsigned long long cmax = kStagedStageBudget / per_col;
    if (cmax > bsv) cmax = bsv;
    if (cmax > kStagedMaxChunkCols) cmax = kStagedMaxChunkCols;
    if (cmax < kStagedMinChunkCols) return G;          // too many workers or tiny blocks: register walk
    if (cmax < bsv) cmax = cmax / 8 * 8;
    unsigned chunks = (unsigned)((bsv + cmax - 1) / cmax);
    unsigned C = (bsv + chunks - 1) / chunks;
    if (chunks > 1) C = (C + 7) / 8 * 8;
    chunks = (bsv + C - 1) / C;
    const size_t stage = (size_t)per_col * C;
    size_t stages = (kStagedCtaBudget - kStagedCtlBytes) / stage;
    if (stages > (size_t)kStagedMaxStages) stages = kStagedMaxStages;
    if (stages < 2) return G;
    G.C = C, G.n_chunks = chunks, G.stages = (unsigned)stages;
    G.smem = kStagedCtlBytes + stages * stage;
    G.ok = true;
    return G;
}

template <bool MOM, bool RESET, bool ERR, bool DENSE>
cudaError_t launch_staged(int device, const StepParams &Q, unsigned grid, size_t smem, cudaStream_t st,
                          cudaLaunchAttribute *attr, int n_attr) {
    static bool configured[64] = {};
    auto kernel = cser_selected_staged_kernel<MOM, RESET, ERR, DENSE>;
    if (device < 0 || device >= 64 || !configured[device]) {
        cudaError_t er = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kStagedCtaBudget);
        if (er != cudaSuccess) return er;
#ifdef CSER_STAGED_CARVEOUT
        cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, CSER_STAGED_CARVEOUT);
#endif
        if (device >= 0 && device < 64) configured[device] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid), cfg.blockDim = dim3(kStagedThreads), cfg.dynamicSmemBytes = smem, cfg.stream = st;
    cfg.attrs = attr, cfg.numAttrs = n_attr;
    return cudaLaunchKernelEx(&cfg, kernel, Q);
}

template <int V>
int launch_step_v(cser_ctx *h, const StepParams &P, bool is_reset, cudaStream_t s, bool use_aux) {
    // (is_reset is a by-value copy: replay mode overrides it below)
    const long long cols = P.c_end - P.c_begin;
    if (cols <= 0) return CSER_OK;
    const long long tiles = (cols + kStepThreads - 1) / kStepThreads;
    if (tiles > 0x7fffffffll) return fail(CSER_ERR_INVALID, "d too large for one launch");
    // The streaming kernel's grid is tiles x workers; more CTAs than one grid holds are launched in
    // groups of whole rows.
    const int rows_per_launch = (int)((0x7fffffffll / tiles) < (long long)P.n ? (0x7fffffffll / tiles) : P.n);
    StepParams Q = P;
    Q.tiles = (unsigned)tiles;
    Q.rctl = h->replay ? h->ctl : nullptr;
    if (h->replay) Q.mask_g = h->sb[0].mask_g, Q.mask_r = h->sb[0].mask_r, Q.list = h->sb[0].list;
    if (h->replay) is_reset = true;   // the reset variants decide on the device whether this step resets
    // Grid of the selected-block kernel: the count lives on the device, so size the grid for
    // the expected number of selected columns in this launch's range plus slack; the kernel
    // strides over whatever the list really holds, so any grid size is correct.
    double frac = h->walk_all ? 1.0 : (h->R1 ? 1.0 / h->R1 : 0.0) + (is_reset ? 1.0 / h->R2 : 0.0);
    if (frac > 1.0) frac = 1.0;
    const double exp_blocks = frac * ((double)cols / P.bsv + 1.0);
    const double blocks = exp_blocks + 6.0 * sqrt(exp_blocks) + 4.0;
    long long wgrid = (long long)(blocks * P.bsv / kWalkThreads) + 1;
    const long long wmax = (cols + kWalkThreads - 1) / kWalkThreads + 1;
    if (wgrid > wmax) wgrid = wmax;
    const bool mom = h->m != nullptr;
    // R1 == 1 selects every block on every step: nothing is left to stream.
    const bool stream_any = h->walk_all || h->R1 != 1;
    const bool have_aux = use_aux && h->aux != nullptr && h->n_total == 0;
    const bool beside = have_aux && stream_any;                       // selected-block kernel beside the streaming one
    // next iteration's select kernel on aux (not where the single-launch kernel will run that iteration)
    const bool prefetch = have_aux && !h->replay && h->n_buf == 2 && !fused_for_iteration(h, h->t + 1);
    const bool fork = beside || prefetch;
    if (fork) {
        CU_TRY(cudaEventRecord(h->ev_fork, s));
        CU_TRY(cudaStreamWaitEvent(h->aux, h->ev_fork, 0));
    }
    cudaStream_t ws = beside ? h->aux : s;
    const bool err = h->e != nullptr;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeAccessPolicyWindow;
    attr[0].val.accessPolicyWindow.base_ptr = h->state_base;
    attr[0].val.accessPolicyWindow.num_bytes = h->state_bytes;
    attr[0].val.accessPolicyWindow.hitRatio = 1.0f;
    attr[0].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
    attr[0].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
    auto launch = [&](void (*kernel)(const StepParams), const StepParams &A, unsigned g, unsigned threads,
                      cudaStream_t st) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(g), cfg.blockDim = dim3(threads), cfg.dynamicSmemBytes = 0, cfg.stream = st;
        cfg.attrs = attr, cfg.numAttrs = h->l2_persist ? 1 : 0;
        return cudaLaunchKernelEx(&cfg, kernel, A);
    };
    // streaming kernel: one launch per group of whole rows (one group unless tiles x workers > 2^31 - 1)
    auto launch_stream = [&](void (*kernel)(const StepParams)) {
        cudaError_t er = cudaSuccess;
        for (int r0 = 0; r0 < P.n && er == cudaSuccess; r0 += rows_per_launch) {
            const int rows = P.n - r0 < rows_per_launch ? P.n - r0 : rows_per_launch;
            StepParams A = Q;
            const long long off = (long long)r0 * P.d;
            A.g += off, A.x += off;
            if (A.e) A.e += off;
            if (A.m) A.m += off;
            er = launch(kernel, A, (unsigned)(tiles * rows), kStepThreads, s);
            h->launches++;
        }
        return er;
    };
    if (h->n_total > 0) {
        // worker-sharded: the selected blocks go through pack / all-reduce / apply; only stream here
        cudaError_t er;
        if (mom) er = is_reset ? launch_stream(cser_stream_kernel<V, true, true, true>)
                               : launch_stream(cser_stream_kernel<V, true, false, true>);
        else     er = is_reset ? launch_stream(cser_stream_kernel<V, false, true, true>)
                               : launch_stream(cser_stream_kernel<V, false, false, true>);
        CU_TRY(er);
        CU_TRY(cudaGetLastError());
        return CSER_OK;
    }
    const bool dense = frac >= kDenseWalkFraction;
    if (dense) wgrid = wmax;
    // The staged kernel (128-bit path only): persistent CTAs, two per SM, over the work units.
    StagedGeom G;
    if (V == 4 && h->staging) G = staged_geometry(P.n, P.bsv, mom, is_reset && err);
    unsigned sgrid = 1;
    if (G.ok) {
        Q.chunk_cols = G.C, Q.n_chunks = G.n_chunks, Q.stages = G.stages, Q.err_word = h->err_dev;
        const double entries = dense ? (double)cols / P.bsv + 2.0 : blocks;
        const double units = entries * G.n_chunks;
        const double cap = (double)kStagedCtasPerSm * (h->sm_count > 0 ? h->sm_count : 148);
        sgrid = (unsigned)(units < cap ? (units < 1.0 ? 1.0 : units) : cap);
    }
    cudaError_t lerr = cudaSuccess;
#define CSER_LAUNCH_PAIR(MOM_, RESET_, ERR_)                                                            \
    do {                                                                                                \
        if (G.ok && dense)                                                                              \
            lerr = launch_staged<MOM_, RESET_, ERR_, true>(h->device, Q, sgrid, G.smem, ws, attr,       \
                                                           h->l2_persist ? 1 : 0);                      \
        else if (G.ok)                                                                                  \
            lerr = launch_staged<MOM_, RESET_, ERR_, false>(h->device, Q, sgrid, G.smem, ws, attr,      \
                                                            h->l2_persist ? 1 : 0);                     \
        else if (dense)                                                                                 \
            lerr = launch(cser_selected_kernel<V, MOM_, RESET_, ERR_, true>, Q, (unsigned)wgrid, kWalkThreads, ws); \
        else                                                                                            \
            lerr = launch(cser_selected_kernel<V, MOM_, RESET_, ERR_, false>, Q, (unsigned)wgrid, kWalkThreads, ws); \
        if (stream_any && lerr == cudaSuccess)                                                          \
            lerr = launch_stream(cser_stream_kernel<V, MOM_, RESET_, ERR_>);                            \
    } while (0)
#define CSER_LAUNCH_ERR(MOM_, RESET_)                                                                   \
    do {                                                                                                \
        if (err) CSER_LAUNCH_PAIR(MOM_, RESET_, true);                                                  \
        else     CSER_LAUNCH_PAIR(MOM_, RESET_, false);                                                 \
    } while (0)
    if (mom) {
        if (is_reset) CSER_LAUNCH_ERR(true, true);
        else          CSER_LAUNCH_ERR(true, false);
    } else {
        if (is_reset) CSER_LAUNCH_ERR(false, true);
        else          CSER_LAUNCH_ERR(false, false);
    }
#undef CSER_LAUNCH_ERR
#undef CSER_LAUNCH_PAIR
    h->launches += 1;
    CU_TRY(lerr);
    CU_TRY(cudaGetLastError());
    if (h->replay) {
        // the following iteration's masks and list, behind the selected-block kernel
        const unsigned sgrid = (unsigned)((h->B + 255) / 256);
        grbs_select_replay_kernel<<<sgrid, 256, 0, ws>>>(h->ctl, h->sb[0].mask_g, h->sb[0].mask_r, h->sb[0].list,
                                                         h->Bpad, h->B, h->block_begin,
                                                         (uint32_t)(h->seed & 0xffffffffu), (uint32_t)(h->seed >> 32),
                                                         h->R1, h->R2, (uint32_t)h->H);
        h->launches++;
        CU_TRY(cudaGetLastError());
    }
    if (beside) {
        // join: the caller's stream continues once the selected-block kernel is done ...
        CU_TRY(cudaEventRecord(h->ev_join, h->aux));
        CU_TRY(cudaStreamWaitEvent(s, h->ev_join, 0));
    }
    if (prefetch) {
        // ... while the next iteration's select kernel runs on the auxiliary stream, off the critical
        // path; the next call that touches the buffer sets waits for ev_pre
        const uint64_t t_next = h->t + 1;
        const int rc = launch_select(h, h->cur ^ 1, t_next, (t_next % (uint64_t)h->H) == 0, true, h->aux,
                                     &h->pre_count);
        h->pre_valid = rc == CSER_OK;
        h->pre_t = t_next;
        CU_TRY(cudaEventRecord(h->ev_pre, h->aux));
        h->pre_pending = true;
        return rc;
    }
    return CSER_OK;
}

// Launch the fused step kernel on element columns [col0, col1) of gradients `grad`.
int launch_step(cser_ctx *h, const float *grad, long long col0, long long col1, bool is_reset,
                cudaStream_t s, bool use_aux = false) {
    StepParams P;
    P.g = grad, P.x = h->x, P.e = h->e, P.m = h->m;
    P.mask_g = h->mask_g, P.mask_r = h->mask_r;
    P.list = h->sel_list, P.count = h->cur_count;
    P.tiles = 0, P.rctl = nullptr;
    P.list_cap = (unsigned)h->B;
    P.chunk_cols = P.n_chunks = P.stages = 0, P.err_word = nullptr;
    P.wait_mcycles = h->wait_mcycles, P.test_stall = h->test_stall ? 1u : 0u;
    P.mask_g_out = P.mask_r_out = nullptr, P.block_begin = h->block_begin;
    P.k0 = P.k1 = P.t_lo = P.t_hi = 0, P.R1 = h->R1, P.R2 = h->R2;
    P.d = h->d, P.n = h->n;
    P.eta = h->eta, P.beta = h->beta, P.n_f = (float)h->n;
    const bool v4 = h->vec4 && ((uintptr_t)grad % 16 == 0) && (col0 % 4 == 0) &&
                    (col1 % 4 == 0 || col1 == h->d);
    if (v4) {
        P.c_begin = col0 / 4, P.c_end = col1 / 4, P.bsv = (unsigned)(h->bs / 4);
        P.cols_total = h->d / 4;
        return launch_step_v<4>(h, P, is_reset, s, use_aux);
    }
    P.c_begin = col0, P.c_end = col1, P.bsv = (unsigned)h->bs;
    P.cols_total = h->d;
    return launch_step_v<1>(h, P, is_reset, s, use_aux);
}

bool fused_applies(const cser_ctx *h, const float *grad) {
    return !h->masks_injected && (uintptr_t)grad % 16 == 0 && fused_for_iteration(h, h->t);
}

// The whole iteration h->t in one launch (small problems): masks drawn inside the kernel and recorded
// in the current buffer set.
int launch_fused_small(cser_ctx *h, const float *grad, bool is_reset, cudaStream_t s, bool replay = false) {
    if (int rc = join_prefetch(h, s)) return rc;       // a select kernel of an earlier three-kernel step
    StepParams P = {};
    P.g = grad, P.x = h->x, P.e = h->e, P.m = h->m;
    P.d = h->d, P.n = h->n, P.cols_total = h->d / 4, P.c_begin = 0, P.c_end = h->d / 4;
    P.bsv = (unsigned)(h->bs / 4), P.list_cap = (unsigned)h->B;
    P.eta = h->eta, P.beta = h->beta, P.n_f = (float)h->n;
    P.block_begin = h->block_begin, P.R1 = h->R1, P.R2 = h->R2;
    P.k0 = (uint32_t)(h->seed & 0xffffffffu), P.k1 = (uint32_t)(h->seed >> 32);
    P.t_lo = (uint32_t)(h->t & 0xffffffffu), P.t_hi = (uint32_t)(h->t >> 32);
    P.mask_g_out = h->sb[h->cur].mask_g;
    P.mask_r_out = reset_mask_of(h, h->t);
    P.H = (uint32_t)h->H;
    if (replay) {
        // the kernel reads the iteration number from the device, decides there whether it resets, and
        // records the masks in buffer set 0 (where cser_read_state looks in replay mode)
        P.rctl = h->ctl;
        P.mask_g_out = h->sb[0].mask_g, P.mask_r_out = h->sb[0].mask_r;
        is_reset = true;
    }
    const unsigned grid = (unsigned)((P.cols_total + kFusedThreads - 1) / kFusedThreads);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeAccessPolicyWindow;
    attr[0].val.accessPolicyWindow.base_ptr = h->state_base;
    attr[0].val.accessPolicyWindow.num_bytes = h->state_bytes;
    attr[0].val.accessPolicyWindow.hitRatio = 1.0f;
    attr[0].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
    attr[0].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid), cfg.blockDim = dim3(kFusedThreads), cfg.dynamicSmemBytes = 0, cfg.stream = s;
    cfg.attrs = attr, cfg.numAttrs = h->l2_persist ? 1 : 0;
    const bool mom = h->m != nullptr, err = h->e != nullptr;
    void (*kernel)(const StepParams);
    if (mom) {
        if (err) kernel = is_reset ? cser_fused_small_kernel<true, true, true> : cser_fused_small_kernel<true, false, true>;
        else     kernel = is_reset ? cser_fused_small_kernel<true, true, false> : cser_fused_small_kernel<true, false, false>;
    } else {
        if (err) kernel = is_reset ? cser_fused_small_kernel<false, true, true> : cser_fused_small_kernel<false, false, true>;
        else     kernel = is_reset ? cser_fused_small_kernel<false, true, false> : cser_fused_small_kernel<false, false, false>;
    }
    // if the next iteration takes the three kernels, its select kernel runs beside this kernel
    const bool prefetch = !replay && h->aux != nullptr && !fused_for_iteration(h, h->t + 1);
    if (prefetch) {
        CU_TRY(cudaEventRecord(h->ev_fork, s));
        CU_TRY(cudaStreamWaitEvent(h->aux, h->ev_fork, 0));
    }
    CU_TRY(cudaLaunchKernelEx(&cfg, kernel, P));
    h->launches++;
    h->pre_valid = false;
    if (prefetch) {
        const uint64_t t_next = h->t + 1;
        const int rc = launch_select(h, h->cur ^ 1, t_next, (t_next % (uint64_t)h->H) == 0, true, h->aux,
                                     &h->pre_count);
        h->pre_valid = rc == CSER_OK;
        h->pre_t = t_next;
        CU_TRY(cudaEventRecord(h->ev_pre, h->aux));
        h->pre_pending = true;
    }
    if (replay) return CSER_OK;
    // what activate_selection does for the three-kernel step
    h->mask_g = h->sb[h->cur].mask_g, h->sel_list = h->sb[h->cur].list;
    if (is_reset) h->mask_r = h->last_mask_r = reset_mask_of(h, h->t);
    h->walk_all = false;
    return CSER_OK;
}

int check_handle(cser_ctx *h) {
    if (!h) return fail(CSER_ERR_INVALID, "NULL handle");
    int dev = -1;
    CU_TRY(cudaGetDevice(&dev));
    if (dev != h->device)
        return fail(CSER_ERR_INVALID, "handle belongs to device %d, current device is %d", h->device, dev);
    return CSER_OK;
}

int check_device_ptr(const void *p, const char *what) {
    if (!p) return fail(CSER_ERR_INVALID, "%s is NULL", what);
    cudaPointerAttributes a;
    cudaError_t er = cudaPointerGetAttributes(&a, p);
    if (er != cudaSuccess) {
        cudaGetLastError();
        return fail(CSER_ERR_INVALID, "%s: cannot query pointer (%s)", what, cudaGetErrorString(er));
    }
    if (a.type != cudaMemoryTypeDevice && a.type != cudaMemoryTypeManaged)
        return fail(CSER_ERR_INVALID, "%s must be device memory", what);
    if (a.type == cudaMemoryTypeDevice) {
        // memory of another GPU would be dereferenced by kernels of this one
        int dev = -1;
        if (cudaGetDevice(&dev) == cudaSuccess && a.device != dev)
            return fail(CSER_ERR_INVALID, "%s lives on device %d, the current device is %d", what, a.device, dev);
    }
    return CSER_OK;
}

// A bounded device-side wait that ran out (see staged_kernel.cuh) left its code in the handle's
// host-visible word: every later call reports it instead of stepping on an incomplete state.
int check_device_error(cser_ctx *h) {
    if (h->err_host) {
        const unsigned code = *reinterpret_cast<volatile unsigned *>(h->err_host);
        if (code)
            return fail(CSER_ERR_CUDA,
                        "a device-side wait ran out in an earlier step (code 0x%x): that step is incomplete, "
                        "restore the state from a checkpoint into a new handle", code);
    }
    return CSER_OK;
}

// An iteration whose launches could not all be enqueued did not happen: t goes back to where it was
// and the prepared masks are dropped, so that a retry draws them again.
int abandon_iteration(cser_ctx *h, uint64_t t_before, int rc) {
    h->t = t_before;
    h->pre_valid = false;
    return rc;
}

// advance t and decide whether this iteration resets (Algorithm 2 line 8)
bool begin_iteration(cser_ctx *h) {
    h->t += 1;
    return (h->t % (uint64_t)h->H) == 0;
}

}  // namespace

namespace {
// Handles with CSER_FLAG_L2_RESIDENT share one limit of the CUDA context (the L2 set-aside): it is raised by
// whoever needs more and put back, with the persisting lines released, only when the last such handle of
// the device is destroyed.
int g_l2_users[64] = {};
size_t g_l2_limit_before[64] = {};
}  // namespace

// ------------------------------------------------------------------ C ABI
extern "C" {

const char *cser_last_error(void) { return g_err; }

#ifndef CSER_BUILD_ID
#define CSER_BUILD_ID "unstamped"
#endif
const char *cser_build_id(void) { return CSER_BUILD_ID; }

cser_handle cser_create_ex(int64_t d, int32_t n_workers, int32_t block_size, uint32_t R1,
                           uint32_t R2, int32_t H, float eta, float beta, uint64_t seed,
                           int64_t block_begin, uint32_t flags) {
    g_err[0] = 0;
    if (d <= 0 || n_workers <= 0 || block_size <= 0 || R2 == 0 || H <= 0 || block_begin < 0) {
        fail(CSER_ERR_INVALID, "cser_create: d, n_workers, block_size, R2, H must be positive");
        return nullptr;
    }
    if (flags & ~(uint32_t)(CSER_FLAG_NO_ERROR_ARRAY | CSER_FLAG_EXACT_COUNT | CSER_FLAG_L2_RESIDENT |
                            CSER_FLAG_STAGED_SELECTED | CSER_FLAG_THREE_KERNELS)) {
        fail(CSER_ERR_INVALID, "cser_create: unknown flags 0x%x", flags);
        return nullptr;
    }
    if ((flags & CSER_FLAG_EXACT_COUNT) &&
        (block_begin != 0 || (d + block_size - 1) / block_size > (1ll << 22))) {
        fail(CSER_ERR_INVALID, "cser_create: exact-count GRBS needs block_begin = 0 and at most 2^22 blocks");
        return nullptr;
    }
    if (!isfinite(eta) || !(beta >= 0.f && beta < 1.f)) {
        fail(CSER_ERR_INVALID, "cser_create: eta must be finite and beta in [0, 1)");
        return nullptr;
    }
    const long long B = (d + block_size - 1) / block_size;
    if (block_begin + B > 0xffffffffll) {
        fail(CSER_ERR_INVALID, "cser_create: more than 2^32 blocks");
        return nullptr;
    }
    cser_ctx *h = new (std::nothrow) cser_ctx();
    if (!h) {
        fail(CSER_ERR_NOMEM, "cser_create: host allocation failed");
        return nullptr;
    }
    h->d = d, h->n = n_workers, h->bs = block_size, h->R1 = R1, h->R2 = R2, h->H = H;
    h->eta = eta, h->beta = beta, h->seed = seed, h->B = B, h->block_begin = block_begin;
    h->vec4 = (d % 4 == 0) && (block_size % 4 == 0);
    const size_t bytes = state_elems(h) * sizeof(float);
    cudaError_t er = cudaGetDevice(&h->device);
    // x, e, m in one allocation (each array starts on a 256-byte boundary)
    const bool with_e_ = !(flags & CSER_FLAG_NO_ERROR_ARRAY);
    const size_t arr_bytes = (bytes + 255) / 256 * 256;
    const int n_arrays = 1 + (with_e_ ? 1 : 0) + (beta != 0.f ? 1 : 0);
    h->state_bytes = arr_bytes * n_arrays;
    if (er == cudaSuccess) er = cudaMalloc(&h->state_base, h->state_bytes);
    if (er == cudaSuccess) {
        char *p = static_cast<char *>(h->state_base);
        h->x = reinterpret_cast<float *>(p), p += arr_bytes;
        if (with_e_) h->e = reinterpret_cast<float *>(p), p += arr_bytes;
        if (beta != 0.f) h->m = reinterpret_cast<float *>(p);
    }
    // the two buffer sets lie B entries apart in one allocation per kind
    const size_t Bpad = ((size_t)B + 15) / 16 * 16;
    h->Bpad = (long long)Bpad;
    if (er == cudaSuccess) er = cudaMalloc(&h->sb[0].mask_g, 2 * Bpad);
    if (er == cudaSuccess) er = cudaMalloc(&h->sb[0].mask_r, 2 * Bpad);
    if (er == cudaSuccess) er = cudaMalloc(&h->sb[0].list, 2 * Bpad * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaMemset(h->sb[0].mask_g, 0, 2 * Bpad);
    if (er == cudaSuccess) er = cudaMemset(h->sb[0].mask_r, 0, 2 * Bpad);
    if (er == cudaSuccess) {
        h->sb[1].mask_g = h->sb[0].mask_g + Bpad, h->sb[1].mask_r = h->sb[0].mask_r + Bpad;
        h->sb[1].list = h->sb[0].list + Bpad;
        h->mask_r_half[0] = h->sb[0].mask_r, h->mask_r_half[1] = h->sb[1].mask_r;
    }
    if (er == cudaSuccess) er = cudaMemset(h->state_base, 0, h->state_bytes);
    if (er == cudaSuccess && (flags & CSER_FLAG_L2_RESIDENT)) {
        // Keep a small state resident in L2 (set-aside persisting lines); larger ones stream.
        int max_persist = 0, max_window = 0;
        cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, h->device);
        cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, h->device);
        if (h->state_bytes <= (size_t)max_persist && h->state_bytes <= (size_t)max_window) {
            size_t cur_limit = 0;
            if (cudaDeviceGetLimit(&cur_limit, cudaLimitPersistingL2CacheSize) == cudaSuccess) {
                const bool slot = h->device >= 0 && h->device < 64;
                const bool first = !slot || g_l2_users[h->device] == 0;
                h->l2_limit_before = first ? cur_limit : (slot ? g_l2_limit_before[h->device] : cur_limit);
                const size_t want = cur_limit > h->state_bytes ? cur_limit : h->state_bytes;
                h->l2_persist = cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) == cudaSuccess;
                if (h->l2_persist && slot) {
                    if (first) g_l2_limit_before[h->device] = cur_limit;
                    g_l2_users[h->device]++;
                }
            }
            cudaGetLastError();
        }
    }
    if (er == cudaSuccess) er = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    if (er == cudaSuccess && (flags & CSER_FLAG_STAGED_SELECTED)) {
        er = cudaHostAlloc(reinterpret_cast<void **>(&h->err_host), 64, cudaHostAllocMapped | cudaHostAllocPortable);
        if (er == cudaSuccess) {
            *h->err_host = 0;
            er = cudaHostGetDevicePointer(reinterpret_cast<void **>(&h->err_dev), h->err_host, 0);
        }
        h->staging = er == cudaSuccess;
    }
    h->fused_small = !(flags & (CSER_FLAG_THREE_KERNELS | CSER_FLAG_STAGED_SELECTED));
    h->exact = (flags & CSER_FLAG_EXACT_COUNT) != 0;
    if (er == cudaSuccess && h->exact) er = cudaMalloc(&h->exact_scratch, sizeof(ExactScratch));
    if (er == cudaSuccess && h->exact) er = cudaMemset(h->exact_scratch, 0, sizeof(ExactScratch));
    if (er == cudaSuccess && h->exact) er = cudaMalloc(&h->exact_words, 2 * (size_t)B * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaMalloc(&h->ctl, sizeof(ReplayCtl));
    if (er == cudaSuccess) er = cudaMemset(h->ctl, 0, sizeof(ReplayCtl));
    if (er == cudaSuccess) er = cudaMalloc(&h->sel_count, 3 * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaMemset(h->sel_count, 0, 3 * sizeof(uint32_t));
    if (er == cudaSuccess) activate_selection(h, 0, h->sel_count, true, 0);
    for (int k = 0; k < 3 && er == cudaSuccess; ++k) er = cudaEventCreate(&h->ev[k]);
    if (er == cudaSuccess) {
        int lo = 0, hi = 0;   // hi = numerically lowest = highest priority
        er = cudaDeviceGetStreamPriorityRange(&lo, &hi);
        if (er == cudaSuccess) er = cudaStreamCreateWithPriority(&h->aux, cudaStreamNonBlocking, hi);
    }
    if (er == cudaSuccess) er = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
    if (er == cudaSuccess) er = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
    if (er == cudaSuccess) er = cudaEventCreateWithFlags(&h->ev_pre, cudaEventDisableTiming);
    if (er == cudaSuccess) er = cudaDeviceSynchronize();
    if (er != cudaSuccess) {
        fail(er == cudaErrorMemoryAllocation ? CSER_ERR_NOMEM : CSER_ERR_CUDA, "cser_create: %s",
             cudaGetErrorString(er));
        cudaGetLastError();
        cser_destroy(h);
        return nullptr;
    }
    return h;
}

cser_handle cser_create_slab(int64_t d, int32_t n_workers, int32_t block_size, uint32_t R1,
                             uint32_t R2, int32_t H, float eta, float beta, uint64_t seed,
                             int64_t block_begin) {
    return cser_create_ex(d, n_workers, block_size, R1, R2, H, eta, beta, seed, block_begin, 0);
}

cser_handle cser_create(int64_t d, int32_t n_workers, int32_t block_size, uint32_t R1, uint32_t R2,
                        int32_t H, float eta, float beta, uint64_t seed) {
    return cser_create_ex(d, n_workers, block_size, R1, R2, H, eta, beta, seed, 0, 0);
}

void cser_destroy(cser_handle h) {
    if (!h) return;
    if (h->aux) cudaStreamSynchronize(h->aux);   // a select kernel may still be running ahead
    if (h->ws_side) cudaStreamSynchronize(h->ws_side), cudaStreamDestroy(h->ws_side);
    if (h->ev_side) cudaEventDestroy(h->ev_side);
    if (h->l2_persist) {
        const bool slot = h->device >= 0 && h->device < 64;
        if (!slot || --g_l2_users[h->device] == 0) {      // the last L2-resident handle of this device
            cudaCtxResetPersistingL2Cache();
            cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, h->l2_limit_before);
            cudaGetLastError();
        }
    }
    cudaFree(h->state_base);
    cudaFree(h->sb[0].mask_g), cudaFree(h->sb[0].mask_r), cudaFree(h->sb[0].list);
    cudaFree(h->x0_stage), cudaFree(h->g_stage);
    if (h->err_host) cudaFreeHost(h->err_host);
    cudaFree(h->sel_count), cudaFree(h->exact_scratch), cudaFree(h->exact_words), cudaFree(h->ctl);
    cudaFree(h->pos_g), cudaFree(h->pos_r), cudaFree(h->olist_g), cudaFree(h->olist_r);
    for (auto &ev : h->ev) if (ev) cudaEventDestroy(ev);
    for (auto &ev : h->h_ev) if (ev) cudaEventDestroy(ev);
    for (auto &s : h->hs) if (s) cudaStreamDestroy(s);
    if (h->aux) cudaStreamDestroy(h->aux);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->ev_pre) cudaEventDestroy(h->ev_pre);
    delete h;
}

int cser_set_x0(cser_handle h, const float *x0, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (!x0) return fail(CSER_ERR_INVALID, "cser_set_x0: x0 is NULL");
    if (h->replay) return fail(CSER_ERR_INVALID, "cser_set_x0: call cser_replay_end first");
    cudaStream_t s = (cudaStream_t)stream;
    cudaPointerAttributes a;
    cudaError_t er = cudaPointerGetAttributes(&a, x0);
    if (er != cudaSuccess) cudaGetLastError();
    const float *src = x0;
    if (er != cudaSuccess || (a.type != cudaMemoryTypeDevice && a.type != cudaMemoryTypeManaged)) {
        if (!h->x0_stage) CU_TRY(cudaMalloc(&h->x0_stage, (size_t)h->d * sizeof(float)));
        CU_TRY(cudaMemcpyAsync(h->x0_stage, x0, (size_t)h->d * sizeof(float), cudaMemcpyHostToDevice, s));
        src = h->x0_stage;
    }
    const unsigned grid = (unsigned)((h->d + 255) / 256);
    broadcast_x0_kernel<<<grid, 256, 0, s>>>(src, h->x, h->e, h->m, h->d, h->n);
    h->launches++;
    CU_TRY(cudaGetLastError());
    h->t = 0;
    h->masks_injected = false;
    h->pre_valid = false;
    return CSER_OK;
}

int cser_step(cser_handle h, const float *grad, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (int rc = check_device_error(h)) return rc;
    if (int rc = check_device_ptr(grad, "cser_step: grad")) return rc;   // every call: an address can be reused
    if ((uintptr_t)grad % 4 != 0) return fail(CSER_ERR_INVALID, "cser_step: grad is not 4-byte aligned");
    if (h->n_total > 0) return fail(CSER_ERR_INVALID, "cser_step: worker-sharded handle; use cser_wshard_pack/apply");
    if (h->replay) return fail(CSER_ERR_INVALID, "cser_step: between cser_replay_begin and cser_replay_end use cser_step_replayable");
    cudaStream_t s = (cudaStream_t)stream;
    const uint64_t t_before = h->t;
    const bool is_reset = begin_iteration(h);
    int rc = CSER_OK;
    const bool fused = fused_applies(h, grad);
    if (h->timing && cudaEventRecord(h->ev[0], s) != cudaSuccess) rc = fail(CSER_ERR_CUDA, "cser_step: event record failed");
    if (!rc && !fused) rc = select_for_iteration(h, is_reset, s);
    if (!rc && h->timing && cudaEventRecord(h->ev[1], s) != cudaSuccess) rc = fail(CSER_ERR_CUDA, "cser_step: event record failed");
    if (!rc) rc = fused ? launch_fused_small(h, grad, is_reset, s) : launch_step(h, grad, 0, h->d, is_reset, s, true);
    h->test_stall = false;
    if (rc) return abandon_iteration(h, t_before, rc);
    if (h->timing) {
        CU_TRY(cudaEventRecord(h->ev[2], s));
        h->ev_valid = true;
    }
    return CSER_OK;
}

int cser_step_host(cser_handle h, const float *grad_host, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (int rc = check_device_error(h)) return rc;
    if (!grad_host) return fail(CSER_ERR_INVALID, "cser_step_host: grad_host is NULL");
    if (h->n_total > 0) return fail(CSER_ERR_INVALID, "cser_step_host: worker-sharded handle");
    if (h->replay) return fail(CSER_ERR_INVALID, "cser_step_host: call cser_replay_end first");
    cudaStream_t s = (cudaStream_t)stream;
    if (!h->g_stage) {
        CU_TRY(cudaMalloc(&h->g_stage, state_elems(h) * sizeof(float)));
        for (auto &st_ : h->hs) CU_TRY(cudaStreamCreateWithFlags(&st_, cudaStreamNonBlocking));
        for (auto &ev : h->h_ev) CU_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    }
    const uint64_t t_before = h->t;
    const bool is_reset = begin_iteration(h);
    // masks first, on the caller's stream; both internal streams start after them
    if (int rc = select_for_iteration(h, is_reset, s)) return abandon_iteration(h, t_before, rc);
    CU_TRY(cudaEventRecord(h->h_ev[0], s));
    CU_TRY(cudaStreamWaitEvent(h->hs[0], h->h_ev[0], 0));
    CU_TRY(cudaStreamWaitEvent(h->hs[1], h->h_ev[0], 0));
    // column slabs of about 64 MB of gradients each, boundaries on multiples of 1024 columns
    const long long d = h->d;
    long long n_slabs = (long long)((state_elems(h) * sizeof(float) + (64u << 20) - 1) / (64u << 20));
    if (n_slabs < 1) n_slabs = 1;
    if (n_slabs > 256) n_slabs = 256;
    long long slab = ((d + n_slabs - 1) / n_slabs + 1023) / 1024 * 1024;
    int k = 0;
    for (long long c0 = 0; c0 < d; c0 += slab, ++k) {
        const long long c1 = (c0 + slab < d) ? c0 + slab : d;
        cudaStream_t cs = h->hs[k & 1];
        CU_TRY(cudaMemcpy2DAsync(h->g_stage + c0, (size_t)d * sizeof(float), grad_host + c0,
                                 (size_t)d * sizeof(float), (size_t)(c1 - c0) * sizeof(float),
                                 (size_t)h->n, cudaMemcpyHostToDevice, cs));
        if (int rc = launch_step(h, h->g_stage, c0, c1, is_reset, cs)) return abandon_iteration(h, t_before, rc);
    }
    CU_TRY(cudaEventRecord(h->h_ev[1], h->hs[0]));
    CU_TRY(cudaEventRecord(h->h_ev[2], h->hs[1]));
    CU_TRY(cudaStreamWaitEvent(s, h->h_ev[1], 0));
    CU_TRY(cudaStreamWaitEvent(s, h->h_ev[2], 0));
    return CSER_OK;
}

static int state_piece(cser_ctx *h, int which, void **ptr, size_t *bytes) {
    switch (which) {
        case CSER_STATE_X: *ptr = h->x, *bytes = state_elems(h) * sizeof(float); return CSER_OK;
        case CSER_STATE_E:
            if (!h->e) return fail(CSER_ERR_INVALID, "no error array (CSER_FLAG_NO_ERROR_ARRAY)");
            *ptr = h->e, *bytes = state_elems(h) * sizeof(float);
            return CSER_OK;
        case CSER_STATE_M:
            if (!h->m) return fail(CSER_ERR_INVALID, "no momentum state (beta == 0)");
            *ptr = h->m, *bytes = state_elems(h) * sizeof(float);
            return CSER_OK;
        case CSER_STATE_MASK_G: *ptr = h->mask_g, *bytes = (size_t)h->B; return CSER_OK;
        case CSER_STATE_MASK_R: *ptr = h->last_mask_r, *bytes = (size_t)h->B; return CSER_OK;
        case CSER_STATE_T: *ptr = nullptr, *bytes = sizeof(uint64_t); return CSER_OK;
        default: return fail(CSER_ERR_INVALID, "unknown state id %d", which);
    }
}

int cser_read_state(cser_handle h, int which, void *dst, size_t dst_bytes, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (int rc = check_device_error(h)) return rc;
    if (!dst) return fail(CSER_ERR_INVALID, "cser_read_state: dst is NULL");
    void *src;
    size_t bytes;
    if (int rc = state_piece(h, which, &src, &bytes)) return rc;
    if (dst_bytes < bytes)
        return fail(CSER_ERR_TOO_SMALL, "cser_read_state: need %zu bytes, got %zu", bytes, dst_bytes);
    if (h->side_pending) {      // worker-sharded step packed but not applied: its streaming kernel may still run
        CU_TRY(cudaStreamWaitEvent((cudaStream_t)stream, h->ev_side, 0));
        h->side_pending = false;
    }
    if (h->replay && (which == CSER_STATE_MASK_G || which == CSER_STATE_MASK_R))
        src = which == CSER_STATE_MASK_G ? h->sb[0].mask_g : h->sb[0].mask_r;   // set 0 is the current one
    if (which == CSER_STATE_T) {
        if (h->replay) {   // the counter lives on the device while steps are replayable
            CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
            ReplayCtl c = {};
            CU_TRY(cudaMemcpy(&c, h->ctl, sizeof(c), cudaMemcpyDeviceToHost));
            CU_TRY(cudaMemcpy(dst, &c.c[0].t, sizeof(uint64_t), cudaMemcpyDefault));
            return CSER_OK;
        }
        CU_TRY(cudaMemcpy(dst, &h->t, sizeof(uint64_t), cudaMemcpyDefault));
        return CSER_OK;
    }
    CU_TRY(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, (cudaStream_t)stream));
    return CSER_OK;
}

int cser_read_columns(cser_handle h, int which, int64_t col_begin, int64_t col_count, float *dst,
                      size_t dst_elems, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (!dst) return fail(CSER_ERR_INVALID, "cser_read_columns: dst is NULL");
    if (which != CSER_STATE_X && which != CSER_STATE_E && which != CSER_STATE_M)
        return fail(CSER_ERR_INVALID, "cser_read_columns: which must be x, e or m");
    if (col_begin < 0 || col_count < 0 || col_begin + col_count > h->d)
        return fail(CSER_ERR_INVALID, "cser_read_columns: column range outside [0, d)");
    void *src;
    size_t bytes;
    if (int rc = state_piece(h, which, &src, &bytes)) return rc;
    if (dst_elems < (size_t)h->n * (size_t)col_count)
        return fail(CSER_ERR_TOO_SMALL, "cser_read_columns: need %zu elements", (size_t)h->n * (size_t)col_count);
    if (col_count == 0) return CSER_OK;
    CU_TRY(cudaMemcpy2DAsync(dst, (size_t)col_count * sizeof(float), static_cast<float *>(src) + col_begin,
                             (size_t)h->d * sizeof(float), (size_t)col_count * sizeof(float), (size_t)h->n,
                             cudaMemcpyDefault, (cudaStream_t)stream));
    return CSER_OK;
}

int cser_set_lr(cser_handle h, float eta) {
    if (int rc = check_handle(h)) return rc;
    if (!isfinite(eta)) return fail(CSER_ERR_INVALID, "cser_set_lr: eta must be finite");
    h->eta = eta;
    return CSER_OK;
}

int cser_write_state(cser_handle h, int which, const void *src, size_t bytes, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (!src) return fail(CSER_ERR_INVALID, "cser_write_state: src is NULL");
    if (h->replay) return fail(CSER_ERR_INVALID, "cser_write_state: call cser_replay_end first");
    if (which == CSER_STATE_MASK_G || which == CSER_STATE_MASK_R)
        return fail(CSER_ERR_INVALID, "masks cannot be written; use cser_debug_set_masks");
    void *dst;
    size_t want;
    if (int rc = state_piece(h, which, &dst, &want)) return rc;
    if (bytes != want)
        return fail(CSER_ERR_TOO_SMALL, "cser_write_state: need exactly %zu bytes, got %zu", want, bytes);
    if (which == CSER_STATE_T) {
        CU_TRY(cudaMemcpy(&h->t, src, sizeof(uint64_t), cudaMemcpyDefault));
        h->pre_valid = false;
        return CSER_OK;
    }
    CU_TRY(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, (cudaStream_t)stream));
    return CSER_OK;
}

int cser_debug_set_masks(cser_handle h, const uint8_t *g_mask, const uint8_t *r_mask, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (!g_mask) return fail(CSER_ERR_INVALID, "cser_debug_set_masks: g_mask is NULL");
    if (h->replay) return fail(CSER_ERR_INVALID, "cser_debug_set_masks: call cser_replay_end first");
    const bool next_is_reset = ((h->t + 1) % (uint64_t)h->H) == 0;
    if (next_is_reset && !r_mask)
        return fail(CSER_ERR_INVALID, "cser_debug_set_masks: next step resets, r_mask is NULL");
    cudaStream_t s = (cudaStream_t)stream;
    if (int rc = join_prefetch(h, s)) return rc;
    const int nb = h->n_buf == 2 ? (h->cur ^ 1) : 0;   // the set the next step's select kernel reads
    CU_TRY(cudaMemcpyAsync(h->sb[nb].mask_g, g_mask, (size_t)h->B, cudaMemcpyDefault, s));
    if (r_mask && next_is_reset)
        CU_TRY(cudaMemcpyAsync(reset_mask_of(h, h->t + 1), r_mask, (size_t)h->B, cudaMemcpyDefault, s));
    h->masks_injected = true;
    return CSER_OK;
}

int cser_grbs_mask(uint64_t seed, uint64_t t, uint32_t which, int64_t block_begin, int64_t n_blocks,
                   uint32_t R, uint8_t *mask_out, void *stream) {
    if (n_blocks < 0 || block_begin < 0 || R == 0 || which > 1 || block_begin + n_blocks > 0xffffffffll)
        return fail(CSER_ERR_INVALID, "cser_grbs_mask: bad arguments");
    if (n_blocks == 0) return CSER_OK;
    if (int rc = check_device_ptr(mask_out, "cser_grbs_mask: mask_out")) return rc;
    const unsigned grid = (unsigned)((n_blocks + 255) / 256);
    grbs_mask_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(
        mask_out, mask_out, n_blocks, block_begin, (uint32_t)(seed & 0xffffffffu),
        (uint32_t)(seed >> 32), (uint32_t)(t & 0xffffffffu), (uint32_t)(t >> 32), R, R, 1, which);
    CU_TRY(cudaGetLastError());
    return CSER_OK;
}

cser_handle cser_create_wshard(int64_t d, int32_t n_local, int32_t n_total, int32_t block_size, uint32_t R1,
                               uint32_t R2, int32_t H, float eta, float beta, uint64_t seed) {
    if (n_local <= 0 || n_total < n_local) {
        fail(CSER_ERR_INVALID, "cser_create_wshard: need 0 < n_local <= n_total");
        return nullptr;
    }
    cser_ctx *h = cser_create_ex(d, n_local, block_size, R1, R2, H, eta, beta, seed, 0, CSER_FLAG_EXACT_COUNT);
    if (!h) return nullptr;
    h->n_total = n_total;
    cudaError_t er = cudaMalloc(&h->pos_g, 2 * (size_t)h->B * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaMalloc(&h->pos_r, 2 * (size_t)h->B * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaMalloc(&h->olist_g, 2 * (size_t)h->B * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaMalloc(&h->olist_r, 2 * (size_t)h->B * sizeof(uint32_t));
    if (er == cudaSuccess) er = cudaStreamCreateWithFlags(&h->ws_side, cudaStreamNonBlocking);
    if (er == cudaSuccess) er = cudaEventCreateWithFlags(&h->ev_side, cudaEventDisableTiming);
    if (er != cudaSuccess) {
        fail(er == cudaErrorMemoryAllocation ? CSER_ERR_NOMEM : CSER_ERR_CUDA, "cser_create_wshard: %s",
             cudaGetErrorString(er));
        cudaGetLastError();
        cser_destroy(h);
        return nullptr;
    }
    return h;
}

int64_t cser_wshard_message_elems(cser_handle h, int reset_step) {
    if (!h || h->n_total <= 0) return -1;
    const int64_t kg = exact_k(h->B, h->R1), kr = reset_step ? exact_k(h->B, h->R2) : 0;
    return (kg + kr) * (int64_t)h->bs;
}

}  // extern "C"

namespace {
template <int V>
int launch_wshard(cser_ctx *h, ShardParams P, bool is_reset, bool pack, cudaStream_t s) {
    const unsigned long long total = (unsigned long long)(P.k_g + (is_reset ? P.k_r : 0u)) * P.bsv;
    if (total == 0) return CSER_OK;
    const unsigned grid = (unsigned)((total + kWalkThreads - 1) / kWalkThreads);
    const bool mom = h->m != nullptr;
    if (pack) {
        if (mom) {
            if (is_reset) wshard_pack_kernel<V, true, true><<<grid, kWalkThreads, 0, s>>>(P);
            else          wshard_pack_kernel<V, true, false><<<grid, kWalkThreads, 0, s>>>(P);
        } else {
            if (is_reset) wshard_pack_kernel<V, false, true><<<grid, kWalkThreads, 0, s>>>(P);
            else          wshard_pack_kernel<V, false, false><<<grid, kWalkThreads, 0, s>>>(P);
        }
    } else {
        if (is_reset) wshard_apply_kernel<V, true><<<grid, kWalkThreads, 0, s>>>(P);
        else          wshard_apply_kernel<V, false><<<grid, kWalkThreads, 0, s>>>(P);
    }
    h->launches++;
    CU_TRY(cudaGetLastError());
    return CSER_OK;
}

// Ordered lists of the masks in buffer set `buf` (those of iteration t), on stream s.
int launch_ordered_lists(cser_ctx *h, int buf, bool is_reset, uint64_t t, cudaStream_t s) {
    const size_t set = (size_t)buf * (size_t)h->B;
    const unsigned grid = (unsigned)((h->B + kScanThreads - 1) / kScanThreads);
    ordered_lists_kernel<<<grid, kScanThreads, 0, s>>>(h->sb[buf].mask_g, is_reset ? reset_mask_of(h, t) : nullptr, h->B,
                                                       h->pos_g + set, h->pos_r + set, h->olist_g + set,
                                                       h->olist_r + set);
    h->launches++;
    CU_TRY(cudaGetLastError());
    return CSER_OK;
}

int wshard_params(cser_ctx *h, const float *grad, float *msg, bool *v4, ShardParams *P) {
    P->g = grad, P->x = h->x, P->e = h->e, P->m = h->m, P->msg = msg;
    P->mask_g = h->mask_g, P->mask_r = h->mask_r;
    const size_t set = (size_t)h->cur * (size_t)h->B;          // the lists of the current mask buffer set
    P->pos_g = h->pos_g + set, P->olist_g = h->olist_g + set, P->olist_r = h->olist_r + set;
    P->d = h->d, P->n = h->n;
    P->k_g = exact_k(h->B, h->R1), P->k_r = exact_k(h->B, h->R2);
    P->eta = h->eta, P->beta = h->beta, P->n_total_f = (float)h->n_total;
    *v4 = h->vec4 && ((uintptr_t)msg % 16 == 0) && (!grad || (uintptr_t)grad % 16 == 0);
    P->bsv = *v4 ? (unsigned)(h->bs / 4) : (unsigned)h->bs;
    P->cols_total = *v4 ? h->d / 4 : h->d;
    return CSER_OK;
}
}  // namespace

extern "C" {

int cser_wshard_pack(cser_handle h, const float *grad, float *msg, size_t msg_elems, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (h->n_total <= 0) return fail(CSER_ERR_INVALID, "cser_wshard_pack: not a worker-sharded handle");
    if (h->wshard_open) return fail(CSER_ERR_INVALID, "cser_wshard_pack: previous step was not applied");
    if (int rc = check_device_ptr(grad, "cser_wshard_pack: grad")) return rc;
    if (int rc = check_device_ptr(msg, "cser_wshard_pack: msg")) return rc;
    if (((uintptr_t)grad | (uintptr_t)msg) % 4 != 0)
        return fail(CSER_ERR_INVALID, "cser_wshard_pack: pointers must be 4-byte aligned");
    const bool next_reset = ((h->t + 1) % (uint64_t)h->H) == 0;
    if ((int64_t)msg_elems < cser_wshard_message_elems(h, next_reset))
        return fail(CSER_ERR_TOO_SMALL, "cser_wshard_pack: message buffer too small");
    cudaStream_t s = (cudaStream_t)stream;
    const uint64_t t_before = h->t;
    const bool is_reset = begin_iteration(h);
    const bool prefetched = h->pre_valid && h->pre_t == h->t && !h->masks_injected;
    if (int rc = select_for_iteration(h, is_reset, s)) return abandon_iteration(h, t_before, rc);
    if (!(prefetched && h->lists_ready[h->cur])) {
        if (int rc = launch_ordered_lists(h, h->cur, is_reset, h->t, s)) return abandon_iteration(h, t_before, rc);
    }
    h->lists_ready[h->cur] = false;          // consumed by this step
    // Fork: the streaming kernel (unselected blocks) goes to the side stream, the next iteration's masks
    // and ordered lists to the auxiliary stream; the pack kernel (selected blocks, disjoint columns) stays
    // on the caller's stream, so the caller's all-reduce can start as soon as the message is complete.
    CU_TRY(cudaEventRecord(h->ev_fork, s));
    CU_TRY(cudaStreamWaitEvent(h->ws_side, h->ev_fork, 0));
    ShardParams P;
    bool v4;
    wshard_params(h, grad, msg, &v4, &P);
    // the pack kernel first: it is small and the message is what the other ranks wait for
    int rc = v4 ? launch_wshard<4>(h, P, is_reset, true, s) : launch_wshard<1>(h, P, is_reset, true, s);
    if (!rc) rc = launch_step(h, grad, 0, h->d, is_reset, h->ws_side, false);
    CU_TRY(cudaEventRecord(h->ev_side, h->ws_side));
    h->side_pending = true;
    if (rc) {
        CU_TRY(cudaStreamWaitEvent(s, h->ev_side, 0));
        h->side_pending = false;
        return abandon_iteration(h, t_before, rc);
    }
    if (h->aux != nullptr && h->n_buf == 2) {
        CU_TRY(cudaStreamWaitEvent(h->aux, h->ev_fork, 0));
        const uint64_t t_next = h->t + 1;
        const bool next_reset = (t_next % (uint64_t)h->H) == 0;
        const int nb = h->cur ^ 1;
        int prc = launch_select(h, nb, t_next, next_reset, true, h->aux, &h->pre_count);
        if (!prc) prc = launch_ordered_lists(h, nb, next_reset, t_next, h->aux);
        h->pre_valid = prc == CSER_OK;
        h->lists_ready[nb] = prc == CSER_OK;
        h->pre_t = t_next;
        CU_TRY(cudaEventRecord(h->ev_pre, h->aux));
        h->pre_pending = true;
    }
    h->wshard_open = true;
    h->wshard_reset = is_reset;
    return CSER_OK;
}

int cser_wshard_apply(cser_handle h, const float *msg, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (h->n_total <= 0) return fail(CSER_ERR_INVALID, "cser_wshard_apply: not a worker-sharded handle");
    if (!h->wshard_open) return fail(CSER_ERR_INVALID, "cser_wshard_apply: no packed step pending");
    if (int rc = check_device_ptr(msg, "cser_wshard_apply: msg")) return rc;
    if (h->side_pending) {      // the streaming kernel of this iteration
        CU_TRY(cudaStreamWaitEvent((cudaStream_t)stream, h->ev_side, 0));
        h->side_pending = false;
    }
    ShardParams P;
    bool v4;
    wshard_params(h, nullptr, const_cast<float *>(msg), &v4, &P);
    const int rc = v4 ? launch_wshard<4>(h, P, h->wshard_reset, false, (cudaStream_t)stream)
                      : launch_wshard<1>(h, P, h->wshard_reset, false, (cudaStream_t)stream);
    if (rc) return rc;
    h->wshard_open = false;
    return CSER_OK;
}

int cser_replay_begin(cser_handle h, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (h->replay) return fail(CSER_ERR_INVALID, "cser_replay_begin: already begun");
    if (h->exact || h->n_total > 0 || h->masks_injected)
        return fail(CSER_ERR_INVALID,
                    "cser_replay_begin: not available with exact-count masks, worker sharding or injected masks");
    cudaStream_t s = (cudaStream_t)stream;
    if (int rc = join_prefetch(h, s)) return rc;
    // In replay mode half 0 of the reset-mask allocation always holds the last executed reset step's
    // mask (the advance kernel copies a prepared mask over it only when its step resets).
    if (h->last_mask_r && h->last_mask_r != h->sb[0].mask_r) {
        CU_TRY(cudaMemcpyAsync(h->sb[0].mask_r, h->last_mask_r, (size_t)h->B, cudaMemcpyDeviceToDevice, s));
        h->last_mask_r = h->sb[0].mask_r;
    }
    ReplayCtl c = {};
    c.c[0].t = h->t;           // block 0 stands for the iteration already done
    CU_TRY(cudaMemcpyAsync(h->ctl, &c, sizeof(c), cudaMemcpyHostToDevice, s));
    CU_TRY(cudaStreamSynchronize(s));   // c is on this function's stack
    // Small problems replay as one launch per step (the kernel draws its masks itself); the choice is made
    // once, here, because the two replay protocols keep different things in the control block.
    h->replay_fused = h->fused_small && h->vec4 && step_bytes_bound(h) <= kFusedMaxBytes;
    if (!h->replay_fused) {
        // masks and list of iteration t + 1 into buffer set 1, published in block 1
        const unsigned grid = (unsigned)((h->B + 255) / 256);
        grbs_select_replay_kernel<<<grid, 256, 0, s>>>(h->ctl, h->sb[0].mask_g, h->sb[0].mask_r, h->sb[0].list,
                                                       h->Bpad, h->B, h->block_begin,
                                                       (uint32_t)(h->seed & 0xffffffffu), (uint32_t)(h->seed >> 32),
                                                       h->R1, h->R2, (uint32_t)h->H);
        h->launches++;
        CU_TRY(cudaGetLastError());
    }
    h->pre_valid = false;
    h->walk_all = false;
    h->replay = true;
    return CSER_OK;
}

int cser_step_replayable(cser_handle h, const float *grad, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (!h->replay) return fail(CSER_ERR_INVALID, "cser_step_replayable: call cser_replay_begin first");
    if (int rc = check_device_error(h)) return rc;
    if (int rc = check_device_ptr(grad, "cser_step_replayable: grad")) return rc;
    if ((uintptr_t)grad % 4 != 0) return fail(CSER_ERR_INVALID, "cser_step_replayable: grad is not 4-byte aligned");
    cudaStream_t s = (cudaStream_t)stream;
    if (h->replay_fused) {
        if ((uintptr_t)grad % 16 != 0)
            return fail(CSER_ERR_INVALID, "cser_step_replayable: this handle replays as one launch per step, "
                                          "which needs a 16-byte aligned grad");
        return launch_fused_small(h, grad, true, s, true);
    }
    // the iteration prepared during the last step becomes the current one
    replay_advance_kernel<<<(unsigned)((h->B + 255) / 256), 256, 0, s>>>(h->ctl, h->sb[0].mask_g, h->sb[0].mask_r,
                                                                         h->sb[0].list, h->Bpad, h->B);
    h->launches++;
    CU_TRY(cudaGetLastError());
    return launch_step(h, grad, 0, h->d, true, s, true);
}

int cser_replay_end(cser_handle h, void *stream) {
    if (int rc = check_handle(h)) return rc;
    if (!h->replay) return fail(CSER_ERR_INVALID, "cser_replay_end: not begun");
    CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    ReplayCtl c = {};
    CU_TRY(cudaMemcpy(&c, h->ctl, sizeof(c), cudaMemcpyDeviceToHost));
    h->t = c.c[0].t;
    h->replay = false;
    h->pre_valid = false;
    // Set 0 holds the masks of the last iteration, half 0 the last executed reset mask.  Ordinary steps
    // keep reset number q's mask in half q & 1: if the next reset step would write half 0, move the last
    // mask to half 1 first so that it stays readable until then.
    h->cur = 0;
    h->mask_g = h->sb[0].mask_g, h->sel_list = h->sb[0].list, h->cur_count = h->sel_count;
    h->mask_r = h->last_mask_r = h->sb[0].mask_r;
    const uint64_t next_reset = (h->t / (uint64_t)h->H + 1) * (uint64_t)h->H;
    if (reset_mask_of(h, next_reset) == h->sb[0].mask_r && h->mask_r_half[1]) {
        CU_TRY(cudaMemcpy(h->mask_r_half[1], h->sb[0].mask_r, (size_t)h->B, cudaMemcpyDeviceToDevice));
        h->mask_r = h->last_mask_r = h->mask_r_half[1];
    }
    return CSER_OK;
}

int cser_debug_stall_next_staged_step(cser_handle h, unsigned wait_mcycles) {
    if (int rc = check_handle(h)) return rc;
    if (!h->staging) return fail(CSER_ERR_INVALID, "cser_debug_stall_next_staged_step: handle has no staged kernel");
    if (wait_mcycles == 0 || wait_mcycles > 2000) return fail(CSER_ERR_INVALID, "wait_mcycles must be in 1 .. 2000");
    h->wait_mcycles = wait_mcycles;
    h->test_stall = true;
    return CSER_OK;
}

int cser_set_timing(cser_handle h, int on) {
    if (int rc = check_handle(h)) return rc;
    h->timing = on != 0;
    h->ev_valid = false;
    return CSER_OK;
}

int cser_last_kernel_ms(cser_handle h, float *mask_ms, float *step_ms) {
    if (int rc = check_handle(h)) return rc;
    if (!h->ev_valid) return fail(CSER_ERR_INVALID, "no timed step recorded");
    CU_TRY(cudaEventSynchronize(h->ev[2]));
    float a = 0.f, b = 0.f;
    CU_TRY(cudaEventElapsedTime(&a, h->ev[0], h->ev[1]));
    CU_TRY(cudaEventElapsedTime(&b, h->ev[1], h->ev[2]));
    if (mask_ms) *mask_ms = a;
    if (step_ms) *step_ms = b;
    return CSER_OK;
}

int64_t cser_launch_count(cser_handle h) { return h ? h->launches : 0; }

}  // extern "C"

// ------------------------------------------------------------------ allocation-free step
// A step's only scratch is what the select kernel hands to the step kernel: the two GRBS
// masks, the list of selected blocks and two list counters.  For callers that must not
// allocate, that scratch lives here: a fixed array that every GPU which loads this
// library keeps until the process exits.  Layout (bytes): update mask [0, MAXB), reset
// mask [MAXB, 2 MAXB), list of uint32 [2 MAXB, 6 MAXB), three uint32 counters after it.
// Static device memory starts zeroed, which is the state the counters need.
constexpr size_t kNoallocMaxB = CSER_NOALLOC_MAX_BLOCKS;
constexpr size_t kNoallocBytes = 6 * kNoallocMaxB + 256;
static __device__ __align__(256) uint8_t g_noalloc_scratch[kNoallocBytes];

namespace {

constexpr int kNoallocMaxDevices = 64;
// Device address of g_noalloc_scratch on each device, looked up once per device.  In host
// code the array's name is only a handle for the runtime, never an address a kernel may
// be given; cudaGetSymbolAddress translates it for the device that is current.
uint8_t *g_noalloc_addr[kNoallocMaxDevices] = {};
unsigned g_noalloc_kseq[kNoallocMaxDevices] = {};  // select launches so far: picks the list counter

int noalloc_scratch(int device, uint8_t **out) {
    if (device < 0 || device >= kNoallocMaxDevices)
        return fail(CSER_ERR_INVALID, "cser_step_noalloc: device %d out of range", device);
    uint8_t *p = __atomic_load_n(&g_noalloc_addr[device], __ATOMIC_ACQUIRE);
    if (!p) {
        void *sym = nullptr;
        cudaError_t er = cudaGetSymbolAddress(&sym, g_noalloc_scratch);
        if (er != cudaSuccess || !sym) {
            cudaGetLastError();
            return fail(CSER_ERR_CUDA, "cser_step_noalloc: cudaGetSymbolAddress: %s",
                        cudaGetErrorString(er));
        }
        p = static_cast<uint8_t *>(sym);
        __atomic_store_n(&g_noalloc_addr[device], p, __ATOMIC_RELEASE);
    }
    *out = p;
    return CSER_OK;
}

}  // namespace

extern "C" int cser_step_noalloc(int64_t d, int32_t n_workers, int32_t block_size, uint32_t R1,
                                 uint32_t R2, int32_t H, float eta, float beta, uint64_t seed,
                                 uint64_t t, const float *grad, float *x, float *e, float *m,
                                 void *stream) {
    if (d <= 0 || n_workers <= 0 || block_size <= 0 || R2 == 0 || H <= 0 || t == 0)
        return fail(CSER_ERR_INVALID,
                    "cser_step_noalloc: d, n_workers, block_size, R2, H, t must be positive");
    if (!isfinite(eta) || !(beta >= 0.f && beta < 1.f))
        return fail(CSER_ERR_INVALID, "cser_step_noalloc: eta must be finite and beta in [0, 1)");
    const long long B = (d + block_size - 1) / block_size;
    if (B > (long long)CSER_NOALLOC_MAX_BLOCKS)
        return fail(CSER_ERR_INVALID,
                    "cser_step_noalloc: %lld blocks exceed the built-in scratch of %d blocks; "
                    "use a larger block_size or the handle API", B, (int)CSER_NOALLOC_MAX_BLOCKS);
    if (int rc = check_device_ptr(grad, "cser_step_noalloc: grad")) return rc;
    if (int rc = check_device_ptr(x, "cser_step_noalloc: x")) return rc;
    if (int rc = check_device_ptr(e, "cser_step_noalloc: e")) return rc;
    if (beta != 0.f) {
        if (int rc = check_device_ptr(m, "cser_step_noalloc: m")) return rc;
    }
    if (((uintptr_t)grad | (uintptr_t)x | (uintptr_t)e | (uintptr_t)m) % 4 != 0)
        return fail(CSER_ERR_INVALID, "cser_step_noalloc: arrays must be 4-byte aligned");

    cser_ctx c;   // plain stack object describing the caller's arrays; owns nothing
    CU_TRY(cudaGetDevice(&c.device));
    uint8_t *scratch = nullptr;
    if (int rc = noalloc_scratch(c.device, &scratch)) return rc;
    c.d = d, c.n = n_workers, c.bs = block_size, c.R1 = R1, c.R2 = R2, c.H = H;
    c.eta = eta, c.beta = beta, c.seed = seed, c.B = B, c.block_begin = 0;
    c.t = t;
    c.x = x, c.e = e, c.m = (beta != 0.f) ? m : nullptr;
    c.n_buf = 1;
    c.sb[0].mask_g = scratch, c.sb[0].mask_r = scratch + kNoallocMaxB;
    c.sb[0].list = reinterpret_cast<uint32_t *>(scratch + 2 * kNoallocMaxB);
    c.sel_count = reinterpret_cast<uint32_t *>(scratch + 6 * kNoallocMaxB);
    c.kseq = g_noalloc_kseq[c.device];
    c.vec4 = (d % 4 == 0) && (block_size % 4 == 0) &&
             (((uintptr_t)x | (uintptr_t)e | (uintptr_t)c.m) % 16 == 0);
    const bool is_reset = (t % (uint64_t)H) == 0;
    cudaStream_t s = (cudaStream_t)stream;
    // The select kernel rewrites every mask entry and list entry the step kernel reads and
    // clears the counter the next call will use, so nothing an earlier call left in the
    // array is ever used and nothing has to be cleared between calls.
    const int rc = select_for_iteration(&c, is_reset, s);
    g_noalloc_kseq[c.device] = c.kseq;
    if (rc) return rc;
    return launch_step(&c, grad, 0, d, is_reset, s);
}
