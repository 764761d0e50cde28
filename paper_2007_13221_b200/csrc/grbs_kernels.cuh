// grbs_kernels.cuh - GRBS block selection (Definition 2): stand-alone mask kernel, exact-count threshold kernels, per-step select kernel
// Device code of the CSER step library; included by cser.cu inside its unnamed namespace.
#pragma once
#include "philox.cuh"

// GRBS block select (Definition 2).  Thread idx < B draws the update mask of block
// idx, thread B <= idx < 2B the reset mask of block idx - B (only on reset steps).
__global__ void __launch_bounds__(256)
grbs_mask_kernel(uint8_t *__restrict__ mask_g, uint8_t *__restrict__ mask_r, long long B,
                 long long block_begin, uint32_t k0, uint32_t k1, uint32_t t_lo, uint32_t t_hi,
                 uint32_t R_g, uint32_t R_r, int n_masks, uint32_t first_which) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * n_masks) return;
    const uint32_t second = idx >= B ? 1u : 0u;
    const long long b = idx - (second ? B : 0);
    const uint32_t which = first_which + second;
    const uint32_t R = which ? R_r : R_g;
    const uint32_t w0 =
        philox4x32_10_word0(k0, k1, (uint32_t)(block_begin + b), t_lo, t_hi, which);
    const uint8_t sel = (R != 0 && (unsigned long long)w0 * R < (1ull << 32)) ? 1 : 0;   // R = 0: C = 0
    (second ? mask_r : mask_g)[b] = sel;
}

// ------------------------------------------------------------------ exact-count GRBS
// Definition 2 read literally: exactly k = round(B / R) blocks, those with the k smallest
// keys (word0, block id).  The k-th smallest key is found in two passes over the B draws
// with no sorting: a 4096-bin histogram of the top 12 bits of word0 locates the bin that
// holds it, then the few keys of that bin (about B / 4096) are ranked against each other.
// Each pass ends in the last CTA to finish (a counter, no waiting), which does the small
// serial part and re-arms the scratch for the next step.
constexpr int kExactBins = 4096;
constexpr int kExactCap = 8192;          // candidate keys kept per mask
struct ExactScratch {
    uint32_t hist[2][kExactBins];
    uint32_t bin[2];                      // bin that holds the k-th smallest key
    uint32_t k_rem[2];                    // its rank inside that bin (1-based)
    uint32_t n_cand[2];
    uint32_t done[2];                     // CTAs finished, one counter per pass
    unsigned long long thr[2];            // the k-th smallest key
    unsigned long long cand[2][kExactCap];
};

__global__ void __launch_bounds__(256)
grbs_exact_hist_kernel(ExactScratch *__restrict__ X, uint32_t *__restrict__ words, long long B,
                       uint32_t k0, uint32_t k1, uint32_t t_lo, uint32_t t_hi, uint32_t kg, uint32_t kr,
                       int n_masks, uint32_t first_which) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < B * n_masks) {
        const uint32_t second = idx >= B ? 1u : 0u;
        const long long b = idx - (second ? B : 0);
        const uint32_t which = first_which + second;
        const uint32_t w = philox4x32_10_word0(k0, k1, (uint32_t)b, t_lo, t_hi, which);
        words[(size_t)which * B + b] = w;
        atomicAdd(&X->hist[which][w >> 20], 1u);
    }
    __shared__ bool last;
    __shared__ uint32_t part[256];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&X->done[0], 1u) == gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    for (int q = 0; q < n_masks; ++q) {
        const uint32_t which = first_which + q;
        const uint32_t k = which ? kr : kg;
        volatile uint32_t *h = X->hist[which];
        constexpr int per = kExactBins / 256;
        uint32_t loc[per], sum = 0;
#pragma unroll
        for (int j = 0; j < per; ++j) { loc[j] = h[threadIdx.x * per + j]; sum += loc[j]; }
        part[threadIdx.x] = sum;
        __syncthreads();
        uint32_t before = 0;                        // draws in bins below this thread's bins
        for (int j = 0; j < (int)threadIdx.x; ++j) before += part[j];
        if (k > before && k <= before + sum) {      // the k-th smallest lies in one of my bins
            uint32_t cum = before;
#pragma unroll
            for (int j = 0; j < per; ++j) {
                if (k > cum && k <= cum + loc[j]) {
                    X->bin[which] = threadIdx.x * per + j;
                    X->k_rem[which] = k - cum;
                }
                cum += loc[j];
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < per; ++j) h[threadIdx.x * per + j] = 0;   // re-arm for the next step
        if (threadIdx.x == 0) X->n_cand[which] = 0;
    }
    if (threadIdx.x == 0) X->done[0] = 0;
}

__global__ void __launch_bounds__(256)
grbs_exact_threshold_kernel(ExactScratch *__restrict__ X, const uint32_t *__restrict__ words, long long B,
                            int n_masks, uint32_t first_which) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < B * n_masks) {
        const uint32_t second = idx >= B ? 1u : 0u;
        const long long b = idx - (second ? B : 0);
        const uint32_t which = first_which + second;
        const uint32_t w = words[(size_t)which * B + b];
        if ((w >> 20) == X->bin[which]) {
            const uint32_t at = atomicAdd(&X->n_cand[which], 1u);
            if (at < (uint32_t)kExactCap) X->cand[which][at] = ((unsigned long long)w << 32) | (uint32_t)b;
        }
    }
    __shared__ bool last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&X->done[1], 1u) == gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    for (int q = 0; q < n_masks; ++q) {
        const uint32_t which = first_which + q;
        const uint32_t m = min(*(volatile uint32_t *)&X->n_cand[which], (uint32_t)kExactCap);
        const uint32_t want = X->k_rem[which] - 1;   // rank (0-based) of the threshold inside the bin
        const volatile unsigned long long *c = X->cand[which];
        for (uint32_t i = threadIdx.x; i < m; i += blockDim.x) {
            const unsigned long long ki = c[i];
            uint32_t rank = 0;
            for (uint32_t j = 0; j < m; ++j) rank += c[j] < ki ? 1u : 0u;
            if (rank == want) X->thr[which] = ki;   // keys are distinct: exactly one writer
        }
    }
    if (threadIdx.x == 0) X->done[1] = 0;
}

// Per-step block select: one thread per block.  With `draw` it draws the update mask (and,
// on a reset step, the reset mask) and stores the flags; without it the flags already in
// mask_g / mask_r are used (injected masks).  Blocks selected by either mask are appended
// to `list` (order irrelevant: blocks are independent) with one atomicAdd per warp on
// *count.  *count_next, the counter the following step will use, is cleared here, so no
// counter ever needs a separate memset.
__global__ void __launch_bounds__(256)
grbs_select_kernel(uint8_t *__restrict__ mask_g, uint8_t *__restrict__ mask_r,
                   uint32_t *__restrict__ list, uint32_t *count, uint32_t *count_next, long long B,
                   long long block_begin, uint32_t k0, uint32_t k1, uint32_t t_lo, uint32_t t_hi,
                   uint32_t R_g, uint32_t R_r, int is_reset, int draw,
                   const unsigned long long *__restrict__ exact_thr, int exact_g, int exact_r) {
    const long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) *count_next = 0;
    bool sg = false, sr = false;
    if (b < B) {
        if (draw) {
            const uint32_t gb = (uint32_t)(block_begin + b);
            // R = 0: the compressor keeps nothing (C = 0).  exact_*: keep the blocks whose key
            // (word0, block id) is not above the k-th smallest key (exact-count GRBS).
            if (R_g != 0) {
                const uint32_t w = philox4x32_10_word0(k0, k1, gb, t_lo, t_hi, 0u);
                sg = exact_g ? ((((unsigned long long)w << 32) | gb) <= exact_thr[0])
                             : ((unsigned long long)w * R_g < (1ull << 32));
            }
            mask_g[b] = sg ? 1 : 0;
            if (is_reset) {
                if (R_r != 0) {
                    const uint32_t w = philox4x32_10_word0(k0, k1, gb, t_lo, t_hi, 1u);
                    sr = exact_r ? ((((unsigned long long)w << 32) | gb) <= exact_thr[1])
                                 : ((unsigned long long)w * R_r < (1ull << 32));
                }
                mask_r[b] = sr ? 1 : 0;
            }
        } else {
            sg = mask_g[b] != 0;
            sr = is_reset ? (mask_r[b] != 0) : false;
        }
    }
    const bool need = sg || sr;
    const unsigned ballot = __ballot_sync(0xffffffffu, need);
    if (ballot == 0) return;
    const unsigned lane = threadIdx.x & 31;
    const int leader = __ffs(ballot) - 1;
    unsigned base = 0;
    if ((int)lane == leader) base = atomicAdd(count, (unsigned)__popc(ballot));
    base = __shfl_sync(0xffffffffu, base, leader);
    // The list holds B entries.  A counter that was not cleared (overlapping allocation-free steps
    // race on it) must not carry an append past the end.
    const unsigned at = base + __popc(ballot & ((1u << lane) - 1u));
    if (need && at < (unsigned long long)B) list[at] = (uint32_t)b;
}


// ------------------------------------------------------------------ replayable steps
// For a step that is captured once in a CUDA graph and replayed, the iteration number cannot
// be a launch argument.  It lives in device memory instead.  Block c[0] and buffer set 0
// describe the iteration the step kernels are working on; while they run, the select kernel
// prepares iteration c[0].t + 1 in buffer set 1 and publishes it in c[1] (its last CTA to
// finish does so: a counter, no waiting).  A small kernel at the start of every step copies
// set 1 and c[1] over set 0 and c[0].  Nothing ever waits on anything, and the step kernels
// read their masks from the same place as in an ordinary step.
struct StepCtl {
    unsigned long long t;      // the iteration this block describes
    uint32_t reset;            // it is a reset step
    uint32_t done;             // CTAs of the select kernel filling this block that have finished
    uint32_t count;            // blocks in this iteration's list
    uint32_t pad;
};
struct ReplayCtl {
    StepCtl c[2];              // [0] current, [1] prepared for the next step
};

// Buffer set 1 lies `stride` entries after set 0.  One thread per block.
__global__ void __launch_bounds__(256)
replay_advance_kernel(ReplayCtl *R, uint8_t *__restrict__ mask_g, uint8_t *__restrict__ mask_r,
                      uint32_t *__restrict__ list, long long stride, long long B) {
    const long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t count = R->c[1].count, reset = R->c[1].reset;
    const unsigned long long t = R->c[1].t;
    if (b < B) {
        mask_g[b] = mask_g[stride + b];
        if (reset) mask_r[b] = mask_r[stride + b];
        if (b < count) list[b] = list[stride + b];
    }
    // the last CTA to finish moves the control block over and re-arms the other one
    __shared__ bool last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        last = atomicAdd(&R->c[0].done, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        R->c[0].t = t, R->c[0].reset = reset, R->c[0].count = count, R->c[0].done = 0;
        R->c[1].count = 0, R->c[1].done = 0;
    }
}

__global__ void __launch_bounds__(256)
grbs_select_replay_kernel(ReplayCtl *R, uint8_t *__restrict__ mask_g, uint8_t *__restrict__ mask_r,
                          uint32_t *__restrict__ list, long long stride, long long B,
                          long long block_begin, uint32_t k0, uint32_t k1, uint32_t R_g, uint32_t R_r,
                          uint32_t H) {
    const unsigned long long t = R->c[0].t + 1ull;      // c[0] does not change while this kernel runs
    const bool is_reset = (t % H) == 0;
    const uint32_t t_lo = (uint32_t)(t & 0xffffffffu), t_hi = (uint32_t)(t >> 32);
    StepCtl *out = &R->c[1];
    mask_g += stride, mask_r += stride, list += stride;
    const long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    bool sg = false, sr = false;
    if (b < B) {
        const uint32_t gb = (uint32_t)(block_begin + b);
        if (R_g != 0)
            sg = (unsigned long long)philox4x32_10_word0(k0, k1, gb, t_lo, t_hi, 0u) * R_g < (1ull << 32);
        mask_g[b] = sg ? 1 : 0;
        if (is_reset) {
            sr = (unsigned long long)philox4x32_10_word0(k0, k1, gb, t_lo, t_hi, 1u) * R_r < (1ull << 32);
            mask_r[b] = sr ? 1 : 0;
        }
    }
    const bool need = sg || sr;
    const unsigned ballot = __ballot_sync(0xffffffffu, need);
    if (ballot != 0) {
        const unsigned lane = threadIdx.x & 31;
        const int leader = __ffs(ballot) - 1;
        unsigned base = 0;
        if ((int)lane == leader) base = atomicAdd(&out->count, (unsigned)__popc(ballot));
        base = __shfl_sync(0xffffffffu, base, leader);
        const unsigned at = base + __popc(ballot & ((1u << lane) - 1u));
        if (need && at < (unsigned long long)B) list[at] = (uint32_t)b;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&out->done, 1u) == gridDim.x - 1) {   // last CTA: publish the iteration
            out->t = t;
            out->reset = is_reset ? 1u : 0u;
        }
    }
}
