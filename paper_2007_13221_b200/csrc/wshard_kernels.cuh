// wshard_kernels.cuh - worker-sharded step: ordered lists of the selected blocks, pack and apply kernels
// Device code of the CSER step library; included by cser.cu inside its unnamed namespace.
#pragma once
#include "step_kernels.cuh"

// ------------------------------------------------------------------ worker-sharded step
// Several GPUs each hold some of the workers (all d columns).  The mean of Algorithm 3 line 7
// then needs one all-reduce per step.  GRBS makes the compressed vectors directly summable
// (Section 3.3): every rank selects the same blocks, so each rank packs the sum over its own
// workers of the selected blocks into a dense message, the messages are summed across ranks,
// and each rank applies sum / n_total.  The message holds the update-selected blocks in
// ascending block order and, on a reset step, the reset-selected blocks after them.

// Exclusive scan of the two masks in block order: pos_*[b] = selected blocks below b, olist_* = the
// selected blocks in ascending order.  One CTA per 1024 blocks; a CTA first counts the flags in front of
// its own blocks (B bytes at most, from L2, four flags per load), then scans its own 1024.  No CTA waits
// for another.  mask_r may be NULL (not a reset step).
constexpr int kScanThreads = 1024;
__device__ __forceinline__ uint32_t block_sum_1024(uint32_t v, uint32_t *warp_sums) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                       // warp_sums may still be read from the previous use
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t t = 0;
    for (int w = 0; w < kScanThreads / 32; ++w) t += warp_sums[w];
    return t;
}

__global__ void __launch_bounds__(kScanThreads)
ordered_lists_kernel(const uint8_t *__restrict__ mask_g, const uint8_t *__restrict__ mask_r, long long B,
                     uint32_t *__restrict__ pos_g, uint32_t *__restrict__ pos_r,
                     uint32_t *__restrict__ olist_g, uint32_t *__restrict__ olist_r) {
    __shared__ uint32_t warp_sums[kScanThreads / 32];
    const long long first = (long long)blockIdx.x * kScanThreads;     // a multiple of 4: word loads stay aligned
    const long long b = first + threadIdx.x;
    for (int which = 0; which < 2; ++which) {
        const uint8_t *__restrict__ mask = which ? mask_r : mask_g;
        if (!mask) continue;
        uint32_t *__restrict__ pos = which ? pos_r : pos_g;
        uint32_t *__restrict__ olist = which ? olist_r : olist_g;
        // flags in front of this CTA's blocks (flags are 0 / 1 bytes: dp4a adds four at a time)
        const uint32_t *words = reinterpret_cast<const uint32_t *>(mask);
        uint32_t part = 0;
        for (long long w = threadIdx.x; w < first / 4; w += kScanThreads) part = __dp4a(words[w], 0x01010101u, part);
        const uint32_t before = block_sum_1024(part, warp_sums);
        // exclusive scan of this CTA's flags
        const uint32_t flag = (b < B && mask[b] != 0) ? 1u : 0u;
        uint32_t incl = flag;
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)(threadIdx.x & 31) >= o) incl += up;
        }
        __syncthreads();
        if ((threadIdx.x & 31) == 31) warp_sums[threadIdx.x >> 5] = incl;
        __syncthreads();
        uint32_t warps_before = 0;
        for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) warps_before += warp_sums[w];
        const uint32_t at = before + warps_before + incl - flag;
        if (b < B) {
            pos[b] = at;
            if (flag) olist[at] = (uint32_t)b;
        }
    }
}

struct ShardParams {
    const float *g;
    float *x, *e, *m;
    float *msg;                       // [k_g * bs | k_r * bs] floats
    const uint8_t *mask_g, *mask_r;
    const uint32_t *pos_g, *olist_g, *olist_r;
    long long d, cols_total;
    unsigned bsv, k_g, k_r;
    int n;                            // local workers
    float eta, beta, n_total_f;
};

// Pack: thread f owns vector column (f % bsv) of message block (f / bsv).
template <int V, bool MOM, bool RESET>
__global__ void __launch_bounds__(kWalkThreads) wshard_pack_kernel(const ShardParams P) {
    constexpr int U = kWalkBatch;
    const unsigned long long total = (unsigned long long)(P.k_g + (RESET ? P.k_r : 0u)) * P.bsv;
    const long long d = P.d;
    const int n = P.n;
    for (unsigned long long f = (unsigned long long)blockIdx.x * kWalkThreads + threadIdx.x; f < total;
         f += (unsigned long long)gridDim.x * kWalkThreads) {
        const unsigned entry = (unsigned)(f / P.bsv);
        const unsigned col = (unsigned)(f - (unsigned long long)entry * P.bsv);
        const bool r_section = entry >= P.k_g;
        const unsigned blk = r_section ? P.olist_r[entry - P.k_g] : P.olist_g[entry];
        const long long c = (long long)blk * P.bsv + col;
        Pack<V> sum;
#pragma unroll
        for (int q = 0; q < V; ++q) sum.v[q] = 0.f;
        if (c < P.cols_total) {
            const float *__restrict__ g = P.g + c * V;
            float *__restrict__ x = P.x + c * V;
            float *__restrict__ e = P.e + c * V;
            float *__restrict__ m = MOM ? P.m + c * V : nullptr;
            if (!r_section) {
                // update-selected block: sum of the local workers' p, ascending; m updated
                for (int i0 = 0; i0 < n; i0 += U) {
                    Pack<V> gv[U], mv[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (i0 + u < n) {
                            const long long o = (long long)(i0 + u) * d;
                            gv[u] = ld_stream<V>(g + o);
                            if constexpr (MOM) mv[u] = ld<V>(m + o);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (i0 + u < n) {
                            const Pack<V> p = get_p<V, MOM>(gv[u], mv[u], P.eta, P.beta);
                            if constexpr (MOM) st<V>(m + (long long)(i0 + u) * d, mv[u]);
#pragma unroll
                            for (int q = 0; q < V; ++q) sum.v[q] = (i0 + u == 0) ? p.v[q] : sum.v[q] + p.v[q];
                        }
                    }
                }
            } else if (P.mask_g[blk] != 0) {
                // reset-selected and update-selected: e is unchanged by this step; sum the local e
                for (int i = 0; i < n; ++i) {
                    const Pack<V> ev = ld<V>(e + (long long)i * d);
#pragma unroll
                    for (int q = 0; q < V; ++q) sum.v[q] = (i == 0) ? ev.v[q] : sum.v[q] + ev.v[q];
                }
            } else {
                // reset-selected only: residual step, store x_{t-1/2} - e_{t-1/2}, zero e, sum e_{t-1/2}
                for (int i = 0; i < n; ++i) {
                    const long long o = (long long)i * d;
                    const Pack<V> gv = ld_stream<V>(g + o);
                    Pack<V> mv, xv = ld<V>(x + o);
                    const Pack<V> ev = ld<V>(e + o);
                    if constexpr (MOM) mv = ld<V>(m + o);
                    const Pack<V> p = get_p<V, MOM>(gv, mv, P.eta, P.beta);
                    if constexpr (MOM) st<V>(m + o, mv);
                    Pack<V> z;
#pragma unroll
                    for (int q = 0; q < V; ++q) {
                        const float xh = xv.v[q] - p.v[q];
                        const float eh = ev.v[q] - p.v[q];
                        sum.v[q] = (i == 0) ? eh : sum.v[q] + eh;
                        xv.v[q] = xh - eh;
                        z.v[q] = 0.f;
                    }
                    st<V>(x + o, xv);
                    st<V>(e + o, z);
                }
            }
        }
        st<V>(P.msg + ((size_t)entry * P.bsv + col) * V, sum);   // columns past the end of the vector: zeros
    }
}

// Apply the summed message: thread f owns one vector column of one message block.
template <int V, bool RESET>
__global__ void __launch_bounds__(kWalkThreads) wshard_apply_kernel(const ShardParams P) {
    const unsigned long long total = (unsigned long long)(P.k_g + (RESET ? P.k_r : 0u)) * P.bsv;
    const long long d = P.d;
    const int n = P.n;
    for (unsigned long long f = (unsigned long long)blockIdx.x * kWalkThreads + threadIdx.x; f < total;
         f += (unsigned long long)gridDim.x * kWalkThreads) {
        const unsigned entry = (unsigned)(f / P.bsv);
        const unsigned col = (unsigned)(f - (unsigned long long)entry * P.bsv);
        const bool r_section = entry >= P.k_g;
        const unsigned blk = r_section ? P.olist_r[entry - P.k_g] : P.olist_g[entry];
        const long long c = (long long)blk * P.bsv + col;
        if (c >= P.cols_total) continue;
        float *__restrict__ x = P.x + c * V;
        float *__restrict__ e = P.e + c * V;
        const Pack<V> sv = ld<V>(P.msg + ((size_t)entry * P.bsv + col) * V);
        Pack<V> mean;
#pragma unroll
        for (int q = 0; q < V; ++q) mean.v[q] = sv.v[q] / P.n_total_f;
        if (!r_section) {
            if (RESET && P.mask_r[blk] != 0) continue;   // its reset-section thread does both updates
            for (int i = 0; i < n; ++i) {                // x_i -= mean_k p_k
                Pack<V> xv = ld<V>(x + (long long)i * d);
#pragma unroll
                for (int q = 0; q < V; ++q) xv.v[q] = xv.v[q] - mean.v[q];
                st<V>(x + (long long)i * d, xv);
            }
        } else if (P.mask_g[blk] != 0) {
            // both masks: x_i = ((x_i - p-bar) - e_i) + e-bar, e_i = 0
            const Pack<V> sp = ld<V>(P.msg + ((size_t)P.pos_g[blk] * P.bsv + col) * V);
            for (int i = 0; i < n; ++i) {
                const long long o = (long long)i * d;
                Pack<V> xv = ld<V>(x + o);
                const Pack<V> ev = ld<V>(e + o);
                Pack<V> z;
#pragma unroll
                for (int q = 0; q < V; ++q) {
                    const float pbar = sp.v[q] / P.n_total_f;
                    xv.v[q] = ((xv.v[q] - pbar) - ev.v[q]) + mean.v[q];
                    z.v[q] = 0.f;
                }
                st<V>(x + o, xv);
                st<V>(e + o, z);
            }
        } else {
            for (int i = 0; i < n; ++i) {                // x_i = (x_{t-1/2} - e_{t-1/2}) + e-bar
                Pack<V> xv = ld<V>(x + (long long)i * d);
#pragma unroll
                for (int q = 0; q < V; ++q) xv.v[q] = xv.v[q] + mean.v[q];
                st<V>(x + (long long)i * d, xv);
            }
        }
    }
}

