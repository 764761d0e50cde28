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

// Exclusive scan of the two masks in block order (one CTA): pos_*[b] = selected blocks below b,
// olist_* = the selected blocks in ascending order.
__global__ void __launch_bounds__(1024)
ordered_lists_kernel(const uint8_t *__restrict__ mask_g, const uint8_t *__restrict__ mask_r, long long B,
                     int is_reset, uint32_t *__restrict__ pos_g, uint32_t *__restrict__ pos_r,
                     uint32_t *__restrict__ olist_g, uint32_t *__restrict__ olist_r) {
    __shared__ uint32_t part[2][1024];
    const long long chunk = (B + blockDim.x - 1) / blockDim.x;
    const long long b0 = min(B, (long long)threadIdx.x * chunk), b1 = min(B, b0 + chunk);
    uint32_t cg = 0, cr = 0;
    for (long long b = b0; b < b1; ++b) {
        cg += mask_g[b] != 0;
        if (is_reset) cr += mask_r[b] != 0;
    }
    part[0][threadIdx.x] = cg, part[1][threadIdx.x] = cr;
    __syncthreads();
    uint32_t og = 0, orr = 0;
    for (int j = 0; j < (int)threadIdx.x; ++j) og += part[0][j], orr += part[1][j];
    for (long long b = b0; b < b1; ++b) {
        pos_g[b] = og;
        if (mask_g[b]) olist_g[og++] = (uint32_t)b;
        if (is_reset) {
            pos_r[b] = orr;
            if (mask_r[b]) olist_r[orr++] = (uint32_t)b;
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

