// step_kernels.cuh - the two step kernels: streaming (unselected blocks) and selected-block walker; vector pack helpers, Get_p
// Device code of the CSER step library; included by cser.cu inside its unnamed namespace.
#pragma once
// ------------------------------------------------------------------ fused step
template <int V>
struct Pack {
    float v[V];
};

template <int V>
__device__ __forceinline__ Pack<V> ld(const float *p) {
    Pack<V> r;
    if constexpr (V == 4) {
        const float4 t = *reinterpret_cast<const float4 *>(p);
        r.v[0] = t.x, r.v[1] = t.y, r.v[2] = t.z, r.v[3] = t.w;
    } else {
        r.v[0] = *p;
    }
    return r;
}

// gradients are read exactly once: stream them past the caches
template <int V>
__device__ __forceinline__ Pack<V> ld_stream(const float *p) {
    Pack<V> r;
    if constexpr (V == 4) {
        const float4 t = __ldcs(reinterpret_cast<const float4 *>(p));
        r.v[0] = t.x, r.v[1] = t.y, r.v[2] = t.z, r.v[3] = t.w;
    } else {
        r.v[0] = __ldcs(p);
    }
    return r;
}

template <int V>
__device__ __forceinline__ void st(float *p, const Pack<V> &a) {
    if constexpr (V == 4) {
        *reinterpret_cast<float4 *>(p) = make_float4(a.v[0], a.v[1], a.v[2], a.v[3]);
    } else {
        *p = a.v[0];
    }
}

struct StepParams {
    const float *g;
    float *x, *e, *m;
    const uint8_t *mask_g, *mask_r;
    const uint32_t *list;    // blocks selected by either mask this step
    const uint32_t *count;   // how many
    const ReplayCtl *rctl;   // replayable steps: reset flag and list length are read on the device (else NULL)
    long long d;             // elements per row
    long long cols_total;    // vector columns per row
    long long c_begin;       // first vector column handled by this launch
    long long c_end;         // one past the last
    unsigned bsv;            // GRBS block size in vector columns
    unsigned tiles;          // tiles of 256 vector columns in [c_begin, c_end)
    int n;
    float eta, beta, n_f;
};

// Get_p (Appendix A.4) for one pack; updates m in place when MOM.
template <int V, bool MOM>
__device__ __forceinline__ Pack<V> get_p(const Pack<V> &g, Pack<V> &m, float eta, float beta) {
    Pack<V> p;
#pragma unroll
    for (int k = 0; k < V; ++k) {
        if constexpr (MOM) {
            const float t1 = beta * m.v[k];
            m.v[k] = t1 + g.v[k];
            const float t2 = beta * m.v[k];
            p.v[k] = eta * (t2 + g.v[k]);
        } else {
            p.v[k] = eta * g.v[k];
        }
    }
    return p;
}

constexpr int kStepThreads = 256;   // streaming kernel: one CTA = 256 vector columns of one row
constexpr int kWalkThreads = 128;   // selected-block kernel
constexpr int kWalkBatch = 4;       // workers whose loads a walking thread keeps in flight (worker-sharded pack)
// Batch sizes of the selected-block kernel.  Measured on B200: 2, 4 and 8 are within 2 % of each
// other on every workload (more loads in flight per thread cost registers, hence occupancy).
#ifndef CSER_WALK_UA
#define CSER_WALK_UA(mom) 4
#define CSER_WALK_UB(reset_err) 4
#define CSER_WALK_UF 4
#define CSER_WALK_UR(mom) 2
#endif
#ifndef CSER_DENSE_WALK_FRACTION
#define CSER_DENSE_WALK_FRACTION 0.3
#endif
constexpr double kDenseWalkFraction = CSER_DENSE_WALK_FRACTION;   // expected selected share from which the walk is dense

// Selected blocks (1/R of the data): the update needs the mean over workers, so here one
// thread owns one vector column of a selected block and walks the worker axis.  Threads
// are laid over the concatenation of the listed blocks, so CTAs are full whatever the
// block size.  Each pass issues the loads of kWalkBatch workers before it consumes any of
// them (the in-place stores would otherwise keep the compiler from hoisting the next
// worker's loads), and sums in ascending worker order starting from worker 0's value.
// This kernel has its own register budget; the streaming kernel stays at 32 registers.
// DENSE = false: threads are laid over the listed blocks (few blocks selected).  DENSE =
// true: one thread per column of the whole range, returning at once if no mask selects its
// block; used when a large share of the blocks is selected, where walking the columns in
// their natural order is worth more than the idle threads cost.
template <int V, bool MOM, bool RESET, bool ERR, bool DENSE>
__global__ void __launch_bounds__(kWalkThreads) cser_selected_kernel(const StepParams P) {
    // workers whose loads are in flight together: fewer arrays per worker allow more workers
    constexpr int UA = CSER_WALK_UA(MOM);                      // pass A: g (+ m)
    constexpr int UB = CSER_WALK_UB(RESET && ERR);             // pass B: x (+ e on reset steps)
    constexpr int UF = CSER_WALK_UF;                           // last pass: x only
    const uint8_t *__restrict__ mask_g = P.mask_g;
    const uint8_t *__restrict__ mask_r = P.mask_r;
    const uint32_t *__restrict__ list = P.list;
    const uint32_t n_listed = DENSE ? 0u : (P.rctl ? P.rctl->c[0].count : *P.count);
    const bool reset_on = RESET && (P.rctl ? P.rctl->c[0].reset != 0 : true);
    const unsigned long long total =
        DENSE ? (unsigned long long)(P.c_end - P.c_begin) : (unsigned long long)n_listed * P.bsv;
    const long long d = P.d;
    const int n = P.n;
    const float eta = P.eta, beta = P.beta;
    for (unsigned long long f = (unsigned long long)blockIdx.x * kWalkThreads + threadIdx.x; f < total;
         f += (unsigned long long)gridDim.x * kWalkThreads) {
        long long c;
        unsigned blk;
        if constexpr (DENSE) {
            c = P.c_begin + (long long)f;
            blk = (P.c_end <= 0xffffffffll) ? (uint32_t)c / P.bsv : (unsigned)((unsigned long long)c / P.bsv);
        } else {
            const unsigned long long entry =
                (total <= 0xffffffffull) ? (unsigned long long)((uint32_t)f / P.bsv) : f / P.bsv;
            blk = list[entry];
            c = (long long)blk * P.bsv + (long long)(f - entry * P.bsv);
            if (c >= P.cols_total || c < P.c_begin || c >= P.c_end) continue;
        }
        const bool sg = mask_g[blk] != 0;
        const bool sr = reset_on ? (mask_r[blk] != 0) : false;
        if constexpr (DENSE) {
            if (!sg && !sr) continue;
        }
        const float *__restrict__ g = P.g + c * V;
        float *__restrict__ x = P.x + c * V;
        float *__restrict__ e = ERR ? P.e + c * V : nullptr;
        float *__restrict__ m = MOM ? P.m + c * V : nullptr;
        // With an error array: sum over workers of e_{t-1/2}.  Without one (implementation
        // II): sum over workers of x_{t-1/2}.  Reset-selected blocks only.
        Pack<V> sum_r;
#pragma unroll
        for (int k = 0; k < V; ++k) sum_r.v[k] = 0.f;

        if (sg) {
            // Update-selected block: r = 0, p' = mean_k p_k.  Pass A forms the mean and updates m.
            Pack<V> sum_p;
#pragma unroll
            for (int k = 0; k < V; ++k) sum_p.v[k] = 0.f;
            for (int i0 = 0; i0 < n; i0 += UA) {
                Pack<V> gv[UA], mv[UA];
#pragma unroll
                for (int u = 0; u < UA; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
                        gv[u] = ld_stream<V>(g + o);
                        if constexpr (MOM) mv[u] = ld<V>(m + o);
                    }
                }
#pragma unroll
                for (int u = 0; u < UA; ++u) {
                    if (i0 + u < n) {
                        const Pack<V> p = get_p<V, MOM>(gv[u], mv[u], eta, beta);
                        if constexpr (MOM) st<V>(m + (long long)(i0 + u) * d, mv[u]);
#pragma unroll
                        for (int k = 0; k < V; ++k)
                            sum_p.v[k] = (i0 + u == 0) ? p.v[k] : sum_p.v[k] + p.v[k];
                    }
                }
            }
            Pack<V> pbar;
#pragma unroll
            for (int k = 0; k < V; ++k) pbar.v[k] = sum_p.v[k] / P.n_f;
            // Pass B: x_i -= p-bar; e untouched.  If the block is reset-selected too: with an
            // error array store (x_i - p-bar) - e_i, zero e and gather sum_k e_k; without one
            // gather sum_k (x_k - p-bar) and store nothing yet.
            for (int i0 = 0; i0 < n; i0 += UB) {
                Pack<V> xv[UB], ev[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
                        xv[u] = ld<V>(x + o);
                        if constexpr (ERR) {
                            if (sr) ev[u] = ld<V>(e + o);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
#pragma unroll
                        for (int k = 0; k < V; ++k) xv[u].v[k] = xv[u].v[k] - pbar.v[k];
                        if (sr) {
                            if constexpr (ERR) {
                                Pack<V> z;
#pragma unroll
                                for (int k = 0; k < V; ++k) {
                                    sum_r.v[k] = (i0 + u == 0) ? ev[u].v[k] : sum_r.v[k] + ev[u].v[k];
                                    xv[u].v[k] = xv[u].v[k] - ev[u].v[k];
                                    z.v[k] = 0.f;
                                }
                                st<V>(e + o, z);
                                st<V>(x + o, xv[u]);
                            } else {
#pragma unroll
                                for (int k = 0; k < V; ++k)
                                    sum_r.v[k] = (i0 + u == 0) ? xv[u].v[k] : sum_r.v[k] + xv[u].v[k];
                            }
                        } else {
                            st<V>(x + o, xv[u]);
                        }
                    }
                }
            }
        } else {
            // Selected by the reset mask only: take the residual step (x_{t-1/2} = x - p,
            // e_{t-1/2} = e - p).  With an error array store x_{t-1/2} - e_{t-1/2}, zero e and
            // gather sum_k e_{k,t-1/2}; without one gather sum_k x_{k,t-1/2}.
            constexpr int U2 = CSER_WALK_UR(MOM);             // g, x, e (+ m)
            for (int i0 = 0; i0 < n; i0 += U2) {
                Pack<V> gv[U2], mv[U2], xv[U2], ev[U2];
#pragma unroll
                for (int u = 0; u < U2; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
                        gv[u] = ld_stream<V>(g + o);
                        if constexpr (MOM) mv[u] = ld<V>(m + o);
                        xv[u] = ld<V>(x + o);
                        if constexpr (ERR) ev[u] = ld<V>(e + o);
                    }
                }
#pragma unroll
                for (int u = 0; u < U2; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
                        const Pack<V> p = get_p<V, MOM>(gv[u], mv[u], eta, beta);
                        if constexpr (MOM) st<V>(m + o, mv[u]);
                        if constexpr (ERR) {
                            Pack<V> z;
#pragma unroll
                            for (int k = 0; k < V; ++k) {
                                const float xh = xv[u].v[k] - p.v[k];
                                const float eh = ev[u].v[k] - p.v[k];
                                sum_r.v[k] = (i0 + u == 0) ? eh : sum_r.v[k] + eh;
                                xv[u].v[k] = xh - eh;
                                z.v[k] = 0.f;
                            }
                            st<V>(x + o, xv[u]);
                            st<V>(e + o, z);
                        } else {
#pragma unroll
                            for (int k = 0; k < V; ++k) {
                                const float xh = xv[u].v[k] - p.v[k];
                                sum_r.v[k] = (i0 + u == 0) ? xh : sum_r.v[k] + xh;
                            }
                        }
                    }
                }
            }
        }

        if (sr) {
            Pack<V> rbar;
#pragma unroll
            for (int k = 0; k < V; ++k) rbar.v[k] = sum_r.v[k] / P.n_f;
            if constexpr (ERR) {
                // Error reset (Algorithm 2 lines 11-12):
                // x_i = (x_{i,t-1/2} - e_{i,t-1/2}) + mean_k e_{k,t-1/2}.
                for (int i0 = 0; i0 < n; i0 += UF) {
                    Pack<V> xv[UF];
#pragma unroll
                    for (int u = 0; u < UF; ++u)
                        if (i0 + u < n) xv[u] = ld<V>(x + (long long)(i0 + u) * d);
#pragma unroll
                    for (int u = 0; u < UF; ++u) {
                        if (i0 + u < n) {
#pragma unroll
                            for (int k = 0; k < V; ++k) xv[u].v[k] = xv[u].v[k] + rbar.v[k];
                            st<V>(x + (long long)(i0 + u) * d, xv[u]);
                        }
                    }
                }
            } else {
                // Implementation II (Appendix A.4): x_i = mean_k x_{k,t-1/2} for every worker.
                for (int i = 0; i < n; ++i) st<V>(x + (long long)i * d, rbar);
            }
        }
    }
}

// Unselected blocks (all but 1/R of the data), purely elementwise.  1-D grid: CTA
// i * tiles + tile streams tile `tile` of worker i, so consecutive CTAs walk one row after
// the other, contiguously.  Thread t owns vector column c = c_begin + 256 * tile + t and
// leaves it alone if a mask selects its block.
template <int V, bool MOM, bool RESET, bool ERR>
__global__ void __launch_bounds__(kStepThreads, 8) cser_stream_kernel(const StepParams P) {
    const unsigned row = blockIdx.x / P.tiles;
    const unsigned tile = blockIdx.x - row * P.tiles;
    const long long c = P.c_begin + (long long)tile * kStepThreads + threadIdx.x;
    if (c >= P.c_end) return;
    const long long b = (P.c_end <= 0xffffffffll) ? (long long)((uint32_t)c / P.bsv)
                                                  : (long long)((unsigned long long)c / P.bsv);
    if (P.mask_g[b] != 0) return;
    if (RESET && P.mask_r[b] != 0 && (P.rctl == nullptr || P.rctl->c[0].reset != 0)) return;
    // C(p) = 0, so p' = r = p (Algorithm 3 lines 4-8): x_i -= p_i, e_i -= p_i (no e array in
    // implementation II).
    const long long o = (long long)row * P.d + c * V;
    const Pack<V> gv = ld_stream<V>(P.g + o);
    Pack<V> mv;
    if constexpr (MOM) mv = ld<V>(P.m + o);
    Pack<V> xv = ld<V>(P.x + o);
    Pack<V> ev;
    if constexpr (ERR) ev = ld<V>(P.e + o);
    const Pack<V> p = get_p<V, MOM>(gv, mv, P.eta, P.beta);
#pragma unroll
    for (int k = 0; k < V; ++k) {
        xv.v[k] = xv.v[k] - p.v[k];
        if constexpr (ERR) ev.v[k] = ev.v[k] - p.v[k];
    }
    if constexpr (MOM) st<V>(P.m + o, mv);
    st<V>(P.x + o, xv);
    if constexpr (ERR) st<V>(P.e + o, ev);
}

// x_i <- x0 for all workers; e, m <- 0
__global__ void __launch_bounds__(256)
broadcast_x0_kernel(const float *__restrict__ x0, float *__restrict__ x, float *__restrict__ e,
                    float *__restrict__ m, long long d, int n) {
    const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    const float v = x0[j];
    for (int i = 0; i < n; ++i) {
        const long long o = (long long)i * d + j;
        x[o] = v;
        if (e) e[o] = 0.f;
        if (m) m[o] = 0.f;
    }
}

