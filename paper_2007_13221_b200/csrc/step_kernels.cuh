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
    ReplayCtl *rctl;         // replayable steps: iteration, reset flag and list length live on the device (else NULL)
    long long d;             // elements per row
    long long cols_total;    // vector columns per row
    long long c_begin;       // first vector column handled by this launch
    long long c_end;         // one past the last
    unsigned bsv;            // GRBS block size in vector columns
    unsigned tiles;          // tiles of 256 vector columns in [c_begin, c_end)
    unsigned list_cap;       // entries the list can hold (blocks of the vector): bounds whatever *count says
    // shared-memory staged selected-block kernel only:
    unsigned chunk_cols;     // vector columns per work unit
    unsigned n_chunks;       // work units per block
    unsigned stages;         // stages of the copy ring
    unsigned *err_word;      // host-visible word a wait that ran out raises (may be NULL)
    unsigned wait_mcycles;   // limit of every barrier wait, in millions of SM clock cycles
    unsigned test_stall;     // test hook: CTA 0 announces 16 bytes for its first unit that never arrive
    // single-launch kernel for small problems only (it draws the masks itself):
    uint8_t *mask_g_out, *mask_r_out;
    long long block_begin;   // global id of block 0
    uint32_t k0, k1, t_lo, t_hi, R1, R2;
    uint32_t H;              // reset interval (replayable single-launch steps decide on the device)
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
// Batch sizes of the selected-block kernel: workers whose loads are in flight together in each pass.
// Measured on B200: 2, 4 and 8 are within 2 % of each other where few blocks are selected; with many
// selected blocks 8 loses to 4 (more loads in flight per thread cost registers, hence occupancy).
#ifndef CSER_WALK_UA
#define CSER_WALK_UA 4      // update-selected, first pass: g (+ m) (+ e when the block is reset too)
#define CSER_WALK_UB 4      // update-selected, second pass: x (+ e)
#define CSER_WALK_UR 2      // reset-selected only: g (+ m) + x + e
#endif
#ifndef CSER_DENSE_WALK_FRACTION
#define CSER_DENSE_WALK_FRACTION 0.3
#endif
constexpr double kDenseWalkFraction = CSER_DENSE_WALK_FRACTION;   // expected selected share from which the walk is dense

// Selected blocks (1/R of the data): the update needs the mean over workers, so here one
// thread owns one vector column of a selected block and walks the worker axis.  Threads
// are laid over the concatenation of the listed blocks, so CTAs are full whatever the
// block size.  Each pass issues the loads of a batch of workers before it consumes any of
// them (the in-place stores would otherwise keep the compiler from hoisting the next
// worker's loads), and sums in ascending worker order starting from worker 0's value.
// An update-selected block takes two passes over the worker axis: the first forms the means
// (p-bar and, if the block is reset-selected too, e-bar), the second writes x (and e) once; the e it
// reads again was read a moment ago by the same thread and comes from cache.
// This kernel has its own register budget; the streaming kernel stays at 32 registers.
//
// walk_selected_column: one vector column c of a block selected by the update mask (sg), the reset
// mask (sr) or both.
template <int V, bool MOM, bool RESET, bool ERR>
__device__ __forceinline__ void walk_selected_column(const StepParams &P, long long c, bool sg, bool sr) {
    constexpr int UA = CSER_WALK_UA, UB = CSER_WALK_UB, UR = CSER_WALK_UR;
    const long long d = P.d;
    const int n = P.n;
    const float eta = P.eta, beta = P.beta, n_f = P.n_f;
    Pack<V> zero;
#pragma unroll
    for (int k = 0; k < V; ++k) zero.v[k] = 0.f;
    const float *__restrict__ g = P.g + c * V;
    float *__restrict__ x = P.x + c * V;
    float *__restrict__ e = ERR ? P.e + c * V : nullptr;
    float *__restrict__ m = MOM ? P.m + c * V : nullptr;
    if (sg) {
        // Update-selected block (Algorithm 3 with C(v) = v): r = 0, p' = mean_k p_k.  First pass:
        // the mean of p, m updated; if the block is reset-selected too (with an error array) the
        // mean of e as well, e being unchanged by this step's update.
        Pack<V> sum_p = zero, sum_r = zero;
        const bool with_e = RESET && ERR && sr;
        for (int i0 = 0; i0 < n; i0 += UA) {
            Pack<V> gv[UA], mv[UA], ev[UA];
#pragma unroll
            for (int u = 0; u < UA; ++u) {
                if (i0 + u < n) {
                    const long long o = (long long)(i0 + u) * d;
                    gv[u] = ld_stream<V>(g + o);
                    if constexpr (MOM) mv[u] = ld<V>(m + o);
                    if constexpr (RESET && ERR) {
                        if (with_e) ev[u] = ld<V>(e + o);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UA; ++u) {
                if (i0 + u < n) {
                    const Pack<V> p = get_p<V, MOM>(gv[u], mv[u], eta, beta);
                    if constexpr (MOM) st<V>(m + (long long)(i0 + u) * d, mv[u]);
#pragma unroll
                    for (int k = 0; k < V; ++k) {
                        sum_p.v[k] = (i0 + u == 0) ? p.v[k] : sum_p.v[k] + p.v[k];
                        if constexpr (RESET && ERR) {
                            if (with_e) sum_r.v[k] = (i0 + u == 0) ? ev[u].v[k] : sum_r.v[k] + ev[u].v[k];
                        }
                    }
                }
            }
        }
        Pack<V> pbar, rbar = zero;
#pragma unroll
        for (int k = 0; k < V; ++k) pbar.v[k] = sum_p.v[k] / n_f;
        if constexpr (RESET && !ERR) {
            if (sr) {
                // implementation II (Appendix A.4): x_i = mean_k (x_k - p-bar); one more pass over x
                for (int i0 = 0; i0 < n; i0 += UB) {
                    Pack<V> xv[UB];
#pragma unroll
                    for (int u = 0; u < UB; ++u)
                        if (i0 + u < n) xv[u] = ld<V>(x + (long long)(i0 + u) * d);
#pragma unroll
                    for (int u = 0; u < UB; ++u) {
                        if (i0 + u < n) {
#pragma unroll
                            for (int k = 0; k < V; ++k) {
                                const float xh = xv[u].v[k] - pbar.v[k];
                                sum_r.v[k] = (i0 + u == 0) ? xh : sum_r.v[k] + xh;
                            }
                        }
                    }
                }
#pragma unroll
                for (int k = 0; k < V; ++k) rbar.v[k] = sum_r.v[k] / n_f;
                for (int i = 0; i < n; ++i) st<V>(x + (long long)i * d, rbar);
                return;
            }
        }
        if constexpr (RESET && ERR) {
#pragma unroll
            for (int k = 0; k < V; ++k) rbar.v[k] = sum_r.v[k] / n_f;
        }
        // Second pass: x_i -= p-bar, e untouched; on a reset-selected block (Algorithm 2 lines
        // 11-12) x_i = ((x_i - p-bar) - e_i) + e-bar and e_i = 0.
        for (int i0 = 0; i0 < n; i0 += UB) {
            Pack<V> xv[UB], ev[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                if (i0 + u < n) {
                    const long long o = (long long)(i0 + u) * d;
                    xv[u] = ld<V>(x + o);
                    if constexpr (RESET && ERR) {
                        if (with_e) ev[u] = ld<V>(e + o);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                if (i0 + u < n) {
                    const long long o = (long long)(i0 + u) * d;
#pragma unroll
                    for (int k = 0; k < V; ++k) xv[u].v[k] = xv[u].v[k] - pbar.v[k];
                    if constexpr (RESET && ERR) {
                        if (with_e) {
#pragma unroll
                            for (int k = 0; k < V; ++k) xv[u].v[k] = (xv[u].v[k] - ev[u].v[k]) + rbar.v[k];
                            st<V>(e + o, zero);
                        }
                    }
                    st<V>(x + o, xv[u]);
                }
            }
        }
    } else if constexpr (RESET) {
        // Selected by the reset mask only: take the residual step (x_{t-1/2} = x - p,
        // e_{t-1/2} = e - p).  With an error array store x_{t-1/2} - e_{t-1/2}, zero e and
        // gather sum_k e_{k,t-1/2}; without one gather sum_k x_{k,t-1/2}.  (Forming the sum in
        // a pass of its own and writing x once was measured and is slower here: it reads g, m
        // and e twice, and these blocks are too few for the re-reads to stay in L1.)
        Pack<V> sum_r = zero;
        for (int i0 = 0; i0 < n; i0 += UR) {
            Pack<V> gv[UR], mv[UR], xv[UR], ev[UR];
#pragma unroll
            for (int u = 0; u < UR; ++u) {
                if (i0 + u < n) {
                    const long long o = (long long)(i0 + u) * d;
                    gv[u] = ld_stream<V>(g + o);
                    if constexpr (MOM) mv[u] = ld<V>(m + o);
                    xv[u] = ld<V>(x + o);
                    if constexpr (ERR) ev[u] = ld<V>(e + o);
                }
            }
#pragma unroll
            for (int u = 0; u < UR; ++u) {
                if (i0 + u < n) {
                    const long long o = (long long)(i0 + u) * d;
                    const Pack<V> p = get_p<V, MOM>(gv[u], mv[u], eta, beta);
                    if constexpr (MOM) st<V>(m + o, mv[u]);
                    if constexpr (ERR) {
#pragma unroll
                        for (int k = 0; k < V; ++k) {
                            const float xh = xv[u].v[k] - p.v[k];
                            const float eh = ev[u].v[k] - p.v[k];
                            sum_r.v[k] = (i0 + u == 0) ? eh : sum_r.v[k] + eh;
                            xv[u].v[k] = xh - eh;
                        }
                        st<V>(x + o, xv[u]);
                        st<V>(e + o, zero);
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
        Pack<V> rbar;
#pragma unroll
        for (int k = 0; k < V; ++k) rbar.v[k] = sum_r.v[k] / n_f;
        if constexpr (ERR) {
            // Error reset (Algorithm 2 lines 11-12):
            // x_i = (x_{i,t-1/2} - e_{i,t-1/2}) + mean_k e_{k,t-1/2}.
            for (int i0 = 0; i0 < n; i0 += UB) {
                Pack<V> xv[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u)
                    if (i0 + u < n) xv[u] = ld<V>(x + (long long)(i0 + u) * d);
#pragma unroll
                for (int u = 0; u < UB; ++u) {
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

// DENSE = false: threads are laid over the listed blocks (few blocks selected).  DENSE =
// true: one thread per column of the whole range, returning at once if no mask selects its
// block; used when a large share of the blocks is selected, where walking the columns in
// their natural order is worth more than the idle threads cost.
template <int V, bool MOM, bool RESET, bool ERR, bool DENSE>
__global__ void __launch_bounds__(kWalkThreads) cser_selected_kernel(const StepParams P) {
    const uint8_t *__restrict__ mask_g = P.mask_g;
    const uint8_t *__restrict__ mask_r = P.mask_r;
    const uint32_t *__restrict__ list = P.list;
    // never trust the counter beyond the list's capacity (a caller that lets two allocation-free
    // steps overlap can leave a stale count behind)
    const uint32_t n_counted = DENSE ? 0u : (P.rctl ? P.rctl->c[0].count : *P.count);
    const uint32_t n_listed = n_counted < P.list_cap ? n_counted : P.list_cap;
    const bool reset_on = RESET && (P.rctl ? P.rctl->c[0].reset != 0 : true);
    const unsigned long long total =
        DENSE ? (unsigned long long)(P.c_end - P.c_begin) : (unsigned long long)n_listed * P.bsv;
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
        if (sg || sr) walk_selected_column<V, MOM, RESET, ERR>(P, c, sg, sr);
    }
}

// Small problems (a step of a few tens of microseconds) are bound by launches, not by bandwidth: three
// kernels, two events and two stream waits cost as much as the traffic.  For them the whole iteration
// is ONE launch: a thread owns one vector column, draws its block's GRBS mask bits itself (Definition
// 2: Philox keyed on seed, t, block; every thread of a block redoes the same few hundred integer
// operations, which is cheaper than a kernel boundary), the first thread of each block records them
// for cser_read_state, and the column is then walked over the workers: selected blocks as in the
// selected-block kernel, unselected ones elementwise (x_i -= p_i, e_i -= p_i).
// CTA width: 64 / 128 / 256 / 512 threads were measured; 128 is best or within 1 % of best on the small
// workload (59.1k steps/s against 54.5k at 256) and on the WRN-40-8-sized vector with R = 1, 2, 4.
#ifndef CSER_FUSED_THREADS
#define CSER_FUSED_THREADS 128
#endif
constexpr int kFusedThreads = CSER_FUSED_THREADS;
// Workers whose loads are in flight together on an unselected block.  Measured: on the d = 2^20, n = 8
// workload 1 / 2 / 4 / 8 give 54.7k / 59.2k / 59.1k / 47.1k steps/s; on the WRN-40-8-sized vector with R = 2,
// 4 give 921 steps/s against 902 with 2.
#ifndef CSER_FUSED_U
#define CSER_FUSED_U 4
#endif
template <bool MOM, bool RESET, bool ERR>
__global__ void __launch_bounds__(kFusedThreads) cser_fused_small_kernel(const StepParams P) {
    constexpr int V = 4, U = CSER_FUSED_U;
    // Replayable steps (P.rctl set; the RESET variant is used): the iteration number lives on the device.
    // Block c[0] holds the last iteration done; every CTA reads it, and the last CTA to finish writes it.
    uint32_t t_lo = P.t_lo, t_hi = P.t_hi;
    bool reset_on = RESET;
    unsigned long long t_dev = 0;
    if (P.rctl) {
        t_dev = P.rctl->c[0].t + 1ull;
        t_lo = (uint32_t)(t_dev & 0xffffffffu), t_hi = (uint32_t)(t_dev >> 32);
        reset_on = RESET && (t_dev % P.H) == 0;
    }
    const long long c = (long long)blockIdx.x * kFusedThreads + threadIdx.x;
    if (c < P.cols_total) {
        const unsigned blk = (uint32_t)c / P.bsv;
        const uint32_t gb = (uint32_t)(P.block_begin + blk);
        bool sg = false, sr = false;
        if (P.R1 != 0)
            sg = (unsigned long long)philox4x32_10_word0(P.k0, P.k1, gb, t_lo, t_hi, 0u) * P.R1 < (1ull << 32);
        if constexpr (RESET) {
            if (reset_on)
                sr = (unsigned long long)philox4x32_10_word0(P.k0, P.k1, gb, t_lo, t_hi, 1u) * P.R2 < (1ull << 32);
        }
        if (c == (long long)blk * P.bsv) {
            P.mask_g_out[blk] = sg ? 1 : 0;
            if constexpr (RESET) {
                if (reset_on) P.mask_r_out[blk] = sr ? 1 : 0;
            }
        }
        if (sg || sr) {
            walk_selected_column<V, MOM, RESET, ERR>(P, c, sg, sr);
        } else {
            // C(p) = 0 on this block, so p' = r = p (Algorithm 3 lines 4-8): x_i -= p_i, e_i -= p_i
            const long long d = P.d;
            const int n = P.n;
            const float *__restrict__ g = P.g + c * V;
            float *__restrict__ x = P.x + c * V;
            float *__restrict__ e = ERR ? P.e + c * V : nullptr;
            float *__restrict__ m = MOM ? P.m + c * V : nullptr;
            for (int i0 = 0; i0 < n; i0 += U) {
                Pack<V> gv[U], mv[U], xv[U], ev[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
                        gv[u] = ld_stream<V>(g + o);
                        if constexpr (MOM) mv[u] = ld<V>(m + o);
                        xv[u] = ld<V>(x + o);
                        if constexpr (ERR) ev[u] = ld<V>(e + o);
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (i0 + u < n) {
                        const long long o = (long long)(i0 + u) * d;
                        const Pack<V> p = get_p<V, MOM>(gv[u], mv[u], P.eta, P.beta);
#pragma unroll
                        for (int k = 0; k < V; ++k) {
                            xv[u].v[k] = xv[u].v[k] - p.v[k];
                            if constexpr (ERR) ev[u].v[k] = ev[u].v[k] - p.v[k];
                        }
                        if constexpr (MOM) st<V>(m + o, mv[u]);
                        st<V>(x + o, xv[u]);
                        if constexpr (ERR) st<V>(e + o, ev[u]);
                    }
                }
            }
        }
    }
    if (P.rctl) {
        // a counter, no waiting: whoever finishes last moves the iteration number on
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            if (atomicAdd(&P.rctl->c[0].done, 1u) == gridDim.x - 1) {
                P.rctl->c[0].t = t_dev;
                P.rctl->c[0].reset = reset_on ? 1u : 0u;
                P.rctl->c[0].done = 0;
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

