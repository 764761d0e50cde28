// membw_probe.cu - measurement companion of the CSER step library (libcser_probe.so).  Not part of the
// optimizer: plain kernels that move the bytes of one M-CSER step over [n, d] fp32 arrays in different
// orders and through different paths, so that the bandwidth ceilings and the design comparisons the
// step kernels are judged against can be re-measured with one command (`python bench.py --ceilings`).
//
// Patterns (all with 128-bit accesses; "row after row" = a 1-D grid of (worker, tile) CTAs dispatched
// tile-fastest, the traversal of cser_stream_kernel):
//   0  read four arrays (g, m, x, e), write nothing                       row after row
//   1  write three arrays (m, x, e), read nothing                         row after row
//   2  copy one array to another (g -> x)                                 row after row
//   3  the step's own mix: read g, m, x, e, write m, x, e in place        row after row
//   4  the same mix, one thread per column walking all n workers with `variant` workers' loads in flight
//   5  the same mix, row after row, staged through shared memory: a producer thread issues one bulk copy
//      per array and tile (variant = tile size in KB per array, 2..16; stages fill 96 KB), 256 consumer
//      threads update from shared memory and store straight to global memory
// The arithmetic is the streaming kernel's (Get_p with momentum, x -= p, e -= p), compiled without
// fused multiply-add like the library.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {
#include "bulk_copy.cuh"

struct ProbeParams {
    float *g, *m, *x, *e;
    long long d;         // elements per row, a multiple of 4
    long long cols;      // d / 4
    unsigned tiles;      // tiles of 256 vector columns per row
    int n;
    float eta, beta;
    unsigned tile_cols;  // pattern 5: vector columns per tile
    unsigned stages;
    float never;         // pattern 0: a value the data never sums to (keeps the loads alive)
};

__device__ __forceinline__ void update(float4 &g, float4 &m, float4 &x, float4 &e, float eta, float beta) {
    float *G = &g.x, *M = &m.x, *X = &x.x, *E = &e.x;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float t1 = beta * M[k];
        M[k] = t1 + G[k];
        const float t2 = beta * M[k];
        const float p = eta * (t2 + G[k]);
        X[k] = X[k] - p;
        E[k] = E[k] - p;
    }
}

template <int PATTERN>
__global__ void __launch_bounds__(256, 8) rows_kernel(const ProbeParams P) {
    const unsigned row = blockIdx.x / P.tiles, tile = blockIdx.x - row * P.tiles;
    const long long c = (long long)tile * 256 + threadIdx.x;
    if (c >= P.cols) return;
    const long long o = (long long)row * P.d + c * 4;
    float4 *g = reinterpret_cast<float4 *>(P.g + o), *m = reinterpret_cast<float4 *>(P.m + o);
    float4 *x = reinterpret_cast<float4 *>(P.x + o), *e = reinterpret_cast<float4 *>(P.e + o);
    if constexpr (PATTERN == 0) {
        const float4 a = __ldcs(g), b = *m, cc = *x, dd = *e;
        if (a.x + b.y + cc.z + dd.w == P.never) *x = a;      // never true: the loads stay, nothing is stored
    } else if constexpr (PATTERN == 1) {
        const float4 v = make_float4(1.f, 2.f, 3.f, (float)threadIdx.x);
        *m = v, *x = v, *e = v;
    } else if constexpr (PATTERN == 2) {
        *x = __ldcs(g);
    } else {
        float4 a = __ldcs(g), b = *m, cc = *x, dd = *e;
        update(a, b, cc, dd, P.eta, P.beta);
        *m = b, *x = cc, *e = dd;
    }
}

// pattern 4: one thread per vector column, all workers, U workers' loads in flight
template <int U>
__global__ void __launch_bounds__(256) column_walk_kernel(const ProbeParams P) {
    const long long c = (long long)blockIdx.x * 256 + threadIdx.x;
    if (c >= P.cols) return;
    for (int i0 = 0; i0 < P.n; i0 += U) {
        float4 a[U], b[U], cc[U], dd[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u < P.n) {
                const long long o = (long long)(i0 + u) * P.d + c * 4;
                a[u] = __ldcs(reinterpret_cast<const float4 *>(P.g + o));
                b[u] = *reinterpret_cast<const float4 *>(P.m + o);
                cc[u] = *reinterpret_cast<const float4 *>(P.x + o);
                dd[u] = *reinterpret_cast<const float4 *>(P.e + o);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u < P.n) {
                const long long o = (long long)(i0 + u) * P.d + c * 4;
                update(a[u], b[u], cc[u], dd[u], P.eta, P.beta);
                *reinterpret_cast<float4 *>(P.m + o) = b[u];
                *reinterpret_cast<float4 *>(P.x + o) = cc[u];
                *reinterpret_cast<float4 *>(P.e + o) = dd[u];
            }
        }
    }
}

// pattern 5: persistent CTAs, 256 consumer threads + one producer warp, a ring of `stages` stages of four
// tiles (g, m, x, e) each.  Every wait is bounded; a wait that runs out makes the CTA leave.
constexpr int kStagedConsumers = 256;
__global__ void __launch_bounds__(kStagedConsumers + 32) staged_rows_kernel(const ProbeParams P) {
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem);
    uint64_t *empty = full + 8;
    unsigned char *stage0 = smem + 128;
    const unsigned S = P.stages, T = P.tile_cols;
    const size_t stage_bytes = (size_t)4 * T * 16;
    const unsigned tiles_per_row = (unsigned)((P.cols + T - 1) / T);
    const unsigned long long total = (unsigned long long)tiles_per_row * P.n;
    const unsigned long long n_my = total > blockIdx.x ? (total - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    if (threadIdx.x == 0) {
        for (unsigned s = 0; s < S; ++s) mbar_init(&full[s], 1), mbar_init(&empty[s], kStagedConsumers / 32);
        mbar_init_fence();
    }
    __syncthreads();
    const unsigned warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == kStagedConsumers / 32) {
        if (lane != 0) return;
        const uint64_t pol = l2_policy_normal(), pol_g = l2_policy_evict_first();
        for (unsigned long long k = 0; k < n_my; ++k) {
            const unsigned s = (unsigned)(k % S), round = (unsigned)(k / S);
            if (round > 0 && !mbar_wait_bounded(&empty[s], (round - 1) & 1u)) return;
            const unsigned long long u = blockIdx.x + k * gridDim.x;
            const unsigned row = (unsigned)(u / tiles_per_row), tile = (unsigned)(u - (unsigned long long)row * tiles_per_row);
            const long long c0 = (long long)tile * T;
            const unsigned cols = (unsigned)((P.cols - c0) < (long long)T ? (P.cols - c0) : T);
            const long long o = (long long)row * P.d + c0 * 4;
            unsigned char *st = stage0 + (size_t)s * stage_bytes;
            mbar_arrive_expect(&full[s], 4u * cols * 16u);
            bulk_load(st, P.g + o, cols * 16u, &full[s], pol_g);
            bulk_load(st + (size_t)T * 16, P.m + o, cols * 16u, &full[s], pol);
            bulk_load(st + (size_t)2 * T * 16, P.x + o, cols * 16u, &full[s], pol);
            bulk_load(st + (size_t)3 * T * 16, P.e + o, cols * 16u, &full[s], pol);
        }
        return;
    }
    for (unsigned long long k = 0; k < n_my; ++k) {
        const unsigned s = (unsigned)(k % S);
        if (!mbar_wait_bounded(&full[s], (unsigned)(k / S) & 1u)) return;
        const unsigned long long u = blockIdx.x + k * gridDim.x;
        const unsigned row = (unsigned)(u / tiles_per_row), tile = (unsigned)(u - (unsigned long long)row * tiles_per_row);
        const long long c0 = (long long)tile * T;
        const unsigned cols = (unsigned)((P.cols - c0) < (long long)T ? (P.cols - c0) : T);
        const float4 *st = reinterpret_cast<const float4 *>(stage0 + (size_t)s * stage_bytes);
        for (unsigned c = threadIdx.x; c < cols; c += kStagedConsumers) {
            float4 a = st[c], b = st[T + c], cc = st[2 * T + c], dd = st[3 * T + c];
            update(a, b, cc, dd, P.eta, P.beta);
            const long long o = (long long)row * P.d + (c0 + c) * 4;
            *reinterpret_cast<float4 *>(P.m + o) = b;
            *reinterpret_cast<float4 *>(P.x + o) = cc;
            *reinterpret_cast<float4 *>(P.e + o) = dd;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
    }
}

}  // namespace

// Runs `pattern` (see the top of this file) `reps` times after 3 warm-up launches on device arrays
// g, m, x, e (fp32 [n, d] each, d a multiple of 4, 16-byte aligned, caller-owned) and stores the mean
// duration of one launch in *ms_out (CUDA events on `stream`; synchronizes it).  Returns 0, or -1 for a
// bad argument, or -3 for a CUDA error.
extern "C" int cser_probe_run(int pattern, int variant, float *g, float *m, float *x, float *e, long long d,
                              int n, int reps, float *ms_out, void *stream) {
    if (!g || !m || !x || !e || !ms_out || d <= 0 || d % 4 != 0 || n <= 0 || reps <= 0) return -1;
    if ((((uintptr_t)g | (uintptr_t)m | (uintptr_t)x | (uintptr_t)e) & 15) != 0) return -1;
    cudaStream_t s = (cudaStream_t)stream;
    ProbeParams P = {};
    P.g = g, P.m = m, P.x = x, P.e = e, P.d = d, P.cols = d / 4, P.n = n, P.eta = 0.1f, P.beta = 0.9f, P.never = 1.2345e38f;
    P.tiles = (unsigned)((P.cols + 255) / 256);
    const unsigned long long row_grid = (unsigned long long)P.tiles * n;
    if (row_grid > 0x7fffffffull) return -1;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    size_t smem = 0;
    if (pattern == 5) {
        if (variant < 2 || variant > 16) return -1;
        P.tile_cols = (unsigned)variant * 1024 / 16;
        P.stages = (96u * 1024) / (4u * (unsigned)variant * 1024);
        if (P.stages > 8) P.stages = 8;
        if (P.stages < 2) return -1;
        smem = 128 + (size_t)P.stages * 4 * P.tile_cols * 16;
        if (cudaFuncSetAttribute(staged_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return -3;
    }
    auto launch = [&]() {
        switch (pattern) {
            case 0: rows_kernel<0><<<(unsigned)row_grid, 256, 0, s>>>(P); break;
            case 1: rows_kernel<1><<<(unsigned)row_grid, 256, 0, s>>>(P); break;
            case 2: rows_kernel<2><<<(unsigned)row_grid, 256, 0, s>>>(P); break;
            case 3: rows_kernel<3><<<(unsigned)row_grid, 256, 0, s>>>(P); break;
            case 4: {
                const unsigned grid = (unsigned)((P.cols + 255) / 256);
                if (variant == 1) column_walk_kernel<1><<<grid, 256, 0, s>>>(P);
                else if (variant == 2) column_walk_kernel<2><<<grid, 256, 0, s>>>(P);
                else if (variant == 4) column_walk_kernel<4><<<grid, 256, 0, s>>>(P);
                else column_walk_kernel<8><<<grid, 256, 0, s>>>(P);
                break;
            }
            default: staged_rows_kernel<<<2 * sms, kStagedConsumers + 32, smem, s>>>(P); break;
        }
    };
    if (pattern < 0 || pattern > 5) return -1;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return -3;
    for (int k = 0; k < 3; ++k) launch();
    cudaEventRecord(e0, s);
    for (int k = 0; k < reps; ++k) launch();
    cudaEventRecord(e1, s);
    cudaError_t er = cudaStreamSynchronize(s);
    float ms = 0.f;
    if (er == cudaSuccess) er = cudaEventElapsedTime(&ms, e0, e1);
    if (er == cudaSuccess) er = cudaGetLastError();
    cudaEventDestroy(e0), cudaEventDestroy(e1);
    if (er != cudaSuccess) return -3;
    *ms_out = ms / (float)reps;
    return 0;
}
