// staged_kernel.cuh - the selected-block kernel, staged through shared memory with bulk copies.
// Device code of the CSER step library; included by cser.cu inside its unnamed namespace.
#pragma once
#include "bulk_copy.cuh"
#include "step_kernels.cuh"

// Blocks selected by a mask need the mean over workers (Algorithm 3 line 7; Algorithm 2 line 11), so
// for them every worker's row segment of g, x, m (and e, when the block is reset) has to be on the SM
// at once.  Holding them in registers limits a thread to a few loads in flight and makes the kernel
// wait on latency.  Here the segments are brought into shared memory by the copy engine instead: a
// work unit is one chunk of C <= 128 vector columns of one listed block; a producer warp issues, for
// all n workers and every array the unit needs, one contiguous bulk copy of C * 16 bytes each (n * 3
// or n * 4 copies, tens of KB, in flight without holding a register), S units ahead of the consumers.
// The consumer threads work on a unit in three phases:
//   A  Get_p (Appendix A.4), elementwise over (worker, column): thread (part h, column c) takes the
//      workers i = h, h + kStagedSplit, ...; m goes to global memory, p_i replaces g_i in the stage;
//   B  the sums over workers in the fixed ascending order, read back from the stage, by every thread
//      for its own column (the kStagedSplit threads of a column redo the same few additions);
//   C  the update of x (and e), elementwise again, written straight to global memory, once.
// The arithmetic and its order are those of the register-walking kernel, so results are bit-identical.
//
// Synchronisation: two rings of shared-memory barriers (full[s]: the unit's bytes have landed;
// empty[s]: the consumer warps are done with stage s) and one named barrier among the consumers.
// Every wait on a shared-memory barrier is bounded: a wait that runs out raises P.err_word
// (host-visible) and the threads leave - the consumers all together, after a vote, so that none is
// left behind at the named barrier.  Nothing in here can spin for ever.
#ifndef CSER_STAGED_SPLIT
#define CSER_STAGED_SPLIT 2
#endif
constexpr int kStagedSplit = CSER_STAGED_SPLIT;             // consumer threads per vector column
constexpr int kStagedColThreads = 128;                      // columns of a unit, at most
constexpr int kStagedConsumers = kStagedColThreads * kStagedSplit;
constexpr int kStagedConsumerWarps = kStagedConsumers / 32;
constexpr int kStagedThreads = kStagedConsumers + 32;      // + the producer warp
constexpr int kStagedMaxStages = 8;
constexpr int kStagedCtlBytes = 256;                        // barriers + unit descriptors, before the stages
#ifndef CSER_STAGE_KB
#define CSER_STAGE_KB 54
#define CSER_CTA_KB 112
#define CSER_STAGED_CTAS_PER_SM 2
#endif
constexpr unsigned kStagedStageBudget = (unsigned)(CSER_STAGE_KB) << 10;   // bytes of one stage, at most
constexpr unsigned kStagedCtaBudget = (unsigned)(CSER_CTA_KB) << 10;       // dynamic shared memory of one CTA
constexpr unsigned kStagedCtasPerSm = CSER_STAGED_CTAS_PER_SM;
constexpr unsigned kStagedMinChunkCols = 16;               // copies of at least 256 bytes
constexpr unsigned kStagedMaxChunkCols = kStagedColThreads;

struct StagedUnit {
    long long c0;        // first vector column
    uint32_t cols;       // vector columns in this unit (0: nothing to do)
    uint32_t flags;      // bit 0: update-selected, bit 1: reset-selected
};

struct StagedCtl {
    uint64_t full[kStagedMaxStages];
    uint64_t empty[kStagedMaxStages];
    StagedUnit unit[kStagedMaxStages];
};
static_assert(sizeof(StagedCtl) <= kStagedCtlBytes, "control block");

__device__ __forceinline__ Pack<4> pack_of(const float4 t) {
    Pack<4> r;
    r.v[0] = t.x, r.v[1] = t.y, r.v[2] = t.z, r.v[3] = t.w;
    return r;
}

__device__ __forceinline__ void staged_fail(const StepParams &P, unsigned where) {
    if (P.err_word) {
        *reinterpret_cast<volatile unsigned *>(P.err_word) = 0x80000000u | where;
        __threadfence_system();
    }
}

__device__ __forceinline__ float4 f4_of(const Pack<4> &a) { return make_float4(a.v[0], a.v[1], a.v[2], a.v[3]); }

// All consumer threads of the CTA (named barrier 1; barrier 0 is __syncthreads').
__device__ __forceinline__ void consumers_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(kStagedConsumers) : "memory");
}
// The same barrier, and whether `ok` holds on every consumer thread.
__device__ __forceinline__ bool consumers_all(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)ok), "n"(kStagedConsumers)
        : "memory");
    return r != 0;
}

// DENSE = false: units are laid over the listed blocks.  DENSE = true: over all blocks of the range
// in their natural order, a block that no mask selects costing one empty unit (used when a large
// share of the blocks is selected).
template <bool MOM, bool RESET, bool ERR, bool DENSE>
__global__ void __launch_bounds__(kStagedThreads) cser_selected_staged_kernel(const StepParams P) {
    extern __shared__ __align__(128) unsigned char staged_smem[];
    StagedCtl *ctl = reinterpret_cast<StagedCtl *>(staged_smem);
    unsigned char *stage0 = staged_smem + kStagedCtlBytes;
    constexpr unsigned NA = 2u + (MOM ? 1u : 0u) + ((RESET && ERR) ? 1u : 0u);
    const unsigned C = P.chunk_cols, S = P.stages;
    const unsigned n = (unsigned)P.n;
    const size_t stage_bytes = (size_t)NA * n * C * 16u;
    const unsigned warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long wait_cycles = (long long)P.wait_mcycles * 1000000ll;

    if (threadIdx.x == 0) {
        for (unsigned s = 0; s < S; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kStagedConsumerWarps);
        }
        mbar_init_fence();
    }
    __syncthreads();

    const bool reset_on = RESET && (P.rctl ? P.rctl->c[0].reset != 0 : true);
    const unsigned first_blk = DENSE ? (unsigned)((unsigned long long)P.c_begin / P.bsv) : 0u;
    unsigned long long n_entries;
    if constexpr (DENSE) {
        n_entries = (P.c_end > P.c_begin) ? ((unsigned long long)(P.c_end - 1) / P.bsv - first_blk + 1ull) : 0ull;
    } else {
        const uint32_t cnt = P.rctl ? P.rctl->c[0].count : *P.count;
        n_entries = cnt < P.list_cap ? cnt : P.list_cap;
    }
    const unsigned long long total = n_entries * P.n_chunks;
    const unsigned long long n_my =
        total > blockIdx.x ? (total - blockIdx.x + gridDim.x - 1ull) / gridDim.x : 0ull;

    if (warp == kStagedConsumerWarps) {
        // ---------------------------------------------------------------- producer warp
        const uint64_t pol_g = l2_policy_evict_first();     // gradients are read exactly once
        const uint64_t pol_s = l2_policy_normal();
        unsigned long long k = 0;
        bool ok = true;
        for (; k < n_my; ++k) {
            const unsigned s = (unsigned)(k % S);
            const unsigned round = (unsigned)(k / S);
            // the unit's block and mask bits are fetched before the wait, so that their latency is
            // hidden behind it
            const unsigned long long u = blockIdx.x + k * gridDim.x;
            const unsigned long long entry = u / P.n_chunks;
            const unsigned chunk = (unsigned)(u - entry * P.n_chunks);
            const unsigned blk = DENSE ? first_blk + (unsigned)entry : P.list[entry];
            const bool sg = P.mask_g[blk] != 0;
            const bool sr = reset_on ? (P.mask_r[blk] != 0) : false;
            if (round > 0 && !mbar_wait_bounded(&ctl->empty[s], (round - 1) & 1u, wait_cycles)) {
                ok = false;
                break;
            }
            long long lo = (long long)blk * P.bsv + (long long)chunk * C;
            long long hi = lo + C;
            const long long blk_end = ((long long)blk + 1) * P.bsv;
            if (hi > blk_end) hi = blk_end;
            if (hi > P.c_end) hi = P.c_end;
            if (hi > P.cols_total) hi = P.cols_total;
            if (lo < P.c_begin) lo = P.c_begin;
            const uint32_t cols = (hi > lo && (sg || sr)) ? (uint32_t)(hi - lo) : 0u;
            const bool with_e = RESET && ERR && sr;
            const unsigned n_arr = 2u + (MOM ? 1u : 0u) + (with_e ? 1u : 0u);
            if (lane == 0) {
                ctl->unit[s].c0 = lo;
                ctl->unit[s].cols = cols;
                ctl->unit[s].flags = (sg ? 1u : 0u) | (sr ? 2u : 0u);
                // (test hook: bytes that never arrive make this unit's wait run out)
                const uint32_t phantom = (P.test_stall && blockIdx.x == 0 && k == 0) ? 16u : 0u;
                if (cols) mbar_arrive_expect(&ctl->full[s], n_arr * n * cols * 16u + phantom);
                else      mbar_arrive(&ctl->full[s]);
            }
            __syncwarp();
            if (cols) {
                unsigned char *stage = stage0 + (size_t)s * stage_bytes;
                const uint32_t bytes = cols * 16u;
                for (unsigned j = lane; j < n_arr * n; j += 32) {
                    const unsigned a = j / n, i = j - a * n;
                    // array order in a stage: g, x, m, e (m only with momentum)
                    const float *src;
                    unsigned slot;
                    if (a == 0) src = P.g, slot = 0;
                    else if (a == 1) src = P.x, slot = 1;
                    else if (MOM && a == 2) src = P.m, slot = 2;
                    else src = P.e, slot = 2u + (MOM ? 1u : 0u);
                    bulk_load(stage + ((size_t)slot * n + i) * C * 16u, src + (long long)i * P.d + lo * 4, bytes,
                              &ctl->full[s], a == 0 ? pol_g : pol_s);
                }
            }
        }
        if (!ok) {
            staged_fail(P, 1u);
            // give the copies already issued a bounded time to land before the CTA's memory goes away
            const unsigned long long from = k > S ? k - S : 0ull;
            for (unsigned long long j = from; j < k; ++j)
                mbar_wait_bounded(&ctl->full[j % S], (unsigned)(j / S) & 1u, wait_cycles / 64);
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    const unsigned col = threadIdx.x & (kStagedColThreads - 1);       // my column of the unit
    const unsigned part = threadIdx.x / kStagedColThreads;             // my share of the workers
    const size_t arr = (size_t)n * C;                                  // float4 per array in a stage
    const float eta = P.eta, beta = P.beta, n_f = P.n_f;
    const long long d = P.d;
    Pack<4> zero;
#pragma unroll
    for (int q = 0; q < 4; ++q) zero.v[q] = 0.f;
    for (unsigned long long k = 0; k < n_my; ++k) {
        const unsigned s = (unsigned)(k % S);
        const bool landed = mbar_wait_bounded(&ctl->full[s], (unsigned)(k / S) & 1u, wait_cycles);
        if (!consumers_all(landed)) {
            if (!landed) staged_fail(P, 2u);
            return;
        }
        const long long c0 = ctl->unit[s].c0;
        const uint32_t cols = ctl->unit[s].cols;
        const uint32_t flags = ctl->unit[s].flags;
        const bool sg = (flags & 1u) != 0, sr = RESET && (flags & 2u) != 0;
        const bool mine = col < cols;
        float4 *sG = reinterpret_cast<float4 *>(stage0 + (size_t)s * stage_bytes) + col;   // g, then p
        const float4 *sX = sG + arr;
        const float4 *sM = sG + 2 * arr;
        const float4 *sE = sG + (2 + (MOM ? 1 : 0)) * arr;
        const long long gcol = (c0 + col) * 4;
        if (mine) {
            // A: p_i for my workers; m_i to global memory; p_i over g_i in the stage
            float *m = MOM ? P.m + gcol : nullptr;
            for (unsigned i = part; i < n; i += kStagedSplit) {
                const Pack<4> gv = pack_of(sG[(size_t)i * C]);
                Pack<4> mv = zero;
                if constexpr (MOM) mv = pack_of(sM[(size_t)i * C]);
                const Pack<4> p = get_p<4, MOM>(gv, mv, eta, beta);
                if constexpr (MOM) st<4>(m + (long long)i * d, mv);
                sG[(size_t)i * C] = f4_of(p);
            }
        }
        // the stage is written by the copy engine next: order these plain writes before that
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        consumers_sync();
        if (mine) {
            // B: sums over all workers, ascending, starting from worker 0's value
            Pack<4> pbar = zero, rbar = zero;
            if (sg) {
                Pack<4> sum = zero;
                for (unsigned i = 0; i < n; ++i) {
                    const Pack<4> p = pack_of(sG[(size_t)i * C]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) sum.v[q] = (i == 0) ? p.v[q] : sum.v[q] + p.v[q];
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) pbar.v[q] = sum.v[q] / n_f;
            }
            if constexpr (RESET) {
                if (sr) {
                    // with an error array: sum of e_{t-1/2}; without one (Appendix A.4,
                    // implementation II): sum of x_{t-1/2}.  On an update-selected block the residual
                    // is zero (e unchanged, x moved by p-bar); else it is p_i.
                    Pack<4> sum = zero;
                    for (unsigned i = 0; i < n; ++i) {
                        const Pack<4> v = pack_of(ERR ? sE[(size_t)i * C] : sX[(size_t)i * C]);
                        Pack<4> sub = zero;
                        if (!sg) sub = pack_of(sG[(size_t)i * C]);
                        else if (!ERR) sub = pbar;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float t = (sg && ERR) ? v.v[q] : v.v[q] - sub.v[q];
                            sum.v[q] = (i == 0) ? t : sum.v[q] + t;
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) rbar.v[q] = sum.v[q] / n_f;
                }
            }
            // C: x (and e) of my workers
            float *x = P.x + gcol;
            float *e = ERR ? P.e + gcol : nullptr;
            for (unsigned i = part; i < n; i += kStagedSplit) {
                Pack<4> xv;
                if (!sr) {
                    // Algorithm 3 on a selected block: x_i -= mean_k p_k, e untouched
                    xv = pack_of(sX[(size_t)i * C]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) xv.v[q] = xv.v[q] - pbar.v[q];
                } else if constexpr (RESET && ERR) {
                    // Algorithm 2 lines 11-12: x_i = (x_{t-1/2} - e_{t-1/2}) + mean_k e_{k,t-1/2}; e_i = 0
                    xv = pack_of(sX[(size_t)i * C]);
                    const Pack<4> ev = pack_of(sE[(size_t)i * C]);
                    Pack<4> p = zero;
                    if (!sg) p = pack_of(sG[(size_t)i * C]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float xh = xv.v[q] - (sg ? pbar.v[q] : p.v[q]);
                        const float eh = sg ? ev.v[q] : ev.v[q] - p.v[q];
                        xv.v[q] = (xh - eh) + rbar.v[q];
                    }
                    st<4>(e + (long long)i * d, zero);
                } else {
                    xv = rbar;       // implementation II: x_i = mean_k x_{k,t-1/2}
                }
                st<4>(x + (long long)i * d, xv);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[s]);
    }
}
