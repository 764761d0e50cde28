// Test helper (not part of the product): returns what cuRAND's device-API Philox4_32_10
// generator produces, so the tests can compare an independent library implementation of
// Philox4x32-10 with the oracle's.  Build: see __graft_entry__.build().
#include <cuda_runtime.h>
#include <curand_kernel.h>
#include <stdint.h>

__global__ void curand_philox_kernel(const unsigned long long *seed, const unsigned long long *subseq,
                                     const unsigned long long *offset, uint32_t *out, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    curandStatePhilox4_32_10_t st;
    curand_init(seed[i], subseq[i], offset[i], &st);
    const uint4 r = curand4(&st);
    out[4 * i + 0] = r.x, out[4 * i + 1] = r.y, out[4 * i + 2] = r.z, out[4 * i + 3] = r.w;
}

// All pointers are device memory: seed/subseq/offset [n] uint64, out [4n] uint32.
extern "C" int curand_philox_words(const unsigned long long *seed, const unsigned long long *subseq,
                                   const unsigned long long *offset, uint32_t *out, int n, void *stream) {
    if (n <= 0) return 0;
    curand_philox_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(seed, subseq, offset, out, n);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}
