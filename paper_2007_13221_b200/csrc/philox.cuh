// philox.cuh - Philox4x32-10 counter-based generator (word 0 only)
// Device code of the CSER step library; included by cser.cu inside its unnamed namespace.
#pragma once
// ------------------------------------------------------------------ Philox4x32-10
// Salmon et al., SC'11.  Ten rounds; key bumped by the Weyl constants each round.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t k0, uint32_t k1, uint32_t c0,
                                                        uint32_t c1, uint32_t c2, uint32_t c3) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += W0;
        k1 += W1;
    }
    return c0;
}

