// Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11),
// device side.  Ten rounds of: two 32x32->64 multiplies by fixed odd constants,
// a word permutation with the key xor-ed in, and a Weyl key schedule.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace ears {

struct U32x4 { uint32_t w0, w1, w2, w3; };

__device__ __forceinline__ U32x4 philox4x32_10(U32x4 ctr, uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(M0, ctr.w0), lo0 = M0 * ctr.w0;
        uint32_t hi1 = __umulhi(M1, ctr.w2), lo1 = M1 * ctr.w2;
        U32x4 n;
        n.w0 = hi1 ^ ctr.w1 ^ k0;
        n.w1 = lo1;
        n.w2 = hi0 ^ ctr.w3 ^ k1;
        n.w3 = lo0;
        ctr = n;
        k0 += W0;
        k1 += W1;
    }
    return ctr;
}

// counter = (offset lo, offset hi, global sequence index, slot); key = seed.
__device__ __forceinline__ U32x4 draw_words(uint64_t seed, uint64_t offset, uint32_t b_global, uint32_t slot) {
    U32x4 c{static_cast<uint32_t>(offset), static_cast<uint32_t>(offset >> 32), b_global, slot};
    return philox4x32_10(c, static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
}

// Accept uniform of position k: 24 bits, exact in fp32 and fp64.
__device__ __forceinline__ double uniform_accept(uint64_t seed, uint64_t offset, uint32_t b_global, uint32_t k) {
    return static_cast<double>(draw_words(seed, offset, b_global, k).w0 >> 8) * (1.0 / 16777216.0);
}

// Final-token uniform (slot K): 53 bits.
__device__ __forceinline__ double uniform_final(uint64_t seed, uint64_t offset, uint32_t b_global, uint32_t K) {
    U32x4 w = draw_words(seed, offset, b_global, K);
    uint64_t bits = ((static_cast<uint64_t>(w.w0) << 32) | w.w1) >> 11;
    return static_cast<double>(bits) * (1.0 / 9007199254740992.0);
}

}  // namespace ears
