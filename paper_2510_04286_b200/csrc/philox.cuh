// Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3", SC'11), the
// counter-based generator behind the library's random draws: every draw is a pure function of
// (key, counter), so results do not depend on the launch shape.
#pragma once
#include <stdint.h>

namespace slicemoe {

// out = Philox4x32-10(counter = (c0, c1, c2, c3), key = (k0, k1)).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4]) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
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
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Figure 6's logit noise eps(n, e), a standard normal per (row, expert): Philox words x0, x1 of counter
// (n, e, 1, 0), u_i = ((x_i >> 8) + 0.5) / 2^24 in (0, 1) (both exact in fp32), Box-Muller.
__device__ __forceinline__ float logit_noise(int n, int e, uint32_t key0, uint32_t key1) {
    uint32_t x[4];
    philox4x32_10((uint32_t)n, (uint32_t)e, 1u, 0u, key0, key1, x);
    const float u0 = ((float)(x[0] >> 8) + 0.5f) * (1.0f / 16777216.0f);
    const float u1 = ((float)(x[1] >> 8) + 0.5f) * (1.0f / 16777216.0f);
    return sqrtf(-2.0f * logf(u0)) * cospif(2.0f * u1);
}

}  // namespace slicemoe
