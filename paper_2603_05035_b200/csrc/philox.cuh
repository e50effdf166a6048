// Device-side Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel Random Numbers:
// As Easy as 1, 2, 3", SC'11) and the Box-Muller transform used for the mixing
// matrix and the shield rows.
#pragma once
#include <stdint.h>

namespace gelo {

// Block q of the stream (seed, stream_id, attempt): counter (lo32 q, hi32 q, stream_id,
// attempt), key (lo32 seed, hi32 seed), ten rounds.
__device__ __forceinline__ void philox_block(uint64_t seed, uint64_t q, uint32_t stream_id,
                                             uint32_t attempt, uint32_t w[4])
{
    uint32_t c0 = (uint32_t)q, c1 = (uint32_t)(q >> 32), c2 = stream_id, c3 = attempt;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    w[0] = c0; w[1] = c1; w[2] = c2; w[3] = c3;
}

// u = ((w >> 9) + 1/2) / 2^23: 23-bit uniform in (0,1), exact in binary32.
__device__ __forceinline__ float uniform_open(uint32_t w)
{
    return ((float)(w >> 9) + 0.5f) * (1.0f / 8388608.0f);
}

// Four standard normals of block q: words (0,1) and (2,3) are Box-Muller pairs
// (u_a, u_b) -> (r cos 2 pi u_b, r sin 2 pi u_b), r = sqrt(-2 ln u_a).
__device__ __forceinline__ void gaussian_block(uint64_t seed, uint64_t q, uint32_t stream_id,
                                               uint32_t attempt, float z[4])
{
    uint32_t w[4];
    philox_block(seed, q, stream_id, attempt, w);
#pragma unroll
    for (int pair = 0; pair < 2; ++pair) {
        const float ua = uniform_open(w[2 * pair]);
        const float ub = uniform_open(w[2 * pair + 1]);
        const float r = sqrtf(-2.0f * logf(ua));
        float s, c;
        sincospif(2.0f * ub, &s, &c);
        z[2 * pair] = r * c;
        z[2 * pair + 1] = r * s;
    }
}

}  // namespace gelo
