// Sampled token (Section 3.1: y_t is "sampled" from p_t): y_t ~ softmax(z / T_s) by the Gumbel-max
// construction, tok = argmax_v (z_v / T_s - ln(-ln U_v)), with U_v from the counter-based generator
// Philox-4x32-10 (Salmon et al., SC'11) so that no random numbers have to be stored or passed:
// U of (row, draw, v) is word (v mod 4) of Philox(counter = (v div 4, row, draw_lo, draw_hi),
// key = (seed_lo, seed_hi)), mapped to ((x >> 9) + 1/2) / 2^23 -- an odd multiple of 2^-24, exact
// in fp32 and strictly inside (0, 1).  Device side only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace rstitch {

struct SampleArgs {
    int      on;          // 0: greedy token
    float    inv_t;       // 1 / T_s
    uint32_t k0, k1;      // seed
    uint32_t d0, d1;      // draw number
    uint32_t v0;          // index of this head's first vocabulary entry in the whole vocabulary
                          // (non-zero for a vocabulary shard: the noise of an entry does not depend on the split)
};

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Standard Gumbel noise -ln(-ln U) of one 32-bit output word.  The draw is decided by the largest
// noise values, whose U sit within ~1/V of 1, so -ln U is taken from the series of 2 atanh(w / (2 - w))
// with w = 1 - U (exact) when U > 1/2; the fast logarithm's absolute error would be a few percent of
// -ln U there.  Elsewhere the fast logarithm's absolute error (~2e-7) is harmless.
__device__ __forceinline__ float gumbel_from_bits(uint32_t x)
{
    const float u = ((float)(x >> 9) + 0.5f) * (1.0f / 8388608.0f);
    float t;
    if (u > 0.5f) {
        const float w = 1.0f - u;
        const float y = __fdividef(w, 2.0f - w);                 // in (0, 1/3]
        const float y2 = y * y;
        float p = fmaf(y2, 1.0f / 17.0f, 1.0f / 15.0f);
        p = fmaf(p, y2, 1.0f / 13.0f);
        p = fmaf(p, y2, 1.0f / 11.0f);
        p = fmaf(p, y2, 1.0f / 9.0f);
        p = fmaf(p, y2, 1.0f / 7.0f);
        p = fmaf(p, y2, 1.0f / 5.0f);
        p = fmaf(p, y2, 1.0f / 3.0f);
        p = fmaf(p, y2, 1.0f);
        t = 2.0f * y * p;
    } else {
        t = -log_approx(u);
    }
    return -log_approx(t);
}

// Score of vocabulary entry v (any v): one generator call per entry.
__device__ __forceinline__ float sample_score(const SampleArgs &sa, float z, uint32_t row, uint32_t v)
{
    uint32_t o[4];
    v += sa.v0;
    philox4x32_10(v >> 2, row, sa.d0, sa.d1, sa.k0, sa.k1, o);
    const uint32_t x = (v & 2u) ? ((v & 1u) ? o[3] : o[2]) : ((v & 1u) ? o[1] : o[0]);
    return fmaf(z, sa.inv_t, gumbel_from_bits(x));
}

}  // namespace rstitch
