// Noise for sample matching (Section 4: a drafted token is accepted only if it equals the token the base
// model samples).  The model's draw at absolute position t is argmax_v(logit_v / T + g(seed, t, v)) with g
// standard Gumbel noise -- a draw from softmax(logits / T) -- and g is a pure function of its arguments, so a
// tree row at position t-1 draws the token plain autoregressive sampling draws at t, whatever else is in the
// block.
//
// g = -log(-log(u)), u = (2n + 1) / 2^24 with n the top 23 bits of word 0 of Philox4x32-10 (Salmon et al.,
// SC'11) on counter (v, t, 0, 0) and key (seed_lo, seed_hi).  The logarithm is spelled out in individually
// rounded fp32 operations (no contraction, no approximate intrinsics), so the noise has the same bits on any
// IEEE machine: log(x) = e ln2 + 2 atanh(z), z = (m-1)/(m+1), x = m 2^e, m in [sqrt(1/2), sqrt(2)).
#pragma once

#include <stdint.h>

namespace esp {

__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        const uint32_t t0 = hi1 ^ c1 ^ k0, t2 = hi0 ^ c3 ^ k1;
        c0 = t0; c1 = lo1; c2 = t2; c3 = lo0;
        k0 += W0; k1 += W1;     // the bump after the last round is never used
    }
    return c0;
}

// natural logarithm of a positive normal number
__device__ __forceinline__ float log_rounded_steps(float x) {
    const uint32_t bits = __float_as_uint(x);
    int e = (int)((bits >> 23) & 255u) - 126;
    float m = __uint_as_float((bits & 0x007fffffu) | 0x3f000000u);     // [1/2, 1)
    if (m < 0.70710678118654752f) { m = __fmul_rn(m, 2.0f); e -= 1; }
    const float z = __fdiv_rn(__fsub_rn(m, 1.0f), __fadd_rn(m, 1.0f));
    const float w = __fmul_rn(z, z);
    float p = __fmaf_rn(w, 1.0f / 9.0f, 1.0f / 7.0f);
    p = __fmaf_rn(w, p, 1.0f / 5.0f);
    p = __fmaf_rn(w, p, 1.0f / 3.0f);
    const float s = __fmaf_rn(__fmul_rn(z, w), p, z);
    return __fmaf_rn((float)e, 0.69314718055994531f, __fadd_rn(s, s));
}

__device__ __forceinline__ float gumbel_noise(uint32_t key0, uint32_t key1, uint32_t position, uint32_t token) {
    const uint32_t x = philox4x32_10_word0(token, position, 0u, 0u, key0, key1);
    const float u = __fmul_rn((float)(2u * (x >> 9) + 1u), 1.0f / 16777216.0f);
    const float t = -log_rounded_steps(u);
    return -log_rounded_steps(t);
}

// the score whose arg-max over the vocabulary is the draw
__device__ __forceinline__ float sample_score(float logit, float inv_temp, float g) {
    return __fadd_rn(__fmul_rn(logit, inv_temp), g);
}

}  // namespace esp
