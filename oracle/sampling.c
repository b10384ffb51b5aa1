/*
 * CPU oracle, part 3: random numbers for sampling verification at
 * temperature > 0 (Section 4, "sample matching"; Appendix "Impact of
 * Sampling").
 *
 * TEST INFRASTRUCTURE ONLY.  Shares no code, header, table or constant with
 * the CUDA library and must never be called from the product path.
 *
 * What it computes.  With sampling, the base model's token at an output
 * position is a draw from softmax(logits / T), and a drafted token is accepted
 * only if it equals that draw.  The paper names no sampler.  The reading taken
 * here: the draw at absolute position t is
 *
 *     y_t = argmax_v ( logits[v] / T + g(seed, t, v) ),   ties to the lower v,
 *
 * with g i.i.d. standard Gumbel noise (the Gumbel-max form of a categorical
 * draw).  Because the noise is a pure function of (seed, position, token), a
 * row of a draft tree that sits at position t-1 draws exactly the token plain
 * autoregressive sampling draws at t: tree verification stays lossless token
 * by token, not only in distribution.
 *
 * The noise: Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random
 * numbers: as easy as 1, 2, 3", SC'11) with counter (v, t, 0, 0) and key
 * (seed_lo, seed_hi); the top 23 bits n of output word 0 give the uniform
 * u = (2n + 1) / 2^24 in (0, 1), exact in fp32; g = -log(-log(u)).
 *
 * The logarithm is written out in single IEEE fp32 operations (add, multiply,
 * divide, fused multiply-add; the build disables contraction), so that it has
 * one value everywhere: log(x) = e ln2 + 2 atanh(z), z = (m-1)/(m+1), x = m 2^e
 * with m in [sqrt(1/2), sqrt(2)), atanh by its odd power series to z^9.
 */
#include <math.h>
#include <stdint.h>

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {              /* the key is bumped between rounds */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* log(x) for a positive normal fp32 x, every step one rounded fp32 operation */
float orc_det_logf(float x) {
    union { float f; uint32_t u; } b;
    b.f = x;
    int e = (int)((b.u >> 23) & 255u) - 126;          /* x = m 2^e, m in [1/2, 1) */
    b.u = (b.u & 0x007fffffu) | 0x3f000000u;
    float m = b.f;
    if (m < 0.70710678118654752f) { m = m * 2.0f; e -= 1; }   /* exact */
    const float z = (m - 1.0f) / (m + 1.0f);
    const float w = z * z;
    float p = fmaf(w, 1.0f / 9.0f, 1.0f / 7.0f);
    p = fmaf(w, p, 1.0f / 5.0f);
    p = fmaf(w, p, 1.0f / 3.0f);
    const float s = fmaf(z * w, p, z);                 /* atanh(z) */
    return fmaf((float)e, 0.69314718055994531f, s + s);
}

float orc_uniform_from_bits(uint32_t x) {
    const uint32_t n = x >> 9;
    return (float)(2u * n + 1u) * (1.0f / 16777216.0f);
}

float orc_gumbel_from_bits(uint32_t x) {
    const float u = orc_uniform_from_bits(x);
    const float t = -orc_det_logf(u);
    return -orc_det_logf(t);
}

/* out[v] = g(seed, position, v) for v = 0..n_vocab-1 */
void orc_gumbel_noise(uint32_t seed_lo, uint32_t seed_hi, uint32_t position, int32_t n_vocab, float* out) {
    const uint32_t key[2] = {seed_lo, seed_hi};
    for (int32_t v = 0; v < n_vocab; ++v) {
        const uint32_t ctr[4] = {(uint32_t)v, position, 0u, 0u};
        uint32_t r[4];
        orc_philox4x32_10(ctr, key, r);
        out[v] = orc_gumbel_from_bits(r[0]);
    }
}
