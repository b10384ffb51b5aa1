// What follows each split GEMM in the decoder layer, as device functions: the sum of the stream-K partials
// in CTA order fused with
//   * the residual add and the next RMSNorm                      (after the O and the down projection),
//   * per-head RMSNorm (Qwen3), rotary embedding at the row's position, q to the query buffer and k, v to
//     the cache                                                   (after the QKV projection),
//   * SiLU(gate) * up                                             (after the gate/up projection).
// The kernels that run one operation per launch and the kernel that runs all layers in one launch call the
// same functions, and every product and sum whose grouping a compiler could choose is spelled out as an
// individually rounded operation: both give the same bits.
#pragma once

#include "esp_common.cuh"

namespace esp {

// An activation that feeds a two-plane GEMM is stored as hi = bf16(x) and lo = bf16(x - hi): hi + lo carries x to
// about 2^-17, and the tensor cores take the product with both.
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(__fsub_rn(x, __bfloat162float(hi)));
}

// ------------------------------------------------------------------ residual add + RMSNorm of one row
// The row is cut into groups of 128 features (= GEMM tiles).  A warp owns a group at a time, lane l the
// features 128*group + 4*l .. +3.  Sum of squares: per lane x0^2 + x1^2 + x2^2 + x3^2 (fused multiply-adds in
// that order), butterfly over the warp, groups added in ascending order.
template <typename T>
struct NormFirst {   // what a warp may fetch for its first group before the partials exist
    SkEntry en;
    T g[4];
};

template <typename T>
__device__ __forceinline__ void load4(T (&o)[4], const T* p) {
    if constexpr (sizeof(T) == 2) *reinterpret_cast<uint2*>(o) = __ldg(reinterpret_cast<const uint2*>(p));
    else *reinterpret_cast<float4*>(o) = __ldg(reinterpret_cast<const float4*>(p));
}

template <typename T>
__device__ __forceinline__ void norm_prefetch(NormFirst<T>& pf, const StreamK& sk, const T* g, int d, int warp, int lane) {
    const int j = warp * TILE_N + lane * 4;
    if (j < d) {
        if (sk.partials) pf.en = sk_entry(sk, warp);
        load4(pf.g, g + j);
    }
}

// hres[row] += partial sums (sk.partials != NULL);  y = hres[row] * rsqrt(mean(hres[row]^2) + eps) * g.
// NW warps cooperate; `red` is shared memory for (d + 127) / 128 floats; bar() synchronises those warps.
// yr_lo (bf16 only, may be NULL): the row of the low-order plane of y.
template <typename T, int NW, typename Bar>
__device__ __forceinline__ void resid_norm_row(float* xr, const StreamK& sk, int sk_row, const T* g, T* yr, T* yr_lo, int d, float eps,
                                               float* copy_row, float* red, const NormFirst<T>& pf, int warp, int lane, Bar bar) {
    const int ng = (d + TILE_N - 1) / TILE_N;
    constexpr int KEEP = 3;
    float4 keep[KEEP];
    int it = 0;
    for (int gi = warp; gi < ng; gi += NW, ++it) {
        const int j = gi * TILE_N + lane * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < d) {
            x = __ldcg(reinterpret_cast<const float4*>(xr + j));
            if (sk.partials) {
                const float4 acc = it == 0 ? sk_sum4(sk, pf.en, sk_row, lane * 4) : sk_sum4(sk, gi, sk_row, lane * 4);
                x.x = __fadd_rn(x.x, acc.x); x.y = __fadd_rn(x.y, acc.y); x.z = __fadd_rn(x.z, acc.z); x.w = __fadd_rn(x.w, acc.w);
                __stcg(reinterpret_cast<float4*>(xr + j), x);
            }
        }
        if (it < KEEP) keep[it] = x;
        float ss = __fmaf_rn(x.w, x.w, __fmaf_rn(x.z, x.z, __fmaf_rn(x.y, x.y, __fmul_rn(x.x, x.x))));
        ss = warp_sum(ss);
        if (lane == 0) red[gi] = ss;
    }
    bar();
    float tot = 0.f;
    for (int gi = 0; gi < ng; ++gi) tot = __fadd_rn(tot, red[gi]);
    const float rinv = 1.0f / sqrtf(__fadd_rn(tot / (float)d, eps));
    it = 0;
    for (int gi = warp; gi < ng; gi += NW, ++it) {
        const int j = gi * TILE_N + lane * 4;
        if (j >= d) continue;
        const float4 x = it < KEEP ? keep[it] : __ldcg(reinterpret_cast<const float4*>(xr + j));   // beyond: this thread's own writes
        const float xv[4] = {x.x, x.y, x.z, x.w};
        T gg[4];
        if (it == 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) gg[i] = pf.g[i];
        } else {
            load4(gg, g + j);
        }
        T o[4];
        if constexpr (sizeof(T) == 2) {
            T ol[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) split_bf16(__fmul_rn(__fmul_rn(xv[i], rinv), to_f32(gg[i])), o[i], ol[i]);
            *reinterpret_cast<uint2*>(yr + j) = *reinterpret_cast<const uint2*>(o);
            if (yr_lo) *reinterpret_cast<uint2*>(yr_lo + j) = *reinterpret_cast<const uint2*>(ol);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) o[i] = from_f32<T>(__fmul_rn(__fmul_rn(xv[i], rinv), to_f32(gg[i])));
            *reinterpret_cast<float4*>(yr + j) = *reinterpret_cast<const float4*>(o);
        }
        if (copy_row) *reinterpret_cast<float4*>(copy_row + j) = x;
    }
}

// ------------------------------------------------------------------ QKV: (row, head) tasks, one warp each
struct QkvArgs {
    void* q_out;              // [seq*RT + row][Hq*h] bf16
    void* kcache;             // this layer, first sequence of the pass: [seq][Hkv][cap][h] bf16
    void* vcache;
    const void* q_norm;       // [h] bf16 or NULL
    const void* k_norm;
    const float* rope_cos;    // [cap][h/2]
    const float* rope_sin;
    int32_t Hq, Hkv, cap, qk_norm;
    float rms_eps;
};

template <int HD>
struct QkvPre {   // fetched before the partials exist: contributor entry, rotary factors, norm weights
    SkEntry en;
    float cs[HD / 32], sn[HD / 32], gw[HD / 32];
};

// hs: head slot in the concatenated [q heads | k heads | v heads] space; pos: the row's position L + depth
template <int HD>
__device__ __forceinline__ void qkv_prefetch(QkvPre<HD>& pf, const QkvArgs& a, const StreamK& sk, int hs, int pos, int lane) {
    typedef __nv_bfloat16 T;
    constexpr int NE = HD / 32, half = HD / 2;
    const int j0 = hs * HD + lane * NE;
    pf.en = sk_entry(sk, j0 / TILE_N);
    const int which = hs < a.Hq ? 0 : (hs < a.Hq + a.Hkv ? 1 : 2);
    if (which != 2) {
#pragma unroll
        for (int i = 0; i < NE; ++i) {
            const int idx = (lane * NE + i) % half;
            pf.cs[i] = __ldg(a.rope_cos + (size_t)pos * half + idx);
            pf.sn[i] = __ldg(a.rope_sin + (size_t)pos * half + idx);
        }
        if (a.qk_norm) {
            const T* g = reinterpret_cast<const T*>(which == 0 ? a.q_norm : a.k_norm);
#pragma unroll
            for (int i = 0; i < NE; ++i) pf.gw[i] = to_f32(g[lane * NE + i]);
        }
    }
}

// sr: row in the partials; pr: row in the query buffer; slot: cache position L + row; seq: sequence within the pass
template <int HD>
__device__ __forceinline__ void qkv_finish_task(const QkvPre<HD>& pf, const QkvArgs& a, const StreamK& sk, int seq, int sr, int pr,
                                                int slot, int hs, int lane) {
    typedef __nv_bfloat16 T;
    constexpr int NE = HD / 32;
    const int j0 = hs * HD + lane * NE;
    const int f = j0 % TILE_N;
    const int which = hs < a.Hq ? 0 : (hs < a.Hq + a.Hkv ? 1 : 2);
    const int head = which == 0 ? hs : (which == 1 ? hs - a.Hq : hs - a.Hq - a.Hkv);
    float v[NE];
    if constexpr (NE == 4) {
        const float4 t = sk_sum4(sk, pf.en, sr, f);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
        // narrower heads: the same sum through the four-float helper on the enclosing aligned group
        const float4 t = sk_sum4(sk, pf.en, sr, f & ~3);
        const float tv[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < NE; ++i) v[i] = tv[(f & 3) + i];
    }
    if (which != 2) {
        if (a.qk_norm) {
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < NE; ++i) ss = __fmaf_rn(v[i], v[i], ss);
            ss = warp_sum(ss);
            const float rinv = 1.0f / sqrtf(__fadd_rn(ss / (float)HD, a.rms_eps));
#pragma unroll
            for (int i = 0; i < NE; ++i) v[i] = __fmul_rn(__fmul_rn(v[i], rinv), pf.gw[i]);
        }
        const bool low = lane < 16;
#pragma unroll
        for (int i = 0; i < NE; ++i) {
            const float other = __shfl_xor_sync(0xffffffffu, v[i], 16);
            const float rot = __fmul_rn(other, pf.sn[i]);
            v[i] = __fmaf_rn(v[i], pf.cs[i], low ? -rot : rot);
        }
    }
    T* dst;
    if (which == 0) dst = reinterpret_cast<T*>(a.q_out) + (size_t)pr * a.Hq * HD + head * HD + lane * NE;
    else dst = reinterpret_cast<T*>(which == 1 ? a.kcache : a.vcache) + (((size_t)seq * a.Hkv + head) * a.cap + slot) * HD + lane * NE;
    T o[NE];
#pragma unroll
    for (int i = 0; i < NE; ++i) o[i] = from_f32<T>(v[i]);
    if constexpr (NE == 4) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(o);
    else if constexpr (NE == 2) *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(o);
    else dst[0] = o[0];
}

// ------------------------------------------------------------------ gate/up: eight features of one row per task
// A tile holds 64 gate features (columns 0..63) and the matching 64 up features (columns 64..127).
// en: the contributor entry of tile j0 / 64; act_row: the row's [F] activations; sr: row in the partials.
// act_lo_row (may be NULL): the row of the low-order plane.
__device__ __forceinline__ void swiglu_task(const StreamK& sk, const SkEntry& en, int sr, __nv_bfloat16* act_row, __nv_bfloat16* act_lo_row,
                                            int j0, int F) {
    float4 g[2], u[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const int j = j0 + 4 * q, f = j % 64;
        if (j >= F) { g[q] = u[q] = make_float4(0.f, 0.f, 0.f, 0.f); continue; }
        g[q] = sk_sum4(sk, en, sr, f);
        u[q] = sk_sum4(sk, en, sr, 64 + f);
    }
    __nv_bfloat16 o[8], ol[8];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const float gv[4] = {g[q].x, g[q].y, g[q].z, g[q].w}, uv[4] = {u[q].x, u[q].y, u[q].z, u[q].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) split_bf16(__fmul_rn(gv[i] / __fadd_rn(1.0f, expf(-gv[i])), uv[i]), o[4 * q + i], ol[4 * q + i]);
    }
    if (j0 + 8 <= F) {
        *reinterpret_cast<uint4*>(act_row + j0) = *reinterpret_cast<const uint4*>(o);
        if (act_lo_row) *reinterpret_cast<uint4*>(act_lo_row + j0) = *reinterpret_cast<const uint4*>(ol);
    } else {
        *reinterpret_cast<uint2*>(act_row + j0) = *reinterpret_cast<const uint2*>(o);
        if (act_lo_row) *reinterpret_cast<uint2*>(act_lo_row + j0) = *reinterpret_cast<const uint2*>(ol);
    }
}

}  // namespace esp
