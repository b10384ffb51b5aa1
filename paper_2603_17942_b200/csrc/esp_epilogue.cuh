// Epilogues of the small-M GEMMs.  Both GEMM implementations (tcgen05 and
// CUDA-core) finish a 128-feature tile by placing the fp32 accumulators in
// shared memory as s_acc[row][feature] and calling run_epilogue with exactly
// 128 threads (thread f owns feature f of the tile).  The fused work is what
// follows the matrix product in the decoder layer: rotary embedding at the
// tree-depth position and the KV-cache write (QKV), the residual add (O,
// down), SiLU(gate)*up (gate/up) and per-row argmax / Top-K' / max+sum-exp
// over the vocabulary tile (LM head).
#pragma once

#include "esp_common.cuh"
#include "esp_sampling.cuh"

namespace esp {

constexpr int ACC_LD = TILE_N + 1;  // padded row stride of s_acc (floats)

// order-preserving map of a float onto an unsigned integer (larger float <=> larger key; every key > 0)
// (-0 and +0 share a key, as they compare equal)
__device__ __forceinline__ uint32_t float_order_key(float v) {
    uint32_t b = __float_as_uint(v);
    if ((b << 1) == 0u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float float_from_order_key(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__device__ __forceinline__ void epi_bar(int bar_id) {
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
}

// s_acc: [RT][ACC_LD] fp32.  s_aux: >= RT*4 floats of scratch.  tid in [0,128).
template <typename T, int EPI>
__device__ void run_epilogue(float* s_acc, float* s_aux, int tile, int seq, const EpiArgs& a, int tid, int bar_id) {
    const int f = tid;
    const int n0 = tile * TILE_N;
    const SeqState* st = a.st ? a.st + seq : nullptr;
    const int n_rows = st ? st->n_rows : a.rows_fixed;
    const int grow0 = seq * RT;

    if constexpr (EPI == EPI_STORE_F32) {
        if (n0 + f < a.n_out)
            for (int r = 0; r < n_rows; ++r) a.y_f32[(size_t)(grow0 + r) * a.n_out + n0 + f] = s_acc[r * ACC_LD + f];
    } else if constexpr (EPI == EPI_RESID) {
        if (n0 + f < a.n_out)
            for (int r = 0; r < n_rows; ++r) {
                size_t i = (size_t)(grow0 + r) * a.n_out + n0 + f;
                a.hres[i] = a.hres[i] + s_acc[r * ACC_LD + f];
            }
    } else if constexpr (EPI == EPI_SWIGLU) {
        // tile rows 0..63 hold gate features [64*tile, 64*tile+64), rows 64..127 the matching up features
        if (f < 64 && tile * 64 + f < a.n_out) {
            T* out = reinterpret_cast<T*>(a.act_out);
            for (int r = 0; r < n_rows; ++r) {
                float g = s_acc[r * ACC_LD + f], u = s_acc[r * ACC_LD + f + 64];
                float v = (g / (1.0f + expf(-g))) * u;
                out[(size_t)(grow0 + r) * a.n_out + tile * 64 + f] = from_f32<T>(v);
            }
        }
    } else if constexpr (EPI == EPI_QKV) {
        const int h = a.h, dq = a.Hq * h, dkv = a.Hkv * h;
        const int feat = n0 + f;  // index in the concatenated [q | k | v] feature space
        const int which = feat < dq ? 0 : (feat < dq + dkv ? 1 : 2);
        const int local = which == 0 ? feat : (which == 1 ? feat - dq : feat - dq - dkv);
        const int head = local / h, fl = local % h, half = h / 2;
        const int L = st ? st->L : 0;
        const int warp = f >> 5;
        if (which != 2) {
            if (a.qk_norm) {
                // per-head RMSNorm: sum of squares over the head's h features, per row
                for (int r = 0; r < n_rows; ++r) {
                    float v = s_acc[r * ACC_LD + f];
                    float ss = warp_sum(v * v);
                    if ((f & 31) == 0) s_aux[r * 4 + warp] = ss;
                }
                epi_bar(bar_id);
                const T* g = reinterpret_cast<const T*>(which == 0 ? a.q_norm : a.k_norm);
                const float gain = to_f32(g[fl]);
                const int wpw = h / 32;                    // warps per head
                const int w0 = (f / h) * wpw;              // first warp of this thread's head
                for (int r = 0; r < n_rows; ++r) {
                    float ss = 0.f;
                    for (int w = 0; w < wpw; ++w) ss += s_aux[r * 4 + w0 + w];
                    float rinv = 1.0f / sqrtf(ss / (float)h + a.rms_eps);
                    s_acc[r * ACC_LD + f] = s_acc[r * ACC_LD + f] * rinv * gain;
                }
            }
            epi_bar(bar_id);
            // rotary embedding at position L + depth, rotate-half pairing (i, i + h/2)
            const int partner = fl < half ? f + half : f - half;
            for (int r = 0; r < n_rows; ++r) {
                const int pos = L + (st ? st->row_depth[r] : r);
                const float cs = a.rope_cos[(size_t)pos * half + (fl % half)];
                const float sn = a.rope_sin[(size_t)pos * half + (fl % half)];
                const float me = s_acc[r * ACC_LD + f], other = s_acc[r * ACC_LD + partner];
                const float v = fl < half ? me * cs - other * sn : me * cs + other * sn;
                if (which == 0) {
                    reinterpret_cast<T*>(a.q_out)[(size_t)(grow0 + r) * dq + head * h + fl] = from_f32<T>(v);
                } else {
                    reinterpret_cast<T*>(a.kcache)[(((size_t)seq * a.Hkv + head) * a.cap + (L + r)) * h + fl] = from_f32<T>(v);
                }
            }
        } else {
            if (a.qk_norm) epi_bar(bar_id);
            epi_bar(bar_id);
            for (int r = 0; r < n_rows; ++r)
                reinterpret_cast<T*>(a.vcache)[(((size_t)seq * a.Hkv + head) * a.cap + (L + r)) * h + fl] =
                    from_f32<T>(s_acc[r * ACC_LD + f]);
        }
    } else if constexpr (EPI == EPI_LOGITS) {
        // warp w takes rows w, w+4, ...; a lane holds features lane, lane+32, lane+64, lane+96 of the row
        const int warp = f >> 5, lane = f & 31;
        const int n_nodes = st ? st->n_nodes : a.rows_fixed;
        const int Mtot = a.batch * RT;
        uint32_t noise_pos = 0xffffffffu;   // rows come in breadth-first order: equal depths are neighbours and
        float noise[4] = {0.f, 0.f, 0.f, 0.f};   // share their noise, which is a function of (position, token)
        // The rows' floors (see below) are fetched once per tile, all rows at a time, and the floors this tile
        // establishes go back in one batch at the end: no L2 round trip or atomic inside the row loop.
        const int S = n_rows <= 80 ? 80 : RT;                             // s_aux holds at least 3 * S words
        uint32_t* s_floor = reinterpret_cast<uint32_t*>(s_aux);          // [S] in, [S] out, [S] "this probe row has entries at or above its floor"
        uint32_t* s_need = s_floor + 2 * S;
        for (int r = f; r < n_rows; r += 128) {
            s_floor[r] = (r >= n_nodes && a.cand_floor) ? __ldcg(a.cand_floor + grow0 + r) : 0u;
            s_floor[S + r] = 0u;
        }
        epi_bar(bar_id);
        // Probe rows, one thread per row (the padded row stride keeps the threads on different banks): the tile's
        // (max, sum-exp) for the row's log-sum-exp, and whether anything of the tile can still reach the row's final
        // list.  A row whose maximum lies below its floor is done: its K' entries of this tile are empty.  With many
        // probe rows per block nearly all rows of nearly all tiles end here, without one warp-wide reduction.
        const bool many_probes = n_rows - n_nodes >= 16;     // block-uniform; a handful of probe rows is cheaper warp by warp
        if (many_probes) {
            const int r = n_nodes + f;
            if (r < n_rows) {
                const int n_valid = a.n_out - n0 < TILE_N ? a.n_out - n0 : TILE_N;
                const float* row = s_acc + r * ACC_LD;
                float tmax = -INFINITY;
                for (int i = 0; i < n_valid; ++i) tmax = fmaxf(tmax, row[i]);
                float sum = 0.f;
                for (int i = 0; i < n_valid; ++i) sum += expf(row[i] - tmax);
                a.cand_ms[(size_t)tile * Mtot + grow0 + r] = make_float2(tmax, sum);
                const bool need = float_order_key(tmax) >= s_floor[r];
                s_need[r] = need ? 1u : 0u;
                if (!need) {
                    Cand* out = a.cand + ((size_t)tile * Mtot + grow0 + r) * a.KP;
                    for (int j = 0; j < a.KP; ++j) { out[j].val = -INFINITY; out[j].id = -1; }
                }
            }
        }
        epi_bar(bar_id);
        for (int r = warp; r < n_rows; r += 4) {
            float v[4];
            int id[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                id[i] = n0 + lane + 32 * i;
                v[i] = id[i] < a.n_out ? s_acc[r * ACC_LD + lane + 32 * i] : -INFINITY;
                if (a.logits_dump && id[i] < a.n_out) a.logits_dump[(size_t)(grow0 + r) * a.n_out + id[i]] = v[i];
            }
            if (many_probes && r >= n_nodes && !s_need[r]) continue;       // warp-uniform
            const bool probe = r >= n_nodes;
            const int kp = probe ? a.KP : 1;
            Cand* out = a.cand + ((size_t)tile * Mtot + grow0 + r) * a.KP;
            if (!probe && st && a.samp_inv_temp > 0.f) {
                // sample matching: this row's token for position L + depth + 1 is the arg-max of the noisy scores
                const uint32_t pos = (uint32_t)(st->L + st->row_depth[r] + 1);
                if (pos != noise_pos) {
                    noise_pos = pos;
#pragma unroll
                    for (int i = 0; i < 4; ++i) noise[i] = gumbel_noise(a.samp_key0, a.samp_key1, pos, (uint32_t)id[i]);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (id[i] < a.n_out) v[i] = sample_score(v[i], a.samp_inv_temp, noise[i]);
            }
            if (probe && !many_probes) {
                float tmax = warp_max(fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3])));
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < 4; ++i) s += id[i] < a.n_out ? expf(v[i] - tmax) : 0.f;
                s = warp_sum(s);
                if (lane == 0) a.cand_ms[(size_t)tile * Mtot + grow0 + r] = make_float2(tmax, s);
            }
            // what other tiles have already established about this row's K'-th largest logit: a tile's own K'-th
            // best is a lower bound of it, so an entry strictly below the bound cannot make the final list
            const uint32_t floor_key = s_floor[r];
            unsigned used = 0;
            float keep_v = -INFINITY;          // lane j keeps the j-th entry (K' <= 32); one coalesced store per row
            int keep_i = -1;
            for (int j = 0; j < kp; ++j) {
                // lane-local best among unused, then warp-wide best by (value desc, id asc)
                float bv = -INFINITY;
                int bi = 0x7fffffff, bslot = -1;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (!(used >> i & 1) && id[i] < a.n_out && cand_before(v[i], id[i], bv, bi)) { bv = v[i]; bi = id[i]; bslot = i; }
                // two warp-wide integer reductions: the largest value (as an order-preserving key), then the smallest
                // token id among the lanes that hold it
                const uint32_t key = bslot >= 0 ? float_order_key(bv) : 0u;
                const uint32_t wkey = __reduce_max_sync(0xffffffffu, key);
                const uint32_t wid = __reduce_min_sync(0xffffffffu, (bslot >= 0 && key == wkey) ? (uint32_t)bi : 0xffffffffu);
                const int wi = wkey == 0u ? 0x7fffffff : (int)wid;
                const float wv = wkey == 0u ? -INFINITY : float_from_order_key(wkey);
                if (wi == bi && bslot >= 0) used |= 1u << bslot;
                if (probe && wi != 0x7fffffff && wkey < floor_key) break;   // warp-uniform: this and all later entries are out
                if (lane == j) { keep_v = wv; keep_i = wi == 0x7fffffff ? -1 : wi; }
                if (probe && a.cand_floor && j == kp - 1 && wi != 0x7fffffff && lane == 0)
                    s_floor[S + r] = wkey;                                    // this tile holds kp entries >= wv
            }
            if (lane < kp) { out[lane].val = keep_v; out[lane].id = keep_i; }
        }
        epi_bar(bar_id);
        for (int r = f; r < n_rows; r += 128)
            if (s_floor[S + r] > s_floor[r]) atomicMax(a.cand_floor + grow0 + r, s_floor[S + r]);
    }
}

}  // namespace esp
