// Device-side pieces of the tensor-core tree attention (bf16, head_dim 128) shared by the kernels that
// run it: the work of one item (one split of the cache x one KV head x one tile of 128 (row, head) pairs)
// on the tcgen05 path, and the per-(row, head) tail and merge.  The kernel that runs one attention per
// launch and the kernel that runs all layers in one launch call the same functions and give the same bits.
#pragma once

#include "esp_launch.h"
#include "esp_tc.cuh"

namespace esp {
namespace attn {

using namespace tc;

constexpr int HD = 128;
constexpr int CK = 128;                   // keys per chunk
constexpr int MP = 128;                   // (row, head) pairs per CTA
constexpr int HALF_BYTES = 128 * 128;     // one 128-row x 64-element (128-byte) swizzled tile
constexpr int Q_BYTES = 2 * HALF_BYTES, K_BYTES = 2 * HALF_BYTES, V_BYTES = 2 * HALF_BYTES, P_BYTES = 2 * HALF_BYTES;
constexpr int KV_STAGE = K_BYTES + V_BYTES;
constexpr int OFF_Q = 0, OFF_KV = Q_BYTES, OFF_P = OFF_KV + 2 * KV_STAGE;
constexpr int ITEM_BYTES = OFF_P + P_BYTES;   // shared memory one item needs: Q, two K/V stages, P
constexpr int TMEM_COLS = 512;            // S0 at 0, S1 at 128, O0 at 256, O1 at 384

__device__ __forceinline__ int tail_start_tc(int P, int dcap) {
    int t = P - dcap;
    return t <= 0 ? 0 : (t / 16) * 16;
}

// kind::f16 instruction descriptors: D = f32, A = B = bf16, M = 128, N = 128; PV takes B (V) MN-major
constexpr uint32_t IDESC_QK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t IDESC_PV = IDESC_QK | (1u << 16);

// 64 consecutive columns of this lane: two loads in flight, one wait
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
    tmem_ld32_issue(taddr, &r[0]);
    tmem_ld32_issue(taddr + 32, &r[32]);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// The producer thread waits for the kernel before this one and only then releases the kernel after it.
__device__ __forceinline__ void trigger_after_wait() {
    pdl_wait();
    pdl_launch_dependents();
}

// 2^x as one special-function instruction (results below 2^-126 flush to zero, which a softmax weight may;
// relative error about 2^-22).  Measured against exp2f(): 0.64 instead of 0.70 us for the 64 exponentials of a chunk.
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- one 128-key chunk of the online softmax, for one thread = one half (64 keys) of one pair's row.
// S (raw scores) is read from tensor memory; keys at or beyond T0row are masked; the two threads of a pair
// exchange their maxima through `xch` ([2 * MP] floats); P goes to shared memory as bf16 in the A-operand
// layout; O is rescaled in tensor memory when the running maximum moved.  Scores enter the exponent as
// fma(s, scale, -m): one rounding, spelled out so that every kernel that inlines this rounds alike.
// All 32 lanes of a warp call this together (the tensor-memory accesses are warp-wide); false = a wait ran out.
__device__ __forceinline__ bool softmax_chunk(uint32_t s_addr, uint32_t o_addr, int cbase, int T0row, float scale_log2, float& m_run,
                                              float& l_run, float* xch, uint64_t* xchg, uint32_t xchg_parity, bool wait_pv,
                                              uint64_t* pv_done, uint32_t pv_parity, bool rescale, unsigned char* prow, int pair,
                                              int hf, uint64_t* p_ready, volatile int* s_abort) {
    uint32_t sv[64];
    tmem_ld64(s_addr, sv);
    float cmax = -INFINITY;
    if (__all_sync(0xffffffffu, cbase + 64 <= T0row)) {     // every key of the half is visible to every row of the warp
#pragma unroll
        for (int i = 0; i < 64; ++i) cmax = fmaxf(cmax, __uint_as_float(sv[i]));
    } else {
#pragma unroll
        for (int i = 0; i < 64; ++i) {
            const float sc = cbase + i < T0row ? __uint_as_float(sv[i]) : -INFINITY;
            sv[i] = __float_as_uint(sc);
            cmax = fmaxf(cmax, sc);
        }
    }
    cmax = __fmul_rn(cmax, scale_log2);     // the half's maximum in the log2 domain (scaling is monotone)
    // the chunk maximum over both halves
    // (double buffered by exchange parity: a thread can be one exchange ahead of its partner, not two)
    // (one arrival per warp, after the warp's values are in shared memory: 256 single arrivals on one barrier
    // word take several hundred cycles)
    xch[hf * MP + pair] = cmax;
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(xchg);
    if (!__all_sync(0xffffffffu, mbar_wait(xchg, xchg_parity, s_abort))) return false;
    cmax = fmaxf(xch[pair], xch[MP + pair]);
    // The running reference follows the maximum lazily: it moves only when the maximum has grown by more than
    // 2^8 over it (or there was none yet).  Until then alpha is exactly 1, O needs no rescaling, and the
    // probabilities of this chunk are at most 2^8, exact in fp32 and as precise as ever in bf16.  The decision is
    // the row's own (both threads of the pair see the same maximum), so a row's bits stay independent of its
    // neighbours; whoever merges the partial takes m_run as what it is, the reference of l and O.
    const float m_max = fmaxf(m_run, cmax);
    const float m_new = (m_run == -INFINITY || __fsub_rn(m_max, m_run) > 8.f) ? m_max : m_run;
    const float m_use = m_new == -INFINITY ? 0.f : m_new;
    const float alpha = exp2f(__fsub_rn(m_run, m_use));
    // probabilities and their sum (key order), packed as bf16 pairs in registers: the P V of the previous chunk may
    // still be reading P from shared memory, and this is the long part of the chunk
    float csum = 0.f;
    const float neg_m = -m_use;
    uint32_t pk[32];
#pragma unroll
    for (int i = 0; i < 64; i += 2) {
        const float p0 = ex2_approx(__fmaf_rn(__uint_as_float(sv[i]), scale_log2, neg_m));
        const float p1 = ex2_approx(__fmaf_rn(__uint_as_float(sv[i + 1]), scale_log2, neg_m));
        csum = __fadd_rn(csum, p0);
        csum = __fadd_rn(csum, p1);
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
        pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&b2);
    }
    // (the values are pinned here: without it the compiler is free to sink the arithmetic behind the wait)
#pragma unroll
    for (int i = 0; i < 32; ++i) asm volatile("" : "+r"(pk[i]));
    // P of the previous chunk must have been consumed before it is overwritten, and O must be final
    // before it is rescaled
    if (wait_pv && !__all_sync(0xffffffffu, mbar_wait(pv_done, pv_parity, s_abort))) return false;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // P as bf16 in the A-operand layout (this half = one swizzled tile)
#pragma unroll
    for (int j = 0; j < 8; ++j)
        *reinterpret_cast<uint4*>(prow + ((j ^ (pair & 7)) << 4)) = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
    if (rescale) {
        // O <- alpha * O (in tensor memory), this thread's 64 of the 128 columns
        if (__any_sync(0xffffffffu, alpha != 1.0f)) {   // warp-uniform: skip when no lane's maximum moved
            tmem_ld64(o_addr, sv);
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
                for (int i = 0; i < 32; ++i) sv[blk * 32 + i] = __float_as_uint(__fmul_rn(__uint_as_float(sv[blk * 32 + i]), alpha));
                tmem_st32(o_addr + blk * 32, *reinterpret_cast<const uint32_t(*)[32]>(&sv[blk * 32]));
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
    }
    l_run = __fmaf_rn(l_run, alpha, csum);     // this half's share of the row sum
    m_run = m_new;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P: generic-proxy writes -> tensor-core reads
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(p_ready);      // one arrival per softmax warp
    return true;
}

// ---- one item, start to finish, on freshly initialised barriers.
struct BulkMaps {
    const CUtensorMap* q;   // [rows][Hq][128], box 64 x group x rows_per_tile
    const CUtensorMap* k;   // [cache rows][128], box 64 x 128 keys
    const CUtensorMap* v;
    int group, rows_per_tile;
};
struct BulkItem {
    int split, kvh, seq, row0, n_rows, L, beg, n_chunks;
    int kv_row0;            // row of position 0 of this (sequence, KV head) in the K/V maps
};
struct BulkShared {
    unsigned char* buf;     // 1024-byte aligned, ITEM_BYTES
    uint64_t *k_full, *k_empty, *v_full, *v_empty, *s_full;   // [2] each, count 1
    uint64_t *q_full, *pv_done;              // count 1
    uint64_t* p_ready;                       // count 8: one arrival per softmax warp
    uint64_t* xchg;                          // [4], count 2: the two warps that share a tensor-memory lane quadrant
    float* s_xchg;          // [2][2 * MP]
    volatile int* s_abort;
};
__device__ __forceinline__ void bulk_init_barriers(const BulkShared& sm) {
    for (int i = 0; i < 2; ++i) {
        mbar_init(&sm.k_full[i], 1); mbar_init(&sm.k_empty[i], 1); mbar_init(&sm.v_full[i], 1); mbar_init(&sm.v_empty[i], 1);
        mbar_init(&sm.s_full[i], 1);
    }
    mbar_init(sm.q_full, 1);
    mbar_init(sm.p_ready, 8);
    mbar_init(sm.pv_done, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&sm.xchg[i], 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 softmax (two threads per pair, 64 keys each; they also
// write the item's partial output).  Other warps fall through.  PDL: the kernel is one link of a chain of
// programmatic dependent launches (the producer thread does the wait and releases the dependent kernel).
template <bool PDL>
__device__ __forceinline__ void bulk_item_roles(const BulkMaps& mp, const AttnArgs& a, const BulkItem& it, const BulkShared& sm,
                                                uint32_t tmem_base, int warp, int lane) {
    unsigned char* smem = sm.buf;
    unsigned char* sQ = smem + OFF_Q;
    unsigned char* sP = smem + OFF_P;
    volatile int* s_abort = sm.s_abort;
    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            const int kvrow0 = it.kv_row0 + it.beg;
            bool ok = true;
            // K and V of a chunk have a stage half and a barrier pair each: a K half is free again when its Q K^T has
            // completed, about one chunk period before the V half (free when P V has), so K runs one chunk ahead of V
            // and both have two chunk periods for their trip from HBM
            auto load_k = [&](int c) -> bool {
                if (!mbar_wait(&sm.k_empty[c & 1], ((c >> 1) & 1) ^ 1, s_abort)) return false;   // a fresh barrier passes parity 1
                unsigned char* st = smem + OFF_KV + (c & 1) * KV_STAGE;
                mbar_expect_tx(&sm.k_full[c & 1], K_BYTES);
                tma_load_2d(st, mp.k, 0, kvrow0 + c * CK, &sm.k_full[c & 1]);
                tma_load_2d(st + HALF_BYTES, mp.k, 64, kvrow0 + c * CK, &sm.k_full[c & 1]);
                return true;
            };
            auto load_v = [&](int c) -> bool {
                if (!mbar_wait(&sm.v_empty[c & 1], ((c >> 1) & 1) ^ 1, s_abort)) return false;
                unsigned char* st = smem + OFF_KV + (c & 1) * KV_STAGE + K_BYTES;
                mbar_expect_tx(&sm.v_full[c & 1], V_BYTES);
                tma_load_2d(st, mp.v, 0, kvrow0 + c * CK, &sm.v_full[c & 1]);
                tma_load_2d(st + HALF_BYTES, mp.v, 64, kvrow0 + c * CK, &sm.v_full[c & 1]);
                return true;
            };
            // the cache below T0 is settled in a decode step: request it before waiting for the kernel that wrote the queries
            if (PDL && a.cache_in_flight) trigger_after_wait();
            const int n = it.n_chunks;
            ok = load_k(0) && (n < 2 || load_k(1)) && load_v(0) && (n < 2 || load_v(1));    // both stages are free
            if (PDL && !a.cache_in_flight) trigger_after_wait();
            mbar_expect_tx(sm.q_full, Q_BYTES);
            tma_load_3d(sQ, mp.q, 0, it.kvh * mp.group, it.seq * RT + it.row0, sm.q_full);
            tma_load_3d(sQ + HALF_BYTES, mp.q, 64, it.kvh * mp.group, it.seq * RT + it.row0, sm.q_full);
            if (ok && n > 2) ok = load_k(2);
            for (int c = 2; c < n && ok; ++c) ok = (c + 1 >= n || load_k(c + 1)) && load_v(c);
            if (!ok) { set_error(a.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            bool ok = true;
            const uint32_t q_addr = smem_u32(sQ), p_addr = smem_u32(sP);
            auto issue_qk = [&](int c) {
                const uint32_t k_addr = smem_u32(smem + OFF_KV + (c & 1) * KV_STAGE);
                const uint32_t tmem_s = tmem_base + (c & 1) * 128;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                    umma(tmem_s, smem_desc(q_addr + off, 16), smem_desc(k_addr + off, 16), IDESC_QK, kk > 0 ? 1u : 0u);
                }
                umma_commit(&sm.s_full[c & 1]);
                umma_commit(&sm.k_empty[c & 1]);
            };
            ok = mbar_wait(sm.q_full, 0, s_abort) && mbar_wait(&sm.k_full[0], 0, s_abort);
            if (ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_qk(0);
            }
            for (int c = 0; c < it.n_chunks && ok; ++c) {
                if (c + 1 < it.n_chunks) {     // S of the next chunk while the softmax of this one runs
                    if (!mbar_wait(&sm.k_full[(c + 1) & 1], ((c + 1) >> 1) & 1, s_abort)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    issue_qk(c + 1);
                }
                if (!mbar_wait(sm.p_ready, c & 1, s_abort) || !mbar_wait(&sm.v_full[c & 1], (c >> 1) & 1, s_abort)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t v_addr = smem_u32(smem + OFF_KV + (c & 1) * KV_STAGE + K_BYTES);
#pragma unroll
                for (int kk = 0; kk < CK / 16; ++kk) {
                    const uint32_t p_off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;     // P: K-major over keys
                    const uint32_t v_off = kk * 16 * 128;                              // V: 16 key rows of 128 bytes further
                    umma(tmem_base + 256, smem_desc(p_addr + p_off, 16), smem_desc(v_addr + v_off, HALF_BYTES), IDESC_PV,
                         (c > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(sm.pv_done);
                umma_commit(&sm.v_empty[c & 1]);
            }
            // the arrivals on the K/V stage barriers are the item's last asynchronous ones: see them land, so that
            // a kernel that runs several items may initialise the barriers again
            for (int c = it.n_chunks - 2 < 0 ? 0 : it.n_chunks - 2; c < it.n_chunks && ok; ++c)
                ok = mbar_wait(&sm.k_empty[c & 1], (c >> 1) & 1, s_abort) && mbar_wait(&sm.v_empty[c & 1], (c >> 1) & 1, s_abort);
            if (!ok) { set_error(a.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else if (warp < 10) {
        // ---------------- softmax warps 2..9: a thread owns one pair (= tensor-memory lane) and one half of the
        // chunk's 128 keys (warps 2-5 keys 0..63, warps 6-9 keys 64..127); the two threads of a pair exchange
        // their maxima (per chunk) and their sums (at the end) through shared memory
        const int q4 = warp & 3;
        const int hf = (warp - 2) >> 2;
        const int pair = q4 * 32 + lane;
        const int r = it.row0 + pair / mp.group, head = it.kvh * mp.group + pair % mp.group;
        const bool pv = pair / mp.group < mp.rows_per_tile && r < it.n_rows && r < RT;
        int T0row = 0;
        if (pv) T0row = tail_start_tc(it.L + (a.st ? a.st[it.seq].row_depth[r] : a.depth[it.seq * RT + r]), a.dcap);
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16) + hf * 64;   // this thread's 64 columns of S / O
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int c = 0; c < it.n_chunks && ok; ++c) {
            // (a wait that fails must take the whole warp out: the tensor-memory accesses below are warp-wide)
            if (!__all_sync(0xffffffffu, mbar_wait(&sm.s_full[c & 1], (c >> 1) & 1, s_abort))) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            ok = softmax_chunk(lane_addr + (c & 1) * 128, lane_addr + 256, it.beg + c * CK + hf * 64, T0row, a.scale_log2, m_run, l_run,
                               sm.s_xchg + (c & 1) * 2 * MP, sm.xchg + q4, c & 1, c > 0, sm.pv_done, (c - 1) & 1, c > 0,
                               sP + hf * HALF_BYTES + pair * 128, pair, hf, sm.p_ready, s_abort);
        }
        if (ok && !__all_sync(0xffffffffu, mbar_wait(sm.pv_done, (it.n_chunks - 1) & 1, s_abort))) ok = false;
        float* xl = sm.s_xchg + (it.n_chunks & 1) * 2 * MP;
        if (ok) {
            // the row sum = first half's share + second half's share
            xl[hf * MP + pair] = l_run;
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.xchg + q4);
            if (!__all_sync(0xffffffffu, mbar_wait(sm.xchg + q4, it.n_chunks & 1, s_abort))) ok = false;
        }
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // O half-row -> shared memory (the K/V stages are free now) -> one 256-byte bulk copy per thread.  The
            // tensor-memory load is warp-wide: every lane takes part, lanes without a pair copy nothing.
            uint32_t ov[64];
            tmem_ld64(lane_addr + 256, ov);
            float* orow = reinterpret_cast<float*>(smem + OFF_KV) + pair * (HD + 4) + hf * 64;   // rows padded by 16 bytes: no bank conflicts
#pragma unroll
            for (int i = 0; i < 64; i += 4)
                *reinterpret_cast<uint4*>(orow + i) = make_uint4(ov[i], ov[i + 1], ov[i + 2], ov[i + 3]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            if (pv) {
                const size_t idx = ((size_t)(it.seq * RT + r) * a.Hq + head) * a.n_split_max + it.split;
                if (hf == 0) __stcg(a.part_ml + idx, make_float2(m_run, __fadd_rn(xl[pair], xl[MP + pair])));
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                             ::"l"(a.part_o + idx * HD + hf * 64), "r"(smem_u32(orow)), "r"(64 * 4) : "memory");
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");        // copies complete: shared memory may be released
        } else if (lane == 0) {
            set_error(a.err, DEV_E_WAIT_TIMEOUT);
            *s_abort = 1;
        }
    }
}

// ---- tail + merge: one warp per (row, head) pair
__device__ __forceinline__ int nth_set_bit128(unsigned long long lo, unsigned long long hi, int n) {
    int c = __popcll(lo);
    unsigned long long m = lo;
    int base = 0;
    if (n >= c) { n -= c; m = hi; base = 64; }
    for (int i = 0; i < n; ++i) m &= m - 1;
    return m ? base + __ffsll((long long)m) - 1 : -1;
}
__device__ __forceinline__ void merge_ml(float& m, float& l, float (&o)[4], float cm, float cl, const float (&co)[4]) {
    // products and sums are rounded one by one, so that every instance of the kernel rounds alike
    const float mn = fmaxf(m, cm);
    const float a = exp2f(__fsub_rn(m, mn)), b = exp2f(__fsub_rn(cm, mn));
    l = __fmaf_rn(l, a, __fmul_rn(cl, b));
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = __fmaf_rn(o[i], a, __fmul_rn(co[i], b));
    m = mn;
}

struct PairCtx {            // one (row, head) pair of one sequence
    int r, head, seq, L, depth;
    unsigned long long lo, hi;   // the row's ancestor-or-self mask over block rows
};
struct TailAcc {            // running (max, sum, weighted values) of a key list, this lane's 4 of the 128 dims
    float m, l, o[4];
};
template <int PB>
struct FirstPartials {      // the first PB split partials of a pair, requested ahead of their use
    float2 ml[PB];
    float4 c4[PB];
};
__device__ __forceinline__ int pair_splits(const AttnArgs& a, const PairCtx& c) {
    return (tail_start_tc(c.L + c.depth, a.dcap) + a.split_len - 1) / a.split_len;
}
template <int PB>
__device__ __forceinline__ void request_partials(FirstPartials<PB>& fp, const AttnArgs& a, const PairCtx& c, int lane) {
    const int n_sp = pair_splits(a, c);
    const size_t base = ((size_t)(c.seq * RT + c.r) * a.Hq + c.head) * a.n_split_max;
#pragma unroll
    for (int u = 0; u < PB; ++u) {
        if (u < n_sp) {
            fp.ml[u] = __ldcg(a.part_ml + base + u);
            fp.c4[u] = __ldcg(reinterpret_cast<const float4*>(a.part_o + (base + u) * HD + lane * 4));
        }
    }
}

// The tail: positions T0..P in position order, lane j owns key j of a 32-key chunk (chunk grid anchored at T0);
// in-flight ancestors are found through the ancestor mask.  s_q: 128 floats of shared memory owned by the warp.
// What this step wrote shortly before, in another kernel or CTA -- the queries and the keys / values of the block's
// own rows (slots >= L) -- is read with L2 loads (ld.global.cg), never through L1; cache positions below L were
// written by earlier steps and go through L1, where the pairs that share a KV head find them again.
// KB8 / VB: 16-byte key pieces / value rows in flight.
template <int KB8, int VB>
__device__ __forceinline__ void tail_pair(TailAcc& t, const AttnArgs& a, const PairCtx& c, float* s_q, int lane) {
    const int kvh = c.head / (a.Hq / a.Hkv);
    const int P = c.L + c.depth, T0 = tail_start_tc(P, a.dcap);
    const __nv_bfloat16* kbase = reinterpret_cast<const __nv_bfloat16*>(a.kc) + ((size_t)c.seq * a.Hkv + kvh) * a.cap * HD;
    const __nv_bfloat16* vbase = reinterpret_cast<const __nv_bfloat16*>(a.vc) + ((size_t)c.seq * a.Hkv + kvh) * a.cap * HD;
    const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((size_t)(c.seq * RT + c.r) * a.Hq + c.head) * HD;
    {
        const uint2 qq = __ldcg(reinterpret_cast<const uint2*>(q + lane * 4));
        const __nv_bfloat162 q01 = *reinterpret_cast<const __nv_bfloat162*>(&qq.x), q23 = *reinterpret_cast<const __nv_bfloat162*>(&qq.y);
        s_q[lane * 4 + 0] = __low2float(q01); s_q[lane * 4 + 1] = __high2float(q01);
        s_q[lane * 4 + 2] = __low2float(q23); s_q[lane * 4 + 3] = __high2float(q23);
    }
    __syncwarp();
    t.m = -INFINITY; t.l = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) t.o[i] = 0.f;
    const int n_tail = P - T0 + 1;
    for (int t0 = 0; t0 < n_tail; t0 += 32) {
        const int tt = t0 + lane;
        bool valid = tt < n_tail;
        int slot = 0;
        if (valid) {
            const int pos = T0 + tt;
            if (pos < c.L) slot = pos;
            else {
                const int b = nth_set_bit128(c.lo, c.hi, pos - c.L);
                if (b < 0) { set_error(a.err, DEV_E_INDEX); valid = false; }
                else slot = c.L + b;
            }
        }
        float sc = -INFINITY;
        if (valid) {
            const uint4* kr = reinterpret_cast<const uint4*>(kbase + (size_t)slot * HD);
            float acc = 0.f;
#pragma unroll
            for (int dh = 0; dh < HD / 8; dh += KB8) {
                uint4 kreg[KB8];
#pragma unroll
                for (int d8 = 0; d8 < KB8; ++d8) kreg[d8] = slot < c.L ? kr[dh + d8] : __ldcg(kr + dh + d8);
#pragma unroll
                for (int d8 = dh; d8 < dh + KB8; ++d8) {
                    const uint4 kk = kreg[d8 - dh];
                    const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kk);
                    const float4 qa = *reinterpret_cast<const float4*>(s_q + d8 * 8), qb = *reinterpret_cast<const float4*>(s_q + d8 * 8 + 4);
                    acc = __fmaf_rn(qa.x, __low2float(k2[0]), acc); acc = __fmaf_rn(qa.y, __high2float(k2[0]), acc);
                    acc = __fmaf_rn(qa.z, __low2float(k2[1]), acc); acc = __fmaf_rn(qa.w, __high2float(k2[1]), acc);
                    acc = __fmaf_rn(qb.x, __low2float(k2[2]), acc); acc = __fmaf_rn(qb.y, __high2float(k2[2]), acc);
                    acc = __fmaf_rn(qb.z, __low2float(k2[3]), acc); acc = __fmaf_rn(qb.w, __high2float(k2[3]), acc);
                }
            }
            sc = __fmul_rn(acc, a.scale_log2);
        }
        float cm = sc;
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, of));
        const float pe = valid ? exp2f(__fsub_rn(sc, cm)) : 0.f;
        float cl = pe;
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) cl = __fadd_rn(cl, __shfl_xor_sync(0xffffffffu, cl, of));
        float co[4] = {0.f, 0.f, 0.f, 0.f};
        // weighted values, keys in position order; the loads of VB keys are issued before their sums
        // (a key that is not in the chunk reads slot 0 with weight 0 and is skipped)
        for (int j0 = 0; j0 < 32; j0 += VB) {
            float pj[VB];
            uint2 vv[VB];
#pragma unroll
            for (int u = 0; u < VB; ++u) {
                pj[u] = __shfl_sync(0xffffffffu, pe, j0 + u);
                const int sj = __shfl_sync(0xffffffffu, slot, j0 + u);
                const uint2* vr = reinterpret_cast<const uint2*>(vbase + (size_t)sj * HD + lane * 4);
                vv[u] = sj < c.L ? *vr : __ldcg(vr);
            }
#pragma unroll
            for (int u = 0; u < VB; ++u) {
                if (pj[u] != 0.f) {
                    const __nv_bfloat162 v01 = *reinterpret_cast<const __nv_bfloat162*>(&vv[u].x), v23 = *reinterpret_cast<const __nv_bfloat162*>(&vv[u].y);
                    co[0] = __fmaf_rn(pj[u], __low2float(v01), co[0]); co[1] = __fmaf_rn(pj[u], __high2float(v01), co[1]);
                    co[2] = __fmaf_rn(pj[u], __low2float(v23), co[2]); co[3] = __fmaf_rn(pj[u], __high2float(v23), co[3]);
                }
            }
        }
        merge_ml(t.m, t.l, t.o, cm, cl, co);
    }
    __syncwarp();     // s_q may be rewritten by the warp's next pair
}

// The merge: bulk partials in split order, the tail last; a lane owns 4 of the 128 output dims.
template <int PB>
__device__ __forceinline__ void merge_pair(const FirstPartials<PB>& fp, const TailAcc& t, const AttnArgs& a, const PairCtx& c, int lane) {
    const int n_sp = pair_splits(a, c);
    const size_t base = ((size_t)(c.seq * RT + c.r) * a.Hq + c.head) * a.n_split_max;
    float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < PB; ++u) {
        if (u < n_sp) {
            const float co[4] = {fp.c4[u].x, fp.c4[u].y, fp.c4[u].z, fp.c4[u].w};
            merge_ml(m, l, o, fp.ml[u].x, fp.ml[u].y, co);
        }
    }
    for (int s0 = PB; s0 < n_sp; s0 += PB) {
        float2 ml[PB];
        float4 c4[PB];
#pragma unroll
        for (int u = 0; u < PB; ++u) {
            if (s0 + u < n_sp) {
                ml[u] = __ldcg(a.part_ml + base + s0 + u);
                c4[u] = __ldcg(reinterpret_cast<const float4*>(a.part_o + (base + s0 + u) * HD + lane * 4));
            }
        }
#pragma unroll
        for (int u = 0; u < PB; ++u) {
            if (s0 + u < n_sp) {
                const float co[4] = {c4[u].x, c4[u].y, c4[u].z, c4[u].w};
                merge_ml(m, l, o, ml[u].x, ml[u].y, co);
            }
        }
    }
    merge_ml(m, l, o, t.m, t.l, t.o);
    const float inv = 1.0f / l;
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out) + ((size_t)(c.seq * RT + c.r) * a.Hq + c.head) * HD + lane * 4;
    __nv_bfloat16 oh[4], ol[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float v = __fmul_rn(o[i], inv);
        oh[i] = __float2bfloat16_rn(v);
        ol[i] = __float2bfloat16_rn(__fsub_rn(v, __bfloat162float(oh[i])));
    }
    *reinterpret_cast<uint2*>(out) = *reinterpret_cast<const uint2*>(oh);
    if (a.out_lo)      // low-order plane for an O projection that reads the output as hi + lo
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(a.out_lo) + ((size_t)(c.seq * RT + c.r) * a.Hq + c.head) * HD + lane * 4) =
            *reinterpret_cast<const uint2*>(ol);
}

}  // namespace attn
}  // namespace esp
