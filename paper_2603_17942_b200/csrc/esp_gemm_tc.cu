// Small-M bf16 GEMM for the decode-and-verify step on the Blackwell tensor
// cores: y[row][n] = sum_k x[row][k] * w[n][k] for at most 80 rows.
//
// The weight matrix is the MMA "A" operand (128 output features on the MMA-M
// dimension), the token rows are the "B" operand (MMA-N = 80), so the large
// operand fills the tensor core and the 80 rows cost no padding.  Both
// operands are K-major and arrive through TMA with the 128-byte swizzle;
// tcgen05.mma accumulates fp32 in tensor memory; four epilogue warps read it
// back with tcgen05.ld.
//
// The step is bound by streaming the weights once from HBM, so the work is
// cut stream-K style: the (tile, k-block) units of one GEMM are dealt out in
// equal contiguous ranges to one persistent CTA per SM.  A tile whose k-range
// is split over several CTAs is summed from fp32 partials in CTA order (a
// fixed order, independent of arrival order and of the number of rows):
//   * EPI_PARTIAL (QKV, O, down: every tile is split): the kernel only stores
//     partials; the kernel that consumes the result (RoPE/cache write,
//     residual add + RMSNorm) sums them, fully parallel and off this kernel's
//     critical path;
//   * fused epilogues (gate/up with SiLU*up, LM head with Top-K'): whichever
//     contributor of a split tile arrives last sums and finishes it.  Each CTA
//     does its split pieces first and its whole tiles after, so this happens
//     while the weight stream of the whole tiles is running.
// No CTA ever waits for another.  The kernel is launched with programmatic
// dependent launch: the weight tiles of the first ring stages are requested
// before waiting for the preceding kernel, the activation tiles after.
// Every mbarrier wait is bounded; on a timeout the kernel records
// DEV_E_WAIT_TIMEOUT, lets its copies drain, frees its tensor memory and
// returns.
#include <new>
#include <string.h>

#include "esp_epilogue.cuh"
#include "esp_launch.h"
#include "esp_gemm_tc.cuh"

namespace esp {

namespace {

using namespace tc;

// NRS = rows of a sequence's block that take part (80, or 128 for blocks of more than 80 rows); NQ = sequences
// one launch covers: the first NRS rows of their activation blocks ([RT][K] each, consecutive) are gathered by
// one 3-D TMA box into one B operand of NQ*NRS <= 256 rows, so the weights are streamed once for all of them
// (partial-only output only).
//
// Ring depth.  The bytes in flight per SM (depth x 16 KB of weights) over the load round trip bound the stream rate,
// and the ring is also what is requested before the preceding kernel has finished: deeper is better.  The
// partial-only kernel keeps no accumulator copy in shared memory and spends that room on the ring.
// Planes (PL).  The activations reach the tensor cores as bf16.  A plan with two planes reads them as a pair
// x = hi + lo (hi = bf16(x), lo = bf16(x - hi), stored PL * n_seq blocks apart in the same buffer) and issues every
// MMA twice into the same accumulator, first with hi, then with lo: the product then sees the activation to 2^-17
// instead of 2^-9, for 10 KB more shared memory per stage and sequence.
__host__ __device__ constexpr int stages_of(int epi, int nq, int nrs, int pl = 1) {
    return pl == 2 ? (nrs == 80 ? (nq == 2 ? 4 : 6) : 4)
                   : (nrs == 80 ? (nq == 3 ? 4 : (nq == 2 ? 6 : (epi == EPI_PARTIAL ? 8 : 6)))
                                : (nq == 2 ? 4 : (epi == EPI_PARTIAL ? 7 : 4)));
}
__host__ __device__ constexpr int b_bytes_of(int nq, int nrs) { return nq * nrs * BK * 2; }   // 10240 per 80-row sequence and plane
__host__ __device__ constexpr int stage_bytes_of(int nq, int nrs, int pl = 1) { return A_BYTES + pl * b_bytes_of(nq, nrs); }
// two accumulator buffers in tensor memory: 128 columns each for up to 128 rows, 256 each beyond
__host__ __device__ constexpr int acc_cols_of(int nr) { return nr <= 128 ? 128 : 256; }
constexpr int NUM_THREADS = 192;
constexpr int MAX_NQ = 3;
__host__ __device__ constexpr int max_nq_of(int nrs, int pl = 1) { return pl == 2 ? (nrs == 80 ? 2 : 1) : (nrs == 80 ? 3 : 2); }

struct TcParams {
    CUtensorMap map_a[3];
    CUtensorMap map_b;      // activations [sequence][RT][K], box = NQ sequences x NRS rows x 64 (one map per NQ)
    int32_t b_seq0;         // first sequence (block of RT activation rows) of this launch
    int32_t b_plane_seqs;   // blocks between the hi and the lo plane of the activations (two-plane plans)
    int32_t rows_w[3];
    int32_t n_tiles, KB, grid, epi;
    int32_t map_swiglu;  // tile = 64 rows of w[0] (gate) + the matching 64 rows of w[1] (up)
    int32_t slots;       // partial slots per CTA
    const unsigned char* a_packed;  // weights repacked per (tile, k-block) unit, or NULL: read w[] through map_a
    float* partials;   // [grid][slots][NQ*NRS][TILE_N]
    int* counters;     // [n_tiles], zero between launches
    int* err;
    EpiArgs a;
};

// which weight matrix / row the two 64-row halves of a tile come from
__device__ __forceinline__ void tile_source(const TcParams& p, int tile, int half, int& m, int& row) {
    if (p.map_swiglu) { m = half; row = tile * 64; return; }
    int feat = tile * TILE_N;
    m = 0;
    while (m < 2 && feat >= p.rows_w[m]) { feat -= p.rows_w[m]; ++m; }
    row = feat + half * 64;
}

template <int EPI, int NQ, int NRS, int PL>
__global__ void __launch_bounds__(NUM_THREADS, 1) k_gemm_tc(const __grid_constant__ TcParams p) {
    static_assert(NQ == 1 || EPI == EPI_PARTIAL, "several sequences per launch: partial-only output");
    static_assert(NQ * NRS <= 256 && (PL == 1 || NQ > 1 || 2 * NRS <= 256) && NRS % 16 == 0 && NRS <= RT, "MMA N");
    static_assert(PL == 1 || EPI == EPI_PARTIAL, "two activation planes: partial-only output");
    // One sequence with two planes: hi and lo rows sit back to back in the stage and form ONE B operand of 2 * NRS
    // rows; the accumulator gets W x_hi in columns [0, NRS) and W x_lo in [NRS, 2 NRS), added by the epilogue.
    // (One MMA per k-step reads the weight slice once from shared memory; two MMAs would read it twice.)
    constexpr bool JOINT = PL == 2 && NQ == 1;
    constexpr int N_MMA = JOINT ? 2 * NRS : NQ * NRS;
    constexpr int STAGE_BYTES = stage_bytes_of(NQ, NRS, PL), ACC_COLS = acc_cols_of(N_MMA), TMEM_COLS = 2 * ACC_COLS;
    constexpr int B_PLANE = b_bytes_of(NQ, NRS);
    constexpr uint32_t IDESC = idesc_of(N_MMA);
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int STAGES = stages_of(EPI, NQ, NRS, PL);
    unsigned char* stages = smem;
    float* s_acc = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES);
    float* s_aux = s_acc + (EPI == EPI_PARTIAL ? 0 : NRS * ACC_LD);
    uint64_t* full = reinterpret_cast<uint64_t*>(s_aux + (EPI == EPI_PARTIAL ? 0 : NRS * 4));
    uint64_t* empty = full + STAGES;
    uint64_t* tfull = empty + STAGES;
    uint64_t* tempty = tfull + 2;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
    int* s_flag = const_cast<int*>(s_abort) + 1;    // [0] = wait failures of the epilogue warps, [1] = "I am last"

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long U = (long long)p.n_tiles * p.KB, G = p.grid;
    const long long u0 = sk_begin(blockIdx.x, U, G), u1 = sk_begin(blockIdx.x + 1, U, G);
    const Range rng = make_range(u0, u1, p.KB, p.slots);

    if (threadIdx.x == 0) {
        pdl_launch_dependents();
        prefetch_tensormap(&p.map_b);
        if (!p.a_packed)
            for (int i = 0; i < 3; ++i)
                if (p.rows_w[i] > 0) prefetch_tensormap(&p.map_a[i]);
        for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 128); }
        *s_abort = 0;
        s_flag[0] = 0;
        s_flag[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            // The weights do not depend on the kernel before this one: fill the ring with weight tiles first,
            // wait for that kernel, then add the activation tiles.
            const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
            const int n_items = (int)(u1 - u0);
            const int n_pre = n_items < STAGES ? n_items : STAGES;
            for (int pass = 0; pass < 2; ++pass) {
                int it = 0;
                for (int i = 0; i < rng.n_seg && it < n_pre; ++i) {
                    const Seg sg = get_seg(rng, i);
                    int m0, r0, m1, r1;
                    tile_source(p, sg.tile, 0, m0, r0);
                    tile_source(p, sg.tile, 1, m1, r1);
                    for (int kb = sg.kb0; kb < sg.kb1 && it < n_pre; ++kb, ++it) {
                        unsigned char* sa = stages + it * STAGE_BYTES;
                        if (pass == 0) {
                            mbar_expect_tx(&full[it], STAGE_BYTES);
                            if (p.a_packed) {
                                bulk_load(sa, p.a_packed + ((size_t)sg.tile * p.KB + kb) * A_BYTES, A_BYTES, &full[it], pol_w);
                            } else {
                                tma_load_2d_hint(sa, &p.map_a[m0], kb * BK, r0, &full[it], pol_w);
                                tma_load_2d_hint(sa + A_BYTES / 2, &p.map_a[m1], kb * BK, r1, &full[it], pol_w);
                            }
                        } else {
#pragma unroll
                            for (int pl = 0; pl < PL; ++pl)
                                tma_load_3d_hint(sa + A_BYTES + pl * B_PLANE, &p.map_b, kb * BK, 0, p.b_seq0 + pl * p.b_plane_seqs, &full[it], pol_x);
                        }
                    }
                }
                if (pass == 0) pdl_wait();
            }
            int stage = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int i = 0; i < rng.n_seg && ok; ++i) {
                const Seg sg = get_seg(rng, i);
                int m0, r0, m1, r1;
                tile_source(p, sg.tile, 0, m0, r0);
                tile_source(p, sg.tile, 1, m1, r1);
                for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
                    if (it >= n_pre) {
                        if (!mbar_wait(&empty[stage], phase ^ 1, s_abort)) { ok = false; break; }
                        unsigned char* sa = stages + stage * STAGE_BYTES;
                        mbar_expect_tx(&full[stage], STAGE_BYTES);
                        if (p.a_packed) {
                            bulk_load(sa, p.a_packed + ((size_t)sg.tile * p.KB + kb) * A_BYTES, A_BYTES, &full[stage], pol_w);
                        } else {
                            tma_load_2d_hint(sa, &p.map_a[m0], kb * BK, r0, &full[stage], pol_w);
                            tma_load_2d_hint(sa + A_BYTES / 2, &p.map_a[m1], kb * BK, r1, &full[stage], pol_w);
                        }
#pragma unroll
                        for (int pl = 0; pl < PL; ++pl)
                            tma_load_3d_hint(sa + A_BYTES + pl * B_PLANE, &p.map_b, kb * BK, 0, p.b_seq0 + pl * p.b_plane_seqs, &full[stage], pol_x);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) { set_error(p.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int i = 0; i < rng.n_seg && ok; ++i) {
                const Seg sg = get_seg(rng, i);
                const int buf = i & 1;
                if (!mbar_wait(&tempty[buf], ((i >> 1) & 1) ^ 1, s_abort)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + buf * ACC_COLS;
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    if (!mbar_wait(&full[stage], phase, s_abort)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = smem_u32(stages + stage * STAGE_BYTES);
                    const uint64_t da = smem_desc(sa, 16), db = smem_desc(sa + A_BYTES, 16);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        umma(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), IDESC, (kb > sg.kb0 || k > 0) ? 1u : 0u);
                        if constexpr (PL == 2 && !JOINT)      // several sequences: the same step with their low-order planes
                            umma(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)((B_PLANE >> 4) + k * 2), IDESC, 1u);
                    }
                    umma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit(&tfull[buf]);
            }
            if (!ok) { set_error(p.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else {
        // ---------------- epilogue warps: TMEM -> registers -> partial and/or fused epilogue
        pdl_wait();
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int f = q * 32 + lane;            // feature of the tile owned by this thread
        const int et = threadIdx.x - 64;        // 0..127 index among the epilogue threads
        const int n_rows = p.a.st ? (p.a.st->active ? p.a.st->n_rows : 0) : p.a.rows_fixed;
        StreamK sk;
        sk.partials = p.partials; sk.table = nullptr; sk.n_tiles = p.n_tiles; sk.KB = p.KB; sk.G = p.grid; sk.slots = p.slots;
        sk.rows = NQ * NRS; sk.seq_rows = NRS;
        bool ok = true;
        for (int i = 0; i < rng.n_seg && ok; ++i) {
            const Seg sg = get_seg(rng, i);
            const int buf = i & 1;
            bool mine = true;
            if (lane == 0) mine = mbar_wait(&tfull[buf], (i >> 1) & 1, s_abort);
            if (lane == 0 && !mine) atomicOr(&s_flag[0], 1);
            epi_bar(2);
            if (s_flag[0]) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + buf * ACC_COLS + ((uint32_t)(q * 32) << 16);
            uint32_t v[NRS];
            if constexpr (NQ > 1) {
                // sequence by sequence: 80 accumulator columns -> that sequence's rows of the partial
                float* part = p.partials + ((size_t)(blockIdx.x * p.slots + sg.slot) * (NQ * NRS)) * TILE_N + f;
#pragma unroll 1
                for (int sq = 0; sq < NQ; ++sq) {
#pragma unroll
                    for (int c = 0; c < NRS / 16; ++c)
                        tmem_ld16_issue(taddr + sq * NRS + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&v[c * 16]));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const SeqState* sst = p.a.st + sq;
                    const int nr = sst->active ? sst->n_rows : 0;
#pragma unroll
                    for (int r = 0; r < NRS; ++r)
                        if (r < nr) __stcg(part + (size_t)(sq * NRS + r) * TILE_N, __uint_as_float(v[r]));
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                mbar_arrive(&tempty[buf]);
                continue;
            }
#pragma unroll
            for (int c = 0; c < NRS / 16; ++c) tmem_ld16_issue(taddr + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&v[c * 16]));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if constexpr (JOINT) {      // + the product with the low-order plane
#pragma unroll
                for (int c = 0; c < NRS / 16; ++c) {
                    uint32_t lo16[16];
                    tmem_ld16_issue(taddr + NRS + c * 16, lo16);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[c * 16 + j] = __float_as_uint(__fadd_rn(__uint_as_float(v[c * 16 + j]), __uint_as_float(lo16[j])));
                }
            }
            // the accumulator is in registers: hand the tensor-memory buffer back to the MMA warp
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(&tempty[buf]);
            const bool direct = EPI != EPI_PARTIAL && sg.whole;
            if (direct) {
#pragma unroll
                for (int r = 0; r < NRS; ++r) s_acc[r * ACC_LD + f] = __uint_as_float(v[r]);
            } else {
                float* part = p.partials + ((size_t)(blockIdx.x * p.slots + sg.slot) * NRS) * TILE_N + f;
#pragma unroll
                for (int r = 0; r < NRS; ++r)
                    if (r < n_rows) __stcg(part + r * TILE_N, __uint_as_float(v[r]));
            }
            if (EPI == EPI_PARTIAL) continue;   // the consumer kernel sums the partials
            bool finish = direct;
            if (!direct) {
                int c_first, c_last;
                sk_contributors(sk, sg.tile, c_first, c_last);
                __threadfence();
                epi_bar(2);
                if (et == 0) {
                    const int old = atomicAdd(&p.counters[sg.tile], 1);
                    s_flag[1] = (old == c_last - c_first) ? 1 : 0;
                }
                epi_bar(2);
                finish = s_flag[1] != 0;
                if (finish) {
                    // last contributor of this tile: sum the partials in CTA order (fixed, whoever arrives last)
                    __threadfence();
                    // thread et: features 4*(et%32)..+3, rows et/32 + 4*i; every load of a batch is issued before the sums
                    const int f4 = (et & 31) * 4, rg = et >> 5;
                    for (int i0 = 0; i0 < NRS / 4; i0 += 4) {
                        if (rg + 4 * i0 >= n_rows) break;
                        float4 acc[4];
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii) acc[ii] = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int cb = c_first; cb <= c_last; cb += 4) {
                            float4 t[4][4];
#pragma unroll
                            for (int cc = 0; cc < 4; ++cc) {
                                const int c = cb + cc;
                                const bool cv = c <= c_last;
                                const float* src = sk_partial(sk, cv ? c : c_first, sg.tile, 0) + f4;
#pragma unroll
                                for (int ii = 0; ii < 4; ++ii) {
                                    const int r = rg + 4 * (i0 + ii);
                                    t[cc][ii] = (cv && r < n_rows) ? __ldcg(reinterpret_cast<const float4*>(src + (size_t)r * TILE_N))
                                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
                                }
                            }
#pragma unroll
                            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                                for (int ii = 0; ii < 4; ++ii) {
                                    acc[ii].x += t[cc][ii].x; acc[ii].y += t[cc][ii].y;
                                    acc[ii].z += t[cc][ii].z; acc[ii].w += t[cc][ii].w;
                                }
                        }
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii) {
                            const int r = rg + 4 * (i0 + ii);
                            if (r < NRS) {
                                float* d = s_acc + r * ACC_LD + f4;
                                d[0] = acc[ii].x; d[1] = acc[ii].y; d[2] = acc[ii].z; d[3] = acc[ii].w;
                            }
                        }
                    }
                    if (et == 0) p.counters[sg.tile] = 0;
                }
            }
            if (finish) {
                epi_bar(2);
                run_epilogue<__nv_bfloat16, EPI>(s_acc, s_aux, sg.tile, 0, p.a, f, 2);
            }
            epi_bar(2);
        }
        if (!ok && lane == 0) { set_error(p.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
    }
    // ---------------- teardown (every thread arrives here)
    __syncthreads();
    if (*s_abort) {
        // give copies that may still be in flight time to land before the block's shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// Repack of the weights for streaming: unit (tile, k-block) = the 128 x 64 bf16 block the main loop consumes per
// stage, stored contiguously (16 KB) in the 128-byte-swizzled layout the MMA descriptor expects, rows and columns
// outside the matrices zero.  One block per unit, thread r copies row r.
struct PackArgs {
    const __nv_bfloat16* w[3];
    int32_t rows_w[3];
    int32_t K, KB, map_swiglu;
};
__global__ void __launch_bounds__(128) k_pack_weights(PackArgs g, unsigned char* out) {
    const long long unit = blockIdx.x;
    const int tile = (int)(unit / g.KB), kb = (int)(unit % g.KB), r = threadIdx.x;
    int m, row;
    if (g.map_swiglu) { m = r >> 6; row = tile * 64 + (r & 63); }
    else {
        row = tile * TILE_N + r;
        m = 0;
        while (m < 2 && row >= g.rows_w[m]) { row -= g.rows_w[m]; ++m; }
    }
    const bool row_ok = g.w[m] != nullptr && row < g.rows_w[m];
    unsigned char* dst = out + (size_t)unit * A_BYTES + r * 128;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int k0 = kb * BK + j * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row_ok && k0 < g.K) v = *reinterpret_cast<const uint4*>(g.w[m] + (size_t)row * g.K + k0);
        *reinterpret_cast<uint4*>(dst + ((j ^ (r & 7)) << 4)) = v;
    }
}

constexpr size_t smem_bytes_of(int epi, int nq, int nrs, int pl = 1) {
    return 1024 + (size_t)stages_of(epi, nq, nrs, pl) * stage_bytes_of(nq, nrs, pl) +
           (epi == EPI_PARTIAL ? 0 : sizeof(float) * (nrs * ACC_LD + nrs * 4)) + 256;
}

// [rows][K] bf16 row-major, box = 64 k-elements x box_rows rows, 128-byte swizzle, out-of-range reads give zero
int make_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows) {
    EncodeFn enc = get_encode();
    if (!enc) return -1;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

// activations [n_seq][RT][K] bf16: box = 64 k-elements x box_rows rows x box_seqs sequences, 128-byte swizzle
int make_map_b(CUtensorMap* m, const void* base, int n_seq, int K, int box_rows, int box_seqs) {
    EncodeFn enc = get_encode();
    if (!enc) return -1;
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)RT, (cuuint64_t)n_seq};
    cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)RT * K * 2};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)box_rows, (cuuint32_t)box_seqs};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

}  // namespace

struct TcGemm {
    TcParams p;
    const TileSrc* table = nullptr;
    CUtensorMap map_b_nq[MAX_NQ];   // activation maps with a box of nrs rows x (i+1) sequences
    int nq_max = 1;
    int nrs = 80;                   // rows of a sequence's block that take part: 80 or RT
    int planes = 1;                 // 2: the activation buffer holds a hi and a lo plane, x_seqs blocks apart
};

constexpr int MAX_SLOTS = 4;
size_t tc_gemm_partial_bytes(int n_sm, int nq, int nrs) { return (size_t)n_sm * MAX_SLOTS * nq * nrs * TILE_N * sizeof(float); }
int tc_gemm_max_nq(int nrs, int planes) { return max_nq_of(nrs, planes); }
int tc_gemm_counter_ints() { return 4096; }
size_t tc_gemm_packed_bytes(int epi, const int32_t rows_w[3], int K) {
    const long long total = (long long)rows_w[0] + rows_w[1] + rows_w[2];
    const long long n_tiles = epi == EPI_SWIGLU ? (rows_w[0] + 63) / 64 : (total + TILE_N - 1) / TILE_N;
    return (size_t)(n_tiles * ((K + BK - 1) / BK)) * A_BYTES;
}
int tc_gemm_tiles(const TcGemm* g) { return g ? g->p.n_tiles : 0; }
void tc_gemm_geometry(const TcGemm* g, TcGemmGeom* out) {
    out->n_tiles = g->p.n_tiles; out->KB = g->p.KB; out->grid = g->p.grid; out->slots = g->p.slots;
    out->table = g->table; out->packed = g->p.a_packed; out->partials = g->p.partials; out->nrs = g->nrs;
    out->planes = g->planes; out->plane_seqs = g->p.b_plane_seqs;
    out->map_b = g->map_b_nq[0];
}

int tc_gemm_create(TcGemm** out, int epi, bool defer, const void* const w[3], const int32_t rows_w[3], int K, const void* x,
                   int x_seqs, int nrs, int nq_max, void* partials, size_t partial_bytes, int* counters, int n_sm, int* err, TileSrc* table_dev,
                   int table_entries, void* packed, cudaStream_t stream, int planes) {
    if (!out || (nrs != 80 && nrs != RT) || (planes != 1 && planes != 2) || nq_max < 1 || nq_max > max_nq_of(nrs, planes) ||
        x_seqs < nq_max || K % 8 || n_sm < 1)
        return -1;
    if ((nq_max > 1 || planes > 1) && !defer) return -1;
    if (reinterpret_cast<uintptr_t>(x) % 16) return -1;
    TcGemm* g = new (std::nothrow) TcGemm();
    if (!g) return -1;
    memset(&g->p, 0, sizeof(g->p));
    TcParams& p = g->p;
    int total_rows = 0;
    for (int i = 0; i < 3; ++i) {
        p.rows_w[i] = rows_w[i];
        if (w[i] && rows_w[i] > 0) {
            if (reinterpret_cast<uintptr_t>(w[i]) % 16 || make_map(&p.map_a[i], w[i], rows_w[i], K, 64)) { delete g; return -1; }
            total_rows += rows_w[i];
        } else if (i > 0) {
            p.map_a[i] = p.map_a[0];
        }
    }
    for (int i = 0; i < nq_max; ++i)
        if (make_map_b(&g->map_b_nq[i], x, planes * x_seqs, K, nrs, i + 1)) { delete g; return -1; }
    g->nq_max = nq_max;
    g->nrs = nrs;
    g->planes = planes;
    p.b_plane_seqs = x_seqs;
    p.map_b = g->map_b_nq[0];
    p.map_swiglu = epi == EPI_SWIGLU;
    p.epi = defer ? (int)EPI_PARTIAL : epi;
    p.n_tiles = epi == EPI_SWIGLU ? (rows_w[0] + 63) / 64 : (total_rows + TILE_N - 1) / TILE_N;
    p.KB = (K + BK - 1) / BK;
    const long long U = (long long)p.n_tiles * p.KB;
    p.grid = (int)(U < n_sm ? U : n_sm);
    if (p.n_tiles > tc_gemm_counter_ints() || tc_gemm_partial_bytes(p.grid, nq_max, nrs) > partial_bytes) { delete g; return -1; }
    // fused epilogues store only the head and tail pieces of a range (2 slots); partial-only output stores every
    // piece, one slot per tile the range touches
    p.slots = 2;
    if (p.epi == EPI_PARTIAL) {
        int most = 1;
        for (int c = 0; c < p.grid; ++c) {
            const long long a0 = sk_begin(c, U, p.grid), a1 = sk_begin(c + 1, U, p.grid);
            const int n = (int)((a1 - 1) / p.KB - a0 / p.KB) + 1;
            most = n > most ? n : most;
        }
        if (most > MAX_SLOTS) { delete g; return -1; }
        p.slots = most < 2 ? 2 : most;
        // contributor table for the consumer kernels
        if (!table_dev || p.n_tiles > table_entries) { delete g; return -1; }
        StreamK k;
        k.partials = nullptr; k.table = nullptr; k.n_tiles = p.n_tiles; k.KB = p.KB; k.G = p.grid; k.slots = p.slots; k.rows = nrs; k.seq_rows = nrs;
        TileSrc* tab = new (std::nothrow) TileSrc[p.n_tiles];
        if (!tab) { delete g; return -1; }
        bool fits = true;
        for (int t = 0; t < p.n_tiles && fits; ++t) {
            int c0, c1;
            sk_contributors(k, t, c0, c1);
            if (c1 - c0 + 1 > 15 || (c1 * p.slots + p.slots) > 65535) { fits = false; break; }
            memset(&tab[t], 0, sizeof(TileSrc));
            tab[t].n = (uint16_t)(c1 - c0 + 1);
            for (int c = c0; c <= c1; ++c) tab[t].idx[c - c0] = (uint16_t)(c * p.slots + sk_slot(k, c, t));
        }
        // stream-ordered after the caller's clearing of the workspace; pageable source: staged before the call returns
        if (fits && cudaMemcpyAsync(table_dev, tab, sizeof(TileSrc) * p.n_tiles, cudaMemcpyHostToDevice, stream) != cudaSuccess) fits = false;
        if (fits && cudaStreamSynchronize(stream) != cudaSuccess) fits = false;
        delete[] tab;
        if (!fits) { delete g; return -1; }
        g->table = table_dev;
    }
    if (packed) {
        PackArgs pa;
        for (int i = 0; i < 3; ++i) { pa.w[i] = reinterpret_cast<const __nv_bfloat16*>(w[i]); pa.rows_w[i] = rows_w[i]; }
        pa.K = K; pa.KB = p.KB; pa.map_swiglu = p.map_swiglu;
        k_pack_weights<<<(unsigned)U, 128, 0, stream>>>(pa, reinterpret_cast<unsigned char*>(packed));
        if (cudaGetLastError() != cudaSuccess) { delete g; return -1; }
        p.a_packed = reinterpret_cast<const unsigned char*>(packed);
    }
    p.partials = reinterpret_cast<float*>(partials);
    p.counters = counters;
    p.err = err;
    *out = g;
    return 0;
}

void tc_gemm_destroy(TcGemm* g) { delete g; }

// A wait that nothing completes: exercises the time bound of mbar_wait without disturbing the device.
__global__ void k_wait_selftest(int* err) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(&bar, 0, &abort_flag)) set_error(err, DEV_E_WAIT_TIMEOUT);
    }
}
int tc_wait_selftest(int* err_dev, cudaStream_t s) {
    k_wait_selftest<<<1, 32, 0, s>>>(err_dev);
    return cudaGetLastError() == cudaSuccess ? 0 : -1;
}

StreamK tc_gemm_streamk(const TcGemm* g, int nq) {
    StreamK k;
    k.seq_rows = g ? g->nrs : 80;
    k.rows = nq * k.seq_rows;
    k.partials = g ? g->p.partials : nullptr;
    k.table = g ? g->table : nullptr;
    k.n_tiles = g ? g->p.n_tiles : 0;
    k.KB = g ? g->p.KB : 1;
    k.G = g ? g->p.grid : 1;
    k.slots = g ? g->p.slots : 2;
    return k;
}

// nq sequences starting at sequence b_seq0 of the plan's activation buffer
int tc_gemm_launch(const TcGemm* g, const EpiArgs& a, cudaStream_t s, bool pdl, int nq, int b_seq0) {
    if (!g || nq < 1 || nq > g->nq_max || b_seq0 < 0) return ESP_E_ARG;
    if (nq > 1 && g->p.epi != EPI_PARTIAL) return ESP_E_ARG;
    TcParams p = g->p;
    p.a = a;
    p.map_b = g->map_b_nq[nq - 1];
    p.b_seq0 = b_seq0;
    cudaError_t e = cudaSuccess;
#define ESP_TC_CASE(E, Q, N, PLN)                                                                                  \
    {                                                                                                              \
        if (ensure_dynamic_smem(reinterpret_cast<const void*>(k_gemm_tc<E, Q, N, PLN>), (int)smem_bytes_of(E, Q, N, PLN))) return ESP_E_CUDA; \
        e = launch_k(k_gemm_tc<E, Q, N, PLN>, dim3(p.grid), dim3(NUM_THREADS), smem_bytes_of(E, Q, N, PLN), s, pdl, p); \
    }
    const bool wide = g->nrs != 80;
    if (g->planes == 2) {
        if (p.epi != EPI_PARTIAL) return ESP_E_ARG;
        if (!wide && nq == 1) ESP_TC_CASE(EPI_PARTIAL, 1, 80, 2)
        else if (!wide && nq == 2) ESP_TC_CASE(EPI_PARTIAL, 2, 80, 2)
        else if (wide && nq == 1) ESP_TC_CASE(EPI_PARTIAL, 1, RT, 2)
        else return ESP_E_ARG;
    }
    else if (p.epi == EPI_STORE_F32 && !wide) ESP_TC_CASE(EPI_STORE_F32, 1, 80, 1)
    else if (p.epi == EPI_STORE_F32) ESP_TC_CASE(EPI_STORE_F32, 1, RT, 1)
    else if (p.epi == EPI_LOGITS && !wide) ESP_TC_CASE(EPI_LOGITS, 1, 80, 1)
    else if (p.epi == EPI_LOGITS) ESP_TC_CASE(EPI_LOGITS, 1, RT, 1)
    else if (p.epi == EPI_PARTIAL && !wide && nq == 1) ESP_TC_CASE(EPI_PARTIAL, 1, 80, 1)
    else if (p.epi == EPI_PARTIAL && !wide && nq == 2) ESP_TC_CASE(EPI_PARTIAL, 2, 80, 1)
    else if (p.epi == EPI_PARTIAL && !wide && nq == 3) ESP_TC_CASE(EPI_PARTIAL, 3, 80, 1)
    else if (p.epi == EPI_PARTIAL && wide && nq == 1) ESP_TC_CASE(EPI_PARTIAL, 1, RT, 1)
    else if (p.epi == EPI_PARTIAL && wide && nq == 2) ESP_TC_CASE(EPI_PARTIAL, 2, RT, 1)
    else return ESP_E_ARG;
#undef ESP_TC_CASE
    return e == cudaSuccess ? ESP_OK : ESP_E_CUDA;
}

}  // namespace esp
