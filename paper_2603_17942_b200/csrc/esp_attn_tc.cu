// Tree attention for bf16, head_dim 128, on the Blackwell tensor cores.
//
// A row at position P = L + depth attends to cache positions 0..P.  Positions
// below T0 = floor((P - dcap)/16)*16 are always cache resident, whatever the
// tree looks like; they are summed by the "bulk" kernel here.  The remaining
// <= dcap+16 positions -- the end of the cache and the row's in-flight tree
// ancestors, found through its ancestor bitmask -- are summed key by key in
// position order by the tail+merge kernel, which also merges the bulk
// partials (split order, tail last) and writes the output.  Every reduction
// order is a function of absolute positions only, so a token verified inside a
// tree block gets the bits it would get decoded alone.
//
// Bulk kernel (k_attn_bulk_tc): one CTA per (split of the cache, KV head, tile
// of 128 (row, query head) pairs).  The KV cache of the split is streamed once
// through shared memory by TMA in chunks of 128 keys and shared by all pairs:
//   S = Q K^T   tcgen05.mma, Q (128 pairs x 128 dims) and the K chunk both
//               K-major in shared memory, S (128 x 128 fp32) in tensor memory;
//   softmax     256 threads, two per pair (= tensor-memory lane): mask by the
//               row's T0, running max / sum in the log2 domain, P as bf16 into
//               shared memory in the A-operand layout;
//   O += P V    tcgen05.mma with V as the MN-major B operand (the cache keeps
//               values as [key][dim]); O (128 x 128 fp32) stays in tensor
//               memory and is rescaled there when the running max moves.
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 softmax (two threads per pair, 64 keys each).  S and the
// K/V stages are double buffered, so Q K^T of chunk c+1 overlaps the softmax of
// chunk c.  Every mbarrier wait is bounded; on a timeout the kernel records
// DEV_E_WAIT_TIMEOUT, frees its tensor memory and returns.
#include <new>
#include <string.h>

#include "esp_launch.h"
#include "esp_tc.cuh"

namespace esp {

namespace {

using namespace tc;

constexpr int HD = 128;
constexpr int CK = 128;                   // keys per chunk
constexpr int MP = 128;                   // (row, head) pairs per CTA
constexpr int HALF_BYTES = 128 * 128;     // one 128-row x 64-element (128-byte) swizzled tile
constexpr int Q_BYTES = 2 * HALF_BYTES, K_BYTES = 2 * HALF_BYTES, V_BYTES = 2 * HALF_BYTES, P_BYTES = 2 * HALF_BYTES;
constexpr int KV_STAGE = K_BYTES + V_BYTES;
constexpr int STG_BYTES = 4 * 32 * 128;     // output staging: 32 rows x 128 bytes for each of the 4 output warps
constexpr int OFF_Q = 0, OFF_KV = Q_BYTES, OFF_P = OFF_KV + 2 * KV_STAGE, OFF_STG = OFF_P + P_BYTES, OFF_BAR = OFF_STG + STG_BYTES;
constexpr size_t SMEM_BYTES = 1024 + OFF_BAR + 256;
constexpr int TMEM_COLS = 512;            // S0 at 0, S1 at 128, O0 at 256, O1 at 384
constexpr int MAX_T0_ENTRIES = 256;       // sequences x row tiles one launch may cover
constexpr int NUM_THREADS = 448;           // producer warp, MMA warp, 8 softmax warps, 4 output warps

struct BulkParams {
    CUtensorMap map_q;   // [batch*RT][Hq][128], box 64 x group x rows_per_tile
    CUtensorMap map_k;   // [batch*Hkv*cap][128], box 64 x 128 keys
    CUtensorMap map_v;
    AttnArgs a;
    int32_t group, rows_per_tile, n_row_tiles;
    int32_t n_splits, n_seq, seq0;   // work items of this launch: n_splits x KV heads x row tiles x sequences [seq0, seq0 + n_seq)
};

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

// ---- one item per CTA (grid = splits x (KV heads x row tiles) x sequences): used when the launch has at most
// about one and a half items per SM, where start-up latency is all that counts.
constexpr int ONCE_THREADS = 320;          // producer warp, MMA warp, 8 softmax warps (they also write the output)
constexpr int ONCE_OFF_BAR = OFF_P + P_BYTES;
constexpr size_t ONCE_SMEM_BYTES = 1024 + ONCE_OFF_BAR + 256;

// The producer thread waits for the kernel before this one and only then releases the kernel after it.
__device__ __forceinline__ void trigger_after_wait() {
    pdl_wait();
    pdl_launch_dependents();
}

__global__ void __launch_bounds__(ONCE_THREADS, 1) k_attn_bulk_tc_once(const __grid_constant__ BulkParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ int s_T0max;
    __shared__ float s_xchg[2][2 * MP];   // [exchange parity][half][pair]
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* kv_full = reinterpret_cast<uint64_t*>(smem + ONCE_OFF_BAR);   // [2]
    uint64_t* kv_empty = kv_full + 2;                                  // [2]
    uint64_t* s_full = kv_empty + 2;                                   // [2]
    uint64_t* q_full = s_full + 2;
    uint64_t* p_ready = q_full + 1;
    uint64_t* pv_done = p_ready + 1;
    uint64_t* xchg = pv_done + 1;                                      // the two threads of a pair exchanged a value
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(xchg + 1);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

    const AttnArgs& a = p.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x;
    const int kvh = blockIdx.y / p.n_row_tiles, rtile = blockIdx.y % p.n_row_tiles;
    const int seq = blockIdx.z;

    // Read before pdl_wait(): the sequence state and the cache below T0, both written by earlier steps.
    // The tail kernel is released only after this kernel's wait has returned (trigger_after_wait), so that it may
    // work on this step's queries and keys while the CTAs here are still running.
    int n_rows, L;
    if (a.st) {
        const SeqState* st = a.st + seq;
        n_rows = st->active ? st->n_rows : 0;
        L = st->L;
    } else {
        n_rows = a.n_rows_fixed;
        L = a.L_fixed;
    }
    const int row0 = rtile * p.rows_per_tile;
    if (row0 >= n_rows) { pdl_wait(); return; }
    if (warp == 2) {
        int t0 = 0;
        for (int r = row0 + lane; r < row0 + p.rows_per_tile && r < n_rows; r += 32) {
            const int depth = a.st ? a.st[seq].row_depth[r] : a.depth[seq * RT + r];
            t0 = max(t0, tail_start_tc(L + depth, a.dcap));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t0 = max(t0, __shfl_xor_sync(0xffffffffu, t0, o));
        if (lane == 0) s_T0max = t0;
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], 1); mbar_init(&s_full[i], 1); }
        mbar_init(q_full, 1);
        mbar_init(p_ready, 256);
        mbar_init(pv_done, 1);
        mbar_init(xchg, 256);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int T0max = s_T0max;
    const int n_bulk = (T0max + a.split_len - 1) / a.split_len;
    if (split >= n_bulk) { pdl_wait(); return; }     // block-uniform: nobody holds tensor memory yet
    const int beg = split * a.split_len;
    const int end = min(beg + a.split_len, T0max);
    const int n_chunks = (end - beg + CK - 1) / CK;

    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *s_tmem;
    unsigned char* sQ = smem + OFF_Q;
    unsigned char* sP = smem + OFF_P;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            const int kvrow0 = (seq * a.Hkv + kvh) * a.cap + beg;
            bool ok = true;
            auto load_chunk = [&](int c) {
                unsigned char* st = smem + OFF_KV + (c & 1) * KV_STAGE;
                mbar_expect_tx(&kv_full[c & 1], KV_STAGE);
                tma_load_2d(st, &p.map_k, 0, kvrow0 + c * CK, &kv_full[c & 1]);
                tma_load_2d(st + HALF_BYTES, &p.map_k, 64, kvrow0 + c * CK, &kv_full[c & 1]);
                tma_load_2d(st + K_BYTES, &p.map_v, 0, kvrow0 + c * CK, &kv_full[c & 1]);
                tma_load_2d(st + K_BYTES + HALF_BYTES, &p.map_v, 64, kvrow0 + c * CK, &kv_full[c & 1]);
            };
            // the cache below T0 is settled in a decode step: request it before waiting for the kernel that wrote the queries
            if (a.cache_in_flight) trigger_after_wait();
            for (int c = 0; c < n_chunks && c < 2; ++c) load_chunk(c);
            if (!a.cache_in_flight) trigger_after_wait();
            mbar_expect_tx(q_full, Q_BYTES);
            tma_load_3d(sQ, &p.map_q, 0, kvh * p.group, seq * RT + row0, q_full);
            tma_load_3d(sQ + HALF_BYTES, &p.map_q, 64, kvh * p.group, seq * RT + row0, q_full);
            for (int c = 2; c < n_chunks && ok; ++c) {
                if (!mbar_wait(&kv_empty[c & 1], ((c >> 1) & 1) ^ 1, s_abort)) { ok = false; break; }
                load_chunk(c);
            }
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
                umma_commit(&s_full[c & 1]);
            };
            ok = mbar_wait(q_full, 0, s_abort) && mbar_wait(&kv_full[0], 0, s_abort);
            if (ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_qk(0);
            }
            for (int c = 0; c < n_chunks && ok; ++c) {
                if (c + 1 < n_chunks) {     // S of the next chunk while the softmax of this one runs
                    if (!mbar_wait(&kv_full[(c + 1) & 1], ((c + 1) >> 1) & 1, s_abort)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    issue_qk(c + 1);
                }
                if (!mbar_wait(p_ready, c & 1, s_abort)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t v_addr = smem_u32(smem + OFF_KV + (c & 1) * KV_STAGE + K_BYTES);
#pragma unroll
                for (int kk = 0; kk < CK / 16; ++kk) {
                    const uint32_t p_off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;     // P: K-major over keys
                    const uint32_t v_off = kk * 16 * 128;                              // V: 16 key rows of 128 bytes further
                    umma(tmem_base + 256, smem_desc(p_addr + p_off, 16), smem_desc(v_addr + v_off, HALF_BYTES), IDESC_PV,
                         (c > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(pv_done);
                umma_commit(&kv_empty[c & 1]);
            }
            if (!ok) { set_error(a.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else {
        // ---------------- softmax warps 2..9: a thread owns one pair (= tensor-memory lane) and one half of the
        // chunk's 128 keys (warps 2-5 keys 0..63, warps 6-9 keys 64..127); the two threads of a pair exchange
        // their maxima (per chunk) and their sums (at the end) through shared memory
        const int q4 = warp & 3;
        const int hf = (warp - 2) >> 2;
        const int pair = q4 * 32 + lane;
        const int r = row0 + pair / p.group, head = kvh * p.group + pair % p.group;
        const bool pv = pair / p.group < p.rows_per_tile && r < n_rows && r < RT;
        int T0row = 0;
        if (pv) T0row = tail_start_tc(L + (a.st ? a.st[seq].row_depth[r] : a.depth[seq * RT + r]), a.dcap);
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16) + hf * 64;   // this thread's 64 columns of S / O
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int c = 0; c < n_chunks && ok; ++c) {
            // (a wait that fails must take the whole warp out: the tensor-memory accesses below are warp-wide)
            if (!__all_sync(0xffffffffu, mbar_wait(&s_full[c & 1], (c >> 1) & 1, s_abort))) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t s_addr = lane_addr + (c & 1) * 128;
            const int cbase = beg + c * CK + hf * 64;
            // the row's scores for this half, masked to its visible keys and scaled to the log2 domain
            uint32_t sv[64];
            tmem_ld64(s_addr, sv);
            float cmax = -INFINITY;
            if (__all_sync(0xffffffffu, cbase + 64 <= T0row)) {     // every key of the half is visible to every row of the warp
#pragma unroll
                for (int i = 0; i < 64; ++i) {
                    const float sc = __uint_as_float(sv[i]) * a.scale_log2;
                    sv[i] = __float_as_uint(sc);
                    cmax = fmaxf(cmax, sc);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 64; ++i) {
                    const float sc = cbase + i < T0row ? __uint_as_float(sv[i]) * a.scale_log2 : -INFINITY;
                    sv[i] = __float_as_uint(sc);
                    cmax = fmaxf(cmax, sc);
                }
            }
            // the chunk maximum over both halves
            // (double buffered by exchange parity: a thread can be one exchange ahead of its partner, not two)
            s_xchg[c & 1][hf * MP + pair] = cmax;
            mbar_arrive(xchg);
            if (!__all_sync(0xffffffffu, mbar_wait(xchg, c & 1, s_abort))) { ok = false; break; }
            cmax = fmaxf(s_xchg[c & 1][pair], s_xchg[c & 1][MP + pair]);
            const float m_new = fmaxf(m_run, cmax);
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            const float alpha = exp2f(m_run - m_use);
            // P of the previous chunk must have been consumed before it is overwritten, and O must be final
            // before it is rescaled
            if (c > 0 && !__all_sync(0xffffffffu, mbar_wait(pv_done, (c - 1) & 1, s_abort))) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // probabilities, their sum (key order), P as bf16 in the A-operand layout (this half = one swizzled tile)
            float csum = 0.f;
            unsigned char* prow = sP + hf * HALF_BYTES + pair * 128;
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = exp2f(__uint_as_float(sv[blk * 32 + i]) - m_use), p1 = exp2f(__uint_as_float(sv[blk * 32 + i + 1]) - m_use);
                    csum += p0;
                    csum += p1;
                    const __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
                    pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&b2);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk16 = blk * 4 + j;
                    *reinterpret_cast<uint4*>(prow + ((chunk16 ^ (pair & 7)) << 4)) = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                }
            }
            if (c > 0) {
                // O <- alpha * O (in tensor memory), this thread's 64 of the 128 columns
                if (__any_sync(0xffffffffu, alpha != 1.0f)) {   // warp-uniform: skip when no lane's maximum moved
                    tmem_ld64(lane_addr + 256, sv);
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) sv[blk * 32 + i] = __float_as_uint(__uint_as_float(sv[blk * 32 + i]) * alpha);
                        tmem_st32(lane_addr + 256 + blk * 32, *reinterpret_cast<const uint32_t(*)[32]>(&sv[blk * 32]));
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                }
            }
            l_run = l_run * alpha + csum;     // this half's share of the row sum
            m_run = m_new;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P: generic-proxy writes -> tensor-core reads
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(p_ready);
        }
        if (ok && !__all_sync(0xffffffffu, mbar_wait(pv_done, (n_chunks - 1) & 1, s_abort))) ok = false;
        if (ok) {
            // the row sum = first half's share + second half's share
            s_xchg[n_chunks & 1][hf * MP + pair] = l_run;
            mbar_arrive(xchg);
            if (!__all_sync(0xffffffffu, mbar_wait(xchg, n_chunks & 1, s_abort))) ok = false;
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
                const size_t idx = ((size_t)(seq * RT + r) * a.Hq + head) * a.n_split_max + split;
                if (hf == 0) a.part_ml[idx] = make_float2(m_run, s_xchg[n_chunks & 1][pair] + s_xchg[n_chunks & 1][MP + pair]);
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
    // ---------------- teardown (every thread arrives here)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (*s_abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);   // let copies in flight land before shared memory goes away
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- persistent CTAs: used when the launch has clearly more items than SMs.
// One work item = (split of the cache, KV head, row tile, sequence); what a role needs to know about it.
struct Item {
    int split, kvh, rtile, seq, row0, n_rows, L, beg, n_chunks;
};

__global__ void __launch_bounds__(NUM_THREADS, 1) k_attn_bulk_tc(const __grid_constant__ BulkParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ int s_T0[MAX_T0_ENTRIES];  // [sequence][row tile]: largest T0 among the tile's rows
    __shared__ int2 s_seq[MAX_T0_ENTRIES];  // [sequence]: (rows in its block, cached positions L)
    __shared__ float s_xchg[2][2 * MP];   // [exchange parity][half][pair]
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* kv_full = reinterpret_cast<uint64_t*>(smem + OFF_BAR);   // [2]
    uint64_t* kv_empty = kv_full + 2;                                  // [2]
    uint64_t* s_full = kv_empty + 2;                                   // [2]
    uint64_t* o_free = s_full + 2;                                     // [2] an O accumulator has been read out
    uint64_t* o_full = o_free + 2;                                     // [2] an item's last P V has completed
    uint64_t* q_full = o_full + 2;
    uint64_t* q_free = q_full + 1;                                     // the item's last Q K^T has completed
    uint64_t* p_ready = q_free + 1;
    uint64_t* pv_done = p_ready + 1;
    uint64_t* xchg = pv_done + 1;                                      // the two threads of a pair exchanged a value
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(xchg + 1);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

    const AttnArgs& a = p.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Read before pdl_wait(): the sequence state and the cache below T0, both written by earlier steps.
    // The dependent kernel is released by the producer thread once its wait has returned (trigger_after_wait).
    for (int e = warp; e < p.n_seq * p.n_row_tiles; e += NUM_THREADS / 32) {   // one warp per entry, a lane per row
        const int seq = p.seq0 + e / p.n_row_tiles, row0 = (e % p.n_row_tiles) * p.rows_per_tile;
        int n_rows, L;
        if (a.st) { n_rows = a.st[seq].active ? a.st[seq].n_rows : 0; L = a.st[seq].L; }
        else { n_rows = a.n_rows_fixed; L = a.L_fixed; }
        int t0 = 0;
        for (int r = row0 + lane; r < row0 + p.rows_per_tile && r < n_rows; r += 32)
            t0 = max(t0, tail_start_tc(L + (a.st ? a.st[seq].row_depth[r] : a.depth[seq * RT + r]), a.dcap));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t0 = max(t0, __shfl_xor_sync(0xffffffffu, t0, o));
        if (lane == 0) {
            s_T0[e] = t0;
            if (e % p.n_row_tiles == 0) s_seq[e / p.n_row_tiles] = make_int2(n_rows, L);
        }
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], 1); mbar_init(&s_full[i], 1); mbar_init(&o_free[i], 128);
            mbar_init(&o_full[i], 1);
        }
        mbar_init(q_full, 1);
        mbar_init(q_free, 1);
        mbar_init(p_ready, 256);
        mbar_init(pv_done, 1);
        mbar_init(xchg, 256);
        *s_abort = 0;
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
    unsigned char* sQ = smem + OFF_Q;
    unsigned char* sP = smem + OFF_P;

    // Items are dealt round-robin; every role walks the same list and skips the same empty items, so the
    // per-chunk and per-item counters below advance identically in all of them.
    const int n_items = p.n_splits * a.Hkv * p.n_row_tiles * p.n_seq;
    auto get_item = [&](int idx, Item& it) -> bool {
        it.split = idx % p.n_splits;
        int y = idx / p.n_splits;
        it.rtile = y % p.n_row_tiles;
        y /= p.n_row_tiles;
        it.kvh = y % a.Hkv;
        const int lseq = y / a.Hkv;
        it.seq = p.seq0 + lseq;
        it.n_rows = s_seq[lseq].x;
        it.L = s_seq[lseq].y;
        it.row0 = it.rtile * p.rows_per_tile;
        if (it.row0 >= it.n_rows) return false;
        const int T0max = s_T0[lseq * p.n_row_tiles + it.rtile];
        it.beg = it.split * a.split_len;
        if (it.beg >= T0max) return false;
        const int end = min(it.beg + a.split_len, T0max);
        it.n_chunks = (end - it.beg + CK - 1) / CK;
        return true;
    };

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            bool ok = true, first = true;
            uint32_t gc = 0, n_it = 0;       // chunks and items issued so far
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                Item it;
                if (!get_item(idx, it)) continue;
                const int kvrow0 = (it.seq * a.Hkv + it.kvh) * a.cap + it.beg;
                auto load_chunk = [&](int c) -> bool {
                    const uint32_t g = gc + c;
                    // a fresh barrier passes a wait on parity 1: the first use of a stage does not block
                    if (!mbar_wait(&kv_empty[g & 1], ((g >> 1) & 1) ^ 1, s_abort)) return false;
                    unsigned char* st = smem + OFF_KV + (g & 1) * KV_STAGE;
                    mbar_expect_tx(&kv_full[g & 1], KV_STAGE);
                    tma_load_2d(st, &p.map_k, 0, kvrow0 + c * CK, &kv_full[g & 1]);
                    tma_load_2d(st + HALF_BYTES, &p.map_k, 64, kvrow0 + c * CK, &kv_full[g & 1]);
                    tma_load_2d(st + K_BYTES, &p.map_v, 0, kvrow0 + c * CK, &kv_full[g & 1]);
                    tma_load_2d(st + K_BYTES + HALF_BYTES, &p.map_v, 64, kvrow0 + c * CK, &kv_full[g & 1]);
                    return true;
                };
                int c0 = 0;
                if (first) {
                    // the cache does not depend on the kernel before this one, the queries do
                    if (a.cache_in_flight) trigger_after_wait();
                    for (; c0 < it.n_chunks && c0 < 2 && ok; ++c0) ok = load_chunk(c0);
                    if (!a.cache_in_flight) trigger_after_wait();
                    first = false;
                } else {
                    // Q is single buffered: the previous item's last Q K^T must have completed
                    ok = mbar_wait(q_free, (n_it - 1) & 1, s_abort);
                }
                if (!ok) break;
                mbar_expect_tx(q_full, Q_BYTES);
                tma_load_3d(sQ, &p.map_q, 0, it.kvh * p.group, it.seq * RT + it.row0, q_full);
                tma_load_3d(sQ + HALF_BYTES, &p.map_q, 64, it.kvh * p.group, it.seq * RT + it.row0, q_full);
                for (int c = c0; c < it.n_chunks && ok; ++c) ok = load_chunk(c);
                gc += it.n_chunks;
                ++n_it;
            }
            if (first) trigger_after_wait();
            if (!ok) { set_error(a.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            bool ok = true;
            uint32_t gc = 0, n_it = 0;
            const uint32_t q_addr = smem_u32(sQ), p_addr = smem_u32(sP);
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                Item it;
                if (!get_item(idx, it)) continue;
                const uint32_t tmem_o = tmem_base + 256 + (n_it & 1) * 128;
                auto issue_qk = [&](int c) {
                    const uint32_t g = gc + c;
                    const uint32_t k_addr = smem_u32(smem + OFF_KV + (g & 1) * KV_STAGE);
                    const uint32_t tmem_s = tmem_base + (g & 1) * 128;
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                        umma(tmem_s, smem_desc(q_addr + off, 16), smem_desc(k_addr + off, 16), IDESC_QK, kk > 0 ? 1u : 0u);
                    }
                    umma_commit(&s_full[g & 1]);
                    if (c == it.n_chunks - 1) umma_commit(q_free);
                };
                ok = mbar_wait(q_full, n_it & 1, s_abort) && mbar_wait(&kv_full[gc & 1], (gc >> 1) & 1, s_abort) &&
                     mbar_wait(&o_free[n_it & 1], ((n_it >> 1) & 1) ^ 1, s_abort);   // this O buffer's previous item was read out
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_qk(0);
                for (int c = 0; c < it.n_chunks && ok; ++c) {
                    const uint32_t g = gc + c;
                    if (c + 1 < it.n_chunks) {     // S of the next chunk while the softmax of this one runs
                        if (!mbar_wait(&kv_full[(g + 1) & 1], ((g + 1) >> 1) & 1, s_abort)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        issue_qk(c + 1);
                    }
                    if (!mbar_wait(p_ready, g & 1, s_abort)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t v_addr = smem_u32(smem + OFF_KV + (g & 1) * KV_STAGE + K_BYTES);
#pragma unroll
                    for (int kk = 0; kk < CK / 16; ++kk) {
                        const uint32_t p_off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;     // P: K-major over keys
                        const uint32_t v_off = kk * 16 * 128;                              // V: 16 key rows of 128 bytes further
                        umma(tmem_o, smem_desc(p_addr + p_off, 16), smem_desc(v_addr + v_off, HALF_BYTES), IDESC_PV,
                             (c > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(pv_done);
                    umma_commit(&kv_empty[g & 1]);
                    if (c == it.n_chunks - 1) umma_commit(&o_full[n_it & 1]);
                }
                gc += it.n_chunks;
                ++n_it;
            }
            if (!ok) { set_error(a.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else if (warp < 10) {
        // ---------------- softmax warps 2..9: a thread owns one pair (= tensor-memory lane) and one half of the
        // chunk's 128 keys (warps 2-5 keys 0..63, warps 6-9 keys 64..127); the two threads of a pair exchange
        // their maxima (per chunk) and their sums (at the end of an item) through shared memory
        const int q4 = warp & 3;
        const int hf = (warp - 2) >> 2;
        const int pair = q4 * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16) + hf * 64;   // this thread's 64 columns of S / O
        uint32_t gc = 0, n_it = 0, xc = 0;   // chunks, items, exchanges so far
        bool ok = true;
        for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
            Item it;
            if (!get_item(idx, it)) continue;
            const int r = it.row0 + pair / p.group, head = it.kvh * p.group + pair % p.group;
            const bool pv = pair / p.group < p.rows_per_tile && r < it.n_rows && r < RT;
            int T0row = 0;
            if (pv) T0row = tail_start_tc(it.L + (a.st ? a.st[it.seq].row_depth[r] : a.depth[it.seq * RT + r]), a.dcap);
            const uint32_t o_addr = lane_addr + 256 + (n_it & 1) * 128;
            float m_run = -INFINITY, l_run = 0.f;
            for (int c = 0; c < it.n_chunks && ok; ++c) {
                const uint32_t g = gc + c;
                // (a wait that fails must take the whole warp out: the tensor-memory accesses below are warp-wide)
                if (!__all_sync(0xffffffffu, mbar_wait(&s_full[g & 1], (g >> 1) & 1, s_abort))) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t s_addr = lane_addr + (g & 1) * 128;
                const int cbase = it.beg + c * CK + hf * 64;
                // the row's scores for this half, masked to its visible keys and scaled to the log2 domain
                uint32_t sv[64];
                tmem_ld64(s_addr, sv);
                float cmax = -INFINITY;
                if (__all_sync(0xffffffffu, cbase + 64 <= T0row)) {     // every key of the half is visible to every row of the warp
#pragma unroll
                    for (int i = 0; i < 64; ++i) {
                        const float sc = __uint_as_float(sv[i]) * a.scale_log2;
                        sv[i] = __float_as_uint(sc);
                        cmax = fmaxf(cmax, sc);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 64; ++i) {
                        const float sc = cbase + i < T0row ? __uint_as_float(sv[i]) * a.scale_log2 : -INFINITY;
                        sv[i] = __float_as_uint(sc);
                        cmax = fmaxf(cmax, sc);
                    }
                }
                // the chunk maximum over both halves
                // (double buffered by exchange parity: a thread can be one exchange ahead of its partner, not two)
                s_xchg[xc & 1][hf * MP + pair] = cmax;
                mbar_arrive(xchg);
                if (!__all_sync(0xffffffffu, mbar_wait(xchg, xc & 1, s_abort))) { ok = false; break; }
                cmax = fmaxf(s_xchg[xc & 1][pair], s_xchg[xc & 1][MP + pair]);
                ++xc;
                const float m_new = fmaxf(m_run, cmax);
                const float m_use = m_new == -INFINITY ? 0.f : m_new;
                const float alpha = exp2f(m_run - m_use);
                // P of the previous chunk must have been consumed before it is overwritten, and O must be final
                // before it is rescaled
                if (g > 0 && !__all_sync(0xffffffffu, mbar_wait(pv_done, (g - 1) & 1, s_abort))) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // probabilities, their sum (key order), P as bf16 in the A-operand layout (this half = one swizzled tile)
                float csum = 0.f;
                unsigned char* prow = sP + hf * HALF_BYTES + pair * 128;
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float p0 = exp2f(__uint_as_float(sv[blk * 32 + i]) - m_use), p1 = exp2f(__uint_as_float(sv[blk * 32 + i + 1]) - m_use);
                        csum += p0;
                        csum += p1;
                        const __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
                        pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&b2);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int chunk16 = blk * 4 + j;
                        *reinterpret_cast<uint4*>(prow + ((chunk16 ^ (pair & 7)) << 4)) = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                    }
                }
                if (c > 0) {
                    // O <- alpha * O (in tensor memory), this thread's 64 of the 128 columns
                    if (__any_sync(0xffffffffu, alpha != 1.0f)) {   // warp-uniform: skip when no lane's maximum moved
                        tmem_ld64(o_addr, sv);
#pragma unroll
                        for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) sv[blk * 32 + i] = __float_as_uint(__uint_as_float(sv[blk * 32 + i]) * alpha);
                            tmem_st32(o_addr + blk * 32, *reinterpret_cast<const uint32_t(*)[32]>(&sv[blk * 32]));
                        }
                        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    }
                }
                l_run = l_run * alpha + csum;     // this half's share of the row sum
                m_run = m_new;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P: generic-proxy writes -> tensor-core reads
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                mbar_arrive(p_ready);
            }
            if (!ok) break;
            gc += it.n_chunks;
            // the row sum = first half's share + second half's share; the output warps take care of O
            s_xchg[xc & 1][hf * MP + pair] = l_run;
            mbar_arrive(xchg);
            if (!__all_sync(0xffffffffu, mbar_wait(xchg, xc & 1, s_abort))) { ok = false; break; }
            const float l_tot = s_xchg[xc & 1][pair] + s_xchg[xc & 1][MP + pair];
            ++xc;
            if (pv && hf == 0) a.part_ml[((size_t)(it.seq * RT + r) * a.Hq + head) * a.n_split_max + it.split] = make_float2(m_run, l_tot);
            ++n_it;
        }
        if (!ok && lane == 0) {
            set_error(a.err, DEV_E_WAIT_TIMEOUT);
            *s_abort = 1;
        }
    } else {
        // ---------------- output warps 10..13: when an item's last P V has completed, its O accumulator goes tensor
        // memory -> registers -> (transposed through 4 KB of shared memory per warp) -> global, so that every store
        // instruction writes whole 128-byte lines, while the softmax warps are already on the next item.  The
        // tensor-memory loads are warp-wide: every lane takes part.
        const int q4 = warp & 3;
        const uint32_t lane_o = tmem_base + ((uint32_t)(q4 * 32) << 16) + 256;
        unsigned char* stg = smem + OFF_STG + (warp - 10) * (32 * 128);
        uint32_t n_it = 0;
        bool ok = true;
        for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
            Item it;
            if (!get_item(idx, it)) continue;
            const int b = n_it & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(&o_full[b], (n_it >> 1) & 1, s_abort))) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // where the 8 rows this lane stores per pass go (-1: no such pair)
            const int j = lane & 7;
            long long obase[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int pr = q4 * 32 + i * 4 + (lane >> 3);
                const int r2 = it.row0 + pr / p.group, head2 = it.kvh * p.group + pr % p.group;
                const bool valid = pr / p.group < p.rows_per_tile && r2 < it.n_rows && r2 < RT;
                obase[i] = valid ? (long long)((((size_t)(it.seq * RT + r2) * a.Hq + head2) * a.n_split_max + it.split) * HD + j * 4) : -1;
            }
#pragma unroll 1
            for (int t = 0; t < 4; ++t) {
                uint32_t ov[32];
                tmem_ld32(lane_o + b * 128 + t * 32, ov);
                if (t == 3) {   // the accumulator is in registers: hand it back to the MMA warp
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    mbar_arrive(&o_free[b]);
                }
#pragma unroll
                for (int jj = 0; jj < 8; ++jj)
                    *reinterpret_cast<uint4*>(stg + lane * 128 + ((jj ^ (lane & 7)) << 4)) =
                        make_uint4(ov[4 * jj], ov[4 * jj + 1], ov[4 * jj + 2], ov[4 * jj + 3]);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = i * 4 + (lane >> 3);                      // pair within the warp
                    if (obase[i] >= 0) {
                        const uint4 val = *reinterpret_cast<const uint4*>(stg + rr * 128 + ((j ^ (rr & 7)) << 4));
                        __stcg(reinterpret_cast<uint4*>(a.part_o + obase[i] + t * 32), val);
                    }
                }
                __syncwarp();
            }
            ++n_it;
        }
        if (!ok && lane == 0) {
            set_error(a.err, DEV_E_WAIT_TIMEOUT);
            *s_abort = 1;
        }
    }
    // ---------------- teardown (every thread arrives here)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (*s_abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);   // let copies in flight land before shared memory goes away
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
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

// The tail: positions T0..P in position order, lane j owns key j of a 32-key chunk (chunk grid anchored at T0).
// Then the merge: bulk partials in split order, the tail last; a lane owns 4 of the 128 output dims.
// TAIL_FIRST: launched behind a bulk kernel with programmatic dependent launch (see below).  LEAN: smaller load
// batches and 64 registers, eight CTAs per SM, for grids of many waves where occupancy counts for more than one
// warp's latency.  All instances add in the same order and give the same bits.
template <bool TAIL_FIRST, bool LEAN>
__global__ void __launch_bounds__(128, LEAN ? 8 : (TAIL_FIRST ? 5 : 4)) k_attn_tail_merge_tc(AttnArgs a) {
    constexpr int KB8 = LEAN ? 8 : HD / 8;      // 16-byte pieces of a key row loaded before they are used
    constexpr int VB = LEAN ? 8 : 16;           // value rows loaded before they are used
    constexpr int PB = LEAN ? 4 : 8;            // split partials loaded before they are merged
    __shared__ float s_qall[4][HD];
    if (threadIdx.x == 0) pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 4 + warp, head = blockIdx.y, seq = blockIdx.z;
    // the sequence state was written by an earlier step; everything else is read after the wait
    int n_rows, L, depth = 0;
    unsigned long long lo = 0, hi = 0;
    if (a.st) {
        const SeqState* st = a.st + seq;
        n_rows = st->active ? st->n_rows : 0;
        L = st->L;
        if (r < n_rows) { depth = st->row_depth[r]; lo = st->row_anc[r][0]; hi = st->row_anc[r][1]; }
    } else {
        n_rows = a.n_rows_fixed;
        L = a.L_fixed;
        if (r < n_rows) { depth = a.depth[seq * RT + r]; lo = a.anc[(size_t)(seq * RT + r) * 2]; hi = a.anc[(size_t)(seq * RT + r) * 2 + 1]; }
    }
    // After a bulk launch this kernel starts once every bulk CTA's wait has returned: the kernel that wrote this
    // step's queries, keys and values has completed by then, and the tail may be computed while the bulk CTAs run.
    // (Nothing reads those buffers through L1 between that kernel's writes and this point: the bulk kernels fetch
    // them by TMA, so no SM can hold a line of them from before the writes.)
    if (!TAIL_FIRST) pdl_wait();
    if (r >= n_rows) { pdl_wait(); return; }
    const int kvh = head / (a.Hq / a.Hkv);
    const int P = L + depth, T0 = tail_start_tc(P, a.dcap);
    const __nv_bfloat16* kbase = reinterpret_cast<const __nv_bfloat16*>(a.kc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    const __nv_bfloat16* vbase = reinterpret_cast<const __nv_bfloat16*>(a.vc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((size_t)(seq * RT + r) * a.Hq + head) * HD;
    float* s_q = s_qall[warp];
    {
        const uint2 qq = *reinterpret_cast<const uint2*>(q + lane * 4);
        const __nv_bfloat162 q01 = *reinterpret_cast<const __nv_bfloat162*>(&qq.x), q23 = *reinterpret_cast<const __nv_bfloat162*>(&qq.y);
        s_q[lane * 4 + 0] = __low2float(q01); s_q[lane * 4 + 1] = __high2float(q01);
        s_q[lane * 4 + 2] = __low2float(q23); s_q[lane * 4 + 3] = __high2float(q23);
    }
    __syncwarp();
    const int n_sp = (T0 + a.split_len - 1) / a.split_len;
    const size_t base = ((size_t)(seq * RT + r) * a.Hq + head) * a.n_split_max;
    float2 ml0[PB];
    float4 c40[PB];
    auto request_partials = [&]() {     // the first bulk partials
#pragma unroll
        for (int u = 0; u < PB; ++u) {
            if (u < n_sp) {
                ml0[u] = __ldcg(a.part_ml + base + u);
                c40[u] = __ldcg(reinterpret_cast<const float4*>(a.part_o + (base + u) * HD + lane * 4));
            }
        }
    };
    if (!TAIL_FIRST) request_partials();      // in flight while the tail is computed
    // ---- tail
    float tm = -INFINITY, tl = 0.f, to[4] = {0.f, 0.f, 0.f, 0.f};
    const int n_tail = P - T0 + 1;
    for (int t0 = 0; t0 < n_tail; t0 += 32) {
        const int t = t0 + lane;
        bool valid = t < n_tail;
        int slot = 0;
        if (valid) {
            const int pos = T0 + t;
            if (pos < L) slot = pos;
            else {
                const int b = nth_set_bit128(lo, hi, pos - L);
                if (b < 0) { set_error(a.err, DEV_E_INDEX); valid = false; }
                else slot = L + b;
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
            for (int d8 = 0; d8 < KB8; ++d8) kreg[d8] = kr[dh + d8];
#pragma unroll
            for (int d8 = dh; d8 < dh + KB8; ++d8) {
                const uint4 kk = kreg[d8 - dh];
                const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kk);
                const float4 qa = *reinterpret_cast<const float4*>(s_q + d8 * 8), qb = *reinterpret_cast<const float4*>(s_q + d8 * 8 + 4);
                acc = fmaf(qa.x, __low2float(k2[0]), acc); acc = fmaf(qa.y, __high2float(k2[0]), acc);
                acc = fmaf(qa.z, __low2float(k2[1]), acc); acc = fmaf(qa.w, __high2float(k2[1]), acc);
                acc = fmaf(qb.x, __low2float(k2[2]), acc); acc = fmaf(qb.y, __high2float(k2[2]), acc);
                acc = fmaf(qb.z, __low2float(k2[3]), acc); acc = fmaf(qb.w, __high2float(k2[3]), acc);
            }
            }
            sc = acc * a.scale_log2;
        }
        float cm = sc;
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, of));
        const float pe = valid ? exp2f(sc - cm) : 0.f;
        float cl = pe;
#pragma unroll
        for (int of = 16; of > 0; of >>= 1) cl += __shfl_xor_sync(0xffffffffu, cl, of);
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
                vv[u] = *reinterpret_cast<const uint2*>(vbase + (size_t)sj * HD + lane * 4);
            }
#pragma unroll
            for (int u = 0; u < VB; ++u) {
                if (pj[u] != 0.f) {
                    const __nv_bfloat162 v01 = *reinterpret_cast<const __nv_bfloat162*>(&vv[u].x), v23 = *reinterpret_cast<const __nv_bfloat162*>(&vv[u].y);
                    co[0] = fmaf(pj[u], __low2float(v01), co[0]); co[1] = fmaf(pj[u], __high2float(v01), co[1]);
                    co[2] = fmaf(pj[u], __low2float(v23), co[2]); co[3] = fmaf(pj[u], __high2float(v23), co[3]);
                }
            }
        }
        merge_ml(tm, tl, to, cm, cl, co);
    }
    // ---- merge: splits in order, then the tail
    if (TAIL_FIRST) { pdl_wait(); request_partials(); }
    float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < PB; ++u) {
        if (u < n_sp) {
            const float co[4] = {c40[u].x, c40[u].y, c40[u].z, c40[u].w};
            merge_ml(m, l, o, ml0[u].x, ml0[u].y, co);
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
    merge_ml(m, l, o, tm, tl, to);
    const float inv = 1.0f / l;
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out) + ((size_t)(seq * RT + r) * a.Hq + head) * HD + lane * 4;
    const __nv_bfloat162 o01 = __floats2bfloat162_rn(o[0] * inv, o[1] * inv), o23 = __floats2bfloat162_rn(o[2] * inv, o[3] * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&o01);
    pk.y = *reinterpret_cast<const uint32_t*>(&o23);
    *reinterpret_cast<uint2*>(out) = pk;
}

}  // namespace

struct AttnTc {
    BulkParams p;
};

bool attn_tc_supported(int h, int Hq, int Hkv) {
    if (h != HD || Hkv < 1 || Hq % Hkv) return false;
    const int group = Hq / Hkv;
    return group <= MP && MP % group == 0 && group <= 256;
}

// TMA descriptors of one layer's query buffer [batch*RT][Hq][128] and KV cache [batch*Hkv*cap][128] (bf16).
int attn_tc_create(AttnTc** out, const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap) {
    if (!out || !attn_tc_supported(HD, Hq, Hkv)) return -1;
    EncodeFn enc = get_encode();
    if (!enc) return -1;
    AttnTc* t = new (std::nothrow) AttnTc();
    if (!t) return -1;
    memset(&t->p, 0, sizeof(t->p));
    const int group = Hq / Hkv, rows_per_tile = MP / group;
    t->p.group = group;
    t->p.rows_per_tile = rows_per_tile;
    t->p.n_row_tiles = (RT + rows_per_tile - 1) / rows_per_tile;
    const cuuint32_t estr3[3] = {1, 1, 1};
    {
        cuuint64_t dims[3] = {(cuuint64_t)HD, (cuuint64_t)Hq, (cuuint64_t)batch * RT};
        cuuint64_t strides[2] = {(cuuint64_t)HD * 2, (cuuint64_t)Hq * HD * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)group, (cuuint32_t)rows_per_tile};
        if (enc(&t->p.map_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, estr3,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { delete t; return -1; }
    }
    for (int i = 0; i < 2; ++i) {
        cuuint64_t dims[2] = {(cuuint64_t)HD, (cuuint64_t)batch * Hkv * cap};
        cuuint64_t strides[1] = {(cuuint64_t)HD * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)CK};
        if (enc(i ? &t->p.map_v : &t->p.map_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(i ? vcache : kcache), dims,
                strides, box, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { delete t; return -1; }
    }
    *out = t;
    return 0;
}

void attn_tc_destroy(AttnTc* t) { delete t; }

// Two launches: the bulk kernel (grid = splits x (KV heads x row tiles) x sequences), then tail + merge.
int attn_tc_launch(const AttnTc* t, const AttnArgs& a, int batch, int n_split_launch, cudaStream_t s, bool pdl) {
    if (!t || n_split_launch + 1 > a.n_split_max || a.split_len % CK) return -1;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_attn_bulk_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess) return -1;
        attr_set = true;
    }
    BulkParams p = t->p;
    p.a = a;
    const int rows_cap = a.rows_cap > 0 && a.rows_cap < RT ? a.rows_cap : RT;
    p.n_row_tiles = (rows_cap + p.rows_per_tile - 1) / p.rows_per_tile;   // row tiles that can hold rows
    if (n_split_launch > 0) {
        static int n_sm = 0;
        if (n_sm == 0) {
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1) {
                n_sm = 0;
                return -1;
            }
        }
        const long long all_items = (long long)n_split_launch * a.Hkv * p.n_row_tiles * batch;
        if (all_items <= n_sm + n_sm / 2) {
            // (nearly) every CTA runs once: one item per CTA.  Measured crossover: the persistent kernel wins from
            // about 1.2 waves when timed alone, a little later inside a step, where its larger register and
            // shared-memory footprint delays its start behind the kernel before it
            static bool once_attr = false;
            if (!once_attr) {
                if (cudaFuncSetAttribute(k_attn_bulk_tc_once, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ONCE_SMEM_BYTES) != cudaSuccess) return -1;
                once_attr = true;
            }
            dim3 grid(n_split_launch, a.Hkv * p.n_row_tiles, batch);
            if (launch_k(k_attn_bulk_tc_once, grid, dim3(ONCE_THREADS), ONCE_SMEM_BYTES, s, pdl, p) != cudaSuccess) return -1;
        } else {
            // persistent CTAs, one per SM, walk the (split, KV head, row tile, sequence) items round-robin
            const int per_launch = MAX_T0_ENTRIES / p.n_row_tiles;
            for (int s0 = 0; s0 < batch; s0 += per_launch) {
                p.seq0 = s0;
                p.n_seq = batch - s0 < per_launch ? batch - s0 : per_launch;
                p.n_splits = n_split_launch;
                const long long items = (long long)p.n_splits * a.Hkv * p.n_row_tiles * p.n_seq;
                const int grid = (int)(items < n_sm ? items : n_sm);
                if (launch_k(k_attn_bulk_tc, dim3(grid), dim3(NUM_THREADS), SMEM_BYTES, s, pdl, p) != cudaSuccess) return -1;
            }
        }
    }
    // the bulk kernels release their dependent after their own wait: behind them the tail is computed first
    // (plain launches run one after the other: there the partials are requested before the tail instead)
    const dim3 tgrid((rows_cap + 3) / 4, a.Hq, batch);
    // several waves of CTAs launched on their own: the lean instance (measured: 333 against 368 us for 16
    // sequences of 4k positions; inside a step, where the tail overlaps the bulk kernel, it is the slower one)
    const bool many = !pdl && (long long)tgrid.x * tgrid.y * tgrid.z > 8 * 148;
    const cudaError_t e = n_split_launch > 0 && many ? launch_k(k_attn_tail_merge_tc<true, true>, tgrid, dim3(128), 0, s, pdl, a)
                          : n_split_launch > 0 && pdl ? launch_k(k_attn_tail_merge_tc<true, false>, tgrid, dim3(128), 0, s, pdl, a)
                                                      : launch_k(k_attn_tail_merge_tc<false, false>, tgrid, dim3(128), 0, s, pdl, a);
    if (e != cudaSuccess) return -1;
    return 0;
}

}  // namespace esp
