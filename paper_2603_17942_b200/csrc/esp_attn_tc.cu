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
//               memory; the softmax reference follows the running max lazily
//               (it moves, and O is rescaled, only after a growth of 2^8).
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 softmax (two threads per pair, 64 keys each).  S and the
// K/V stages are double buffered, so Q K^T of chunk c+1 overlaps the softmax of
// chunk c; a stage's K half is released by its Q K^T and its V half by its P V,
// and the producer keeps K one chunk ahead of V.  Every mbarrier wait is bounded;
// on a timeout the kernel records DEV_E_WAIT_TIMEOUT, frees its tensor memory
// and returns.
#include <new>
#include <string.h>

#include "esp_attn_tc.cuh"

namespace esp {

namespace {

using namespace tc;
using namespace attn;

constexpr int STG_BYTES = 4 * 32 * 128;     // output staging: 32 rows x 128 bytes for each of the 4 output warps
constexpr int OFF_STG = OFF_P + P_BYTES, OFF_BAR = OFF_STG + STG_BYTES;
constexpr size_t SMEM_BYTES = 1024 + OFF_BAR + 256;
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

// ---- one item per CTA (grid = splits x (KV heads x row tiles) x sequences): used when the launch has at most
// about one and a half items per SM, where start-up latency is all that counts.
constexpr int ONCE_THREADS = 320;          // producer warp, MMA warp, 8 softmax warps (they also write the output)
constexpr int ONCE_OFF_BAR = ITEM_BYTES;
constexpr size_t ONCE_SMEM_BYTES = 1024 + ONCE_OFF_BAR + 256;

__global__ void __launch_bounds__(ONCE_THREADS, 1) k_attn_bulk_tc_once(const __grid_constant__ BulkParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ int s_T0max;
    __shared__ float s_xchg[2][2 * MP];   // [exchange parity][half][pair]
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    BulkShared sm;
    sm.buf = smem;
    sm.k_full = reinterpret_cast<uint64_t*>(smem + ONCE_OFF_BAR);    // [2]
    sm.k_empty = sm.k_full + 2;                                      // [2]
    sm.v_full = sm.k_empty + 2;                                      // [2]
    sm.v_empty = sm.v_full + 2;                                      // [2]
    sm.s_full = sm.v_empty + 2;                                      // [2]
    sm.q_full = sm.s_full + 2;
    sm.p_ready = sm.q_full + 1;
    sm.pv_done = sm.p_ready + 1;
    sm.xchg = sm.pv_done + 1;                                        // [4] the two threads of a pair exchanged a value
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm.xchg + 4);
    sm.s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
    sm.s_xchg = &s_xchg[0][0];

    const AttnArgs& a = p.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    BulkItem it;
    it.split = blockIdx.x;
    it.kvh = blockIdx.y / p.n_row_tiles;
    const int rtile = blockIdx.y % p.n_row_tiles;
    it.seq = blockIdx.z;

    // Read before pdl_wait(): the sequence state and the cache below T0, both written by earlier steps.
    // The tail kernel is released only after this kernel's wait has returned (trigger_after_wait), so that it may
    // work on this step's queries and keys while the CTAs here are still running.
    if (a.st) {
        const SeqState* st = a.st + it.seq;
        it.n_rows = st->active ? st->n_rows : 0;
        it.L = st->L;
    } else {
        it.n_rows = a.n_rows_fixed;
        it.L = a.L_fixed;
    }
    it.row0 = rtile * p.rows_per_tile;
    if (it.row0 >= it.n_rows) { pdl_wait(); return; }
    if (warp == 2) {
        int t0 = 0;
        for (int r = it.row0 + lane; r < it.row0 + p.rows_per_tile && r < it.n_rows; r += 32) {
            const int depth = a.st ? a.st[it.seq].row_depth[r] : a.depth[it.seq * RT + r];
            t0 = max(t0, tail_start_tc(it.L + depth, a.dcap));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t0 = max(t0, __shfl_xor_sync(0xffffffffu, t0, o));
        if (lane == 0) s_T0max = t0;
    }
    if (threadIdx.x == 0) {
        prefetch_tensormap(&p.map_k);
        prefetch_tensormap(&p.map_v);
        prefetch_tensormap(&p.map_q);
        bulk_init_barriers(sm);
        *sm.s_abort = 0;
    }
    __syncthreads();
    const int T0max = s_T0max;
    const int n_bulk = (T0max + a.split_len - 1) / a.split_len;
    if (it.split >= n_bulk) { pdl_wait(); return; }     // block-uniform: nobody holds tensor memory yet
    it.beg = it.split * a.split_len;
    const int end = min(it.beg + a.split_len, T0max);
    it.n_chunks = (end - it.beg + CK - 1) / CK;
    it.kv_row0 = (it.seq * a.Hkv + it.kvh) * a.cap;

    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *s_tmem;
    BulkMaps mp;
    mp.q = &p.map_q; mp.k = &p.map_k; mp.v = &p.map_v; mp.group = p.group; mp.rows_per_tile = p.rows_per_tile;
    bulk_item_roles<true>(mp, a, it, sm, tmem_base, warp, lane);
    // ---------------- teardown (every thread arrives here)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (*sm.s_abort) {
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
    uint64_t* k_full = reinterpret_cast<uint64_t*>(smem + OFF_BAR);    // [2] a stage's K half has landed
    uint64_t* k_empty = k_full + 2;                                    // [2] ... its Q K^T has completed
    uint64_t* v_full = k_empty + 2;                                    // [2] a stage's V half has landed
    uint64_t* v_empty = v_full + 2;                                    // [2] ... its P V has completed
    uint64_t* s_full = v_empty + 2;                                    // [2]
    uint64_t* o_free = s_full + 2;                                     // [2] an O accumulator has been read out
    uint64_t* o_full = o_free + 2;                                     // [2] an item's last P V has completed
    uint64_t* q_full = o_full + 2;
    uint64_t* q_free = q_full + 1;                                     // the item's last Q K^T has completed
    uint64_t* p_ready = q_free + 1;
    uint64_t* pv_done = p_ready + 1;
    uint64_t* xchg = pv_done + 1;                                      // [4] the two threads of a pair exchanged a value (per lane quadrant)
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(xchg + 4);
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
        prefetch_tensormap(&p.map_k);
        prefetch_tensormap(&p.map_v);
        prefetch_tensormap(&p.map_q);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1); mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
            mbar_init(&s_full[i], 1); mbar_init(&o_free[i], 128);
            mbar_init(&o_full[i], 1);
        }
        mbar_init(q_full, 1);
        mbar_init(q_free, 1);
        mbar_init(p_ready, 8);
        mbar_init(pv_done, 1);
        for (int i = 0; i < 4; ++i) mbar_init(&xchg[i], 2);
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
            // Two cursors walk the CTA's chunks (item after item): K, which also requests an item's Q, and V.  A K
            // half is free again when its Q K^T has completed, about a chunk period before the V half (free when
            // P V has), so K runs one chunk ahead of V and both have two chunk periods for their trip from HBM.
            struct Cursor { int idx, c; uint32_t g; bool live; Item it; };
            auto seek = [&](Cursor& k, int from) {
                k.live = false;
                for (int idx = from; idx < n_items; idx += gridDim.x)
                    if (get_item(idx, k.it)) { k.idx = idx; k.c = 0; k.live = true; return; }
            };
            auto advance = [&](Cursor& k) {
                ++k.g;
                if (++k.c == k.it.n_chunks) seek(k, k.idx + gridDim.x);
            };
            auto load_half = [&](const Cursor& k, bool is_k) -> bool {
                uint64_t* empty = is_k ? k_empty : v_empty;
                uint64_t* full = is_k ? k_full : v_full;
                // a fresh barrier passes a wait on parity 1: the first use of a stage does not block
                if (!mbar_wait(&empty[k.g & 1], ((k.g >> 1) & 1) ^ 1, s_abort)) return false;
                const int row = (k.it.seq * a.Hkv + k.it.kvh) * a.cap + k.it.beg + k.c * CK;
                unsigned char* st = smem + OFF_KV + (k.g & 1) * KV_STAGE + (is_k ? 0 : K_BYTES);
                const CUtensorMap* map = is_k ? &p.map_k : &p.map_v;
                mbar_expect_tx(&full[k.g & 1], K_BYTES);
                tma_load_2d(st, map, 0, row, &full[k.g & 1]);
                tma_load_2d(st + HALF_BYTES, map, 64, row, &full[k.g & 1]);
                return true;
            };
            auto load_q = [&](const Item& it) {
                mbar_expect_tx(q_full, Q_BYTES);
                tma_load_3d(sQ, &p.map_q, 0, it.kvh * p.group, it.seq * RT + it.row0, q_full);
                tma_load_3d(sQ + HALF_BYTES, &p.map_q, 64, it.kvh * p.group, it.seq * RT + it.row0, q_full);
            };
            bool ok = true;
            uint32_t n_q = 0;                // items whose Q has been requested
            Cursor ck, cv;
            ck.g = 0;
            seek(ck, blockIdx.x);
            cv = ck;
            if (!ck.live) {
                trigger_after_wait();
            } else {
                // the first item: the cache does not depend on the kernel before this one, the queries do
                const Item it0 = ck.it;
                if (a.cache_in_flight) trigger_after_wait();
                const int pre = it0.n_chunks < 2 ? 1 : 2;
                for (int i = 0; i < pre && ok; ++i) { ok = load_half(ck, true); advance(ck); }
                for (int i = 0; i < pre && ok; ++i) { ok = load_half(cv, false); advance(cv); }
                if (!a.cache_in_flight) trigger_after_wait();
                load_q(it0);
                n_q = 1;
                auto k_step = [&]() -> bool {
                    if (!ck.live) return true;
                    if (ck.c == 0) {
                        // Q is single buffered: the previous item's last Q K^T must have completed
                        if (!mbar_wait(q_free, (n_q - 1) & 1, s_abort)) return false;
                        load_q(ck.it);
                        ++n_q;
                    }
                    const bool done = load_half(ck, true);
                    advance(ck);
                    return done;
                };
                ok = ok && k_step();                      // K one chunk ahead of V from here on
                while (ok && cv.live) {
                    ok = k_step();
                    if (!ok) break;
                    ok = load_half(cv, false);
                    advance(cv);
                }
            }
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
                    umma_commit(&k_empty[g & 1]);
                    if (c == it.n_chunks - 1) umma_commit(q_free);
                };
                ok = mbar_wait(q_full, n_it & 1, s_abort) && mbar_wait(&k_full[gc & 1], (gc >> 1) & 1, s_abort) &&
                     mbar_wait(&o_free[n_it & 1], ((n_it >> 1) & 1) ^ 1, s_abort);   // this O buffer's previous item was read out
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                issue_qk(0);
                for (int c = 0; c < it.n_chunks && ok; ++c) {
                    const uint32_t g = gc + c;
                    if (c + 1 < it.n_chunks) {     // S of the next chunk while the softmax of this one runs
                        if (!mbar_wait(&k_full[(g + 1) & 1], ((g + 1) >> 1) & 1, s_abort)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        issue_qk(c + 1);
                    }
                    if (!mbar_wait(p_ready, g & 1, s_abort) || !mbar_wait(&v_full[g & 1], (g >> 1) & 1, s_abort)) { ok = false; break; }
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
                    umma_commit(&v_empty[g & 1]);
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
                ok = softmax_chunk(lane_addr + (g & 1) * 128, o_addr, it.beg + c * CK + hf * 64, T0row, a.scale_log2, m_run, l_run,
                                   &s_xchg[xc & 1][0], xchg + q4, xc & 1, g > 0, pv_done, (g - 1) & 1, c > 0,
                                   sP + hf * HALF_BYTES + pair * 128, pair, hf, p_ready, s_abort);
                ++xc;
            }
            if (!ok) break;
            gc += it.n_chunks;
            // the row sum = first half's share + second half's share; the output warps take care of O
            s_xchg[xc & 1][hf * MP + pair] = l_run;
            __syncwarp();
            if (lane == 0) mbar_arrive(xchg + q4);
            if (!__all_sync(0xffffffffu, mbar_wait(xchg + q4, xc & 1, s_abort))) { ok = false; break; }
            const float l_tot = __fadd_rn(s_xchg[xc & 1][pair], s_xchg[xc & 1][MP + pair]);
            ++xc;
            if (pv && hf == 0) __stcg(a.part_ml + ((size_t)(it.seq * RT + r) * a.Hq + head) * a.n_split_max + it.split, make_float2(m_run, l_tot));
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
// ---- tail + merge: one warp per (row, head) pair (tail_pair, merge_pair).
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
    PairCtx c;
    c.r = blockIdx.x * 4 + warp; c.head = blockIdx.y; c.seq = blockIdx.z;
    c.depth = 0; c.lo = 0; c.hi = 0;
    // the sequence state was written by an earlier step; everything else is read after the wait
    int n_rows;
    if (a.st) {
        const SeqState* st = a.st + c.seq;
        n_rows = st->active ? st->n_rows : 0;
        c.L = st->L;
        if (c.r < n_rows) { c.depth = st->row_depth[c.r]; c.lo = st->row_anc[c.r][0]; c.hi = st->row_anc[c.r][1]; }
    } else {
        n_rows = a.n_rows_fixed;
        c.L = a.L_fixed;
        if (c.r < n_rows) { c.depth = a.depth[c.seq * RT + c.r]; c.lo = a.anc[(size_t)(c.seq * RT + c.r) * 2]; c.hi = a.anc[(size_t)(c.seq * RT + c.r) * 2 + 1]; }
    }
    // After a bulk launch this kernel starts once every bulk CTA's wait has returned: the kernel that wrote this
    // step's queries, keys and values has completed by then, and the tail may be computed while the bulk CTAs run.
    // The tail reads those buffers with L2 loads only, so no stale line of an SM's L1 can be seen.
    if (!TAIL_FIRST) pdl_wait();
    if (c.r >= n_rows) { pdl_wait(); return; }
    FirstPartials<PB> fp;
    if (!TAIL_FIRST) request_partials<PB>(fp, a, c, lane);      // in flight while the tail is computed
    TailAcc t;
    tail_pair<KB8, VB>(t, a, c, s_qall[warp], lane);
    if (TAIL_FIRST) { pdl_wait(); request_partials<PB>(fp, a, c, lane); }
    merge_pair<PB>(fp, t, a, c, lane);
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
static int attn_tc_fill(AttnTc* t, const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap);

int attn_tc_create(AttnTc** out, const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap) {
    if (!out) return -1;
    AttnTc* t = new (std::nothrow) AttnTc();
    if (!t) return -1;
    if (attn_tc_fill(t, q, kcache, vcache, batch, Hq, Hkv, cap)) { delete t; return -1; }
    *out = t;
    return 0;
}

// One attention with the descriptors built in this call's own frame: nothing is allocated, on the host or the device.
int attn_tc_run(const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap, const AttnArgs& a,
                int n_split_launch, cudaStream_t s) {
    AttnTc t;
    if (attn_tc_fill(&t, q, kcache, vcache, batch, Hq, Hkv, cap)) return -1;
    return attn_tc_launch(&t, a, batch, n_split_launch, s, false);     // the descriptors travel by value
}

static int attn_tc_fill(AttnTc* t, const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap) {
    if (!attn_tc_supported(HD, Hq, Hkv)) return -1;
    EncodeFn enc = get_encode();
    if (!enc) return -1;
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
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return -1;
    }
    for (int i = 0; i < 2; ++i) {
        cuuint64_t dims[2] = {(cuuint64_t)HD, (cuuint64_t)batch * Hkv * cap};
        cuuint64_t strides[1] = {(cuuint64_t)HD * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)CK};
        if (enc(i ? &t->p.map_v : &t->p.map_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(i ? vcache : kcache), dims,
                strides, box, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return -1;
    }
    return 0;
}

void attn_tc_destroy(AttnTc* t) { delete t; }

// Two launches: the bulk kernel (grid = splits x (KV heads x row tiles) x sequences), then tail + merge.
int attn_tc_launch(const AttnTc* t, const AttnArgs& a, int batch, int n_split_launch, cudaStream_t s, bool pdl) {
    if (!t || n_split_launch + 1 > a.n_split_max || a.split_len % CK) return -1;
    BulkParams p = t->p;
    p.a = a;
    const int rows_cap = a.rows_cap > 0 && a.rows_cap < RT ? a.rows_cap : RT;
    p.n_row_tiles = (rows_cap + p.rows_per_tile - 1) / p.rows_per_tile;   // row tiles that can hold rows
    if (n_split_launch > 0) {
        const int n_sm = current_sm_count();
        if (n_sm < 1) return -1;
        const long long all_items = (long long)n_split_launch * a.Hkv * p.n_row_tiles * batch;
        if (all_items <= n_sm + n_sm / 2) {
            // (nearly) every CTA runs once: one item per CTA.  Measured crossover: the persistent kernel wins from
            // about 1.2 waves when timed alone, a little later inside a step, where its larger register and
            // shared-memory footprint delays its start behind the kernel before it
            if (ensure_dynamic_smem(reinterpret_cast<const void*>(k_attn_bulk_tc_once), (int)ONCE_SMEM_BYTES)) return -1;
            dim3 grid(n_split_launch, a.Hkv * p.n_row_tiles, batch);
            if (launch_k(k_attn_bulk_tc_once, grid, dim3(ONCE_THREADS), ONCE_SMEM_BYTES, s, pdl, p) != cudaSuccess) return -1;
        } else {
            // persistent CTAs, one per SM, walk the (split, KV head, row tile, sequence) items round-robin
            if (ensure_dynamic_smem(reinterpret_cast<const void*>(k_attn_bulk_tc), (int)SMEM_BYTES)) return -1;
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
