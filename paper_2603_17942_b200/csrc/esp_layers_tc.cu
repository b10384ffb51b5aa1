// All decoder layers of one decode-and-verify step in ONE persistent launch (bf16, head_dim 128, blocks of at
// most 80 rows, one sequence per pass).
//
// The step is bound by streaming the weights once from HBM.  With one kernel per operation a layer is ten
// launches, and around every boundary the weight stream stops: a GEMM's ring ramps up, its CTAs finish a few
// microseconds apart, the consumer of its partials starts, ends, and the next GEMM ramps up again.  Here one CTA
// per SM stays resident for all layers (cooperative launch) and walks the same phases in order:
//
//   norm -> QKV GEMM -> q/k/v finish (RoPE, cache write) -> attention over the cache (tcgen05) ->
//   attention tail + merge -> O GEMM -> residual + norm -> gate/up GEMM -> SiLU*up -> down GEMM -> next layer
//
// separated by grid-wide barriers.  The producer warp keeps the ring of repacked weight units running across
// the phases: the units of the next GEMM are requested as soon as ring slots free up, while the epilogue of the
// current GEMM, the barrier and the small phase in between are still running; only the activation tiles wait for
// the barrier.  Tensor memory, the ring's barriers and the descriptors are set up once per step.
//
// Every phase is the device function the one-operation-per-launch kernels run (esp_consumers.cuh,
// esp_attn_tc.cuh), the stream-K partition of each GEMM is the same, and every sum has the same order: the
// two paths give the same bits, and a row has the same bits alone (greedy decoding) and inside a tree block.
//
// Waits: every mbarrier wait and every grid barrier is bounded by wall time.  A wait that runs out records
// DEV_E_WAIT_TIMEOUT; the other CTAs see the error word in their own waits and leave too; every CTA lets its
// copies land, frees its tensor memory and returns.
#include <new>
#include <stddef.h>
#include <string.h>

#include "esp_attn_tc.cuh"
#include "esp_consumers.cuh"
#include "esp_gemm_tc.cuh"

namespace esp {

namespace {

using namespace tc;

constexpr int STAGES = 6;
constexpr int NRS = 80;                                  // rows of the block that take part in the GEMMs
constexpr int PLANES = 2;                                // the activations arrive as hi + lo bf16 pairs (see esp_gemm_tc.cu)
constexpr int B_PLANE = NRS * BK * 2;                    // 10240
constexpr int B_BYTES = PLANES * B_PLANE;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;           // 36864, a multiple of 1024
constexpr int RING_BYTES = STAGES * STAGE_BYTES;         // 221184; the attention phase reuses it (attn::ITEM_BYTES fit)
constexpr int ACC_COLS = 256;                            // two accumulators: W x_hi in columns [0, 80), W x_lo in [80, 160); attention: S0, S1, O
constexpr int NUM_THREADS = 448;                         // producer warp, MMA warp, 12 consumer warps
constexpr int CONS_WARPS = 12;
constexpr int CONS_THREADS = CONS_WARPS * 32;
constexpr uint32_t IDESC = idesc_of(PLANES * NRS);     // hi and lo rows form one B operand of 160 rows
static_assert(attn::ITEM_BYTES <= RING_BYTES, "the attention item must fit into the ring");

enum { G_QKV = 0, G_O = 1, G_GU = 2, G_DOWN = 3 };

struct GemmDesc {
    int32_t n_tiles, KB, G, slots;
    unsigned long long pk_off;     // of this GEMM's units inside a layer's block of repacked weights
    const TileSrc* table;
};

struct LayersParams {
    CUtensorMap map_b[4];          // activations of the four GEMMs: [plane][sequence][RT][K], box 64 x 80 x 1
    int32_t b_plane_seqs;          // blocks between the hi and the lo plane
    CUtensorMap map_q, map_k, map_v;   // attention: query buffer; K and V cache of ALL layers as [rows][128]
    GemmDesc g[4];
    const unsigned char* packed;   // layer 0's repacked weights
    unsigned long long pk_layer;   // bytes per layer
    float* partials;
    // per-sequence state and activations (the pass's sequence uses activation block 0)
    const SeqState* st;
    float* hres;
    __nv_bfloat16 *xn, *qbuf, *attn_out, *act;
    __nv_bfloat16 *xn_lo, *attn_out_lo, *act_lo;   // low-order planes
    char *kcache, *vcache;         // layer 0, this sequence
    unsigned long long layer_kv_stride;   // bytes
    const void* const* norm_attn;  // [n_layers] device pointers
    const void* const* norm_ffn;
    const void* const* q_norm;
    const void* const* k_norm;
    const float *rope_cos, *rope_sin;
    int32_t n_layers, d, Hq, Hkv, F, cap, qk_norm;
    float rms_eps;
    // attention
    float* part_o;
    float2* part_ml;
    int32_t split_len, n_split_max, dcap, group, rows_per_tile;
    int32_t kv_rows_layer;         // rows of one layer in the K/V maps (batch * Hkv * cap)
    int32_t kv_row_seq;            // first row of this sequence inside a layer
    float scale_log2;
    // synchronisation
    unsigned int* sync_counter;    // arrivals, counted up launch after launch
    unsigned int sync_base;        // its value before this launch
    int* err;
    unsigned long long* timeline;  // optional: CTA 0 stamps the global timer when it arrives at and when it leaves every grid barrier
};

struct Shared {                    // behind the ring
    uint64_t full[STAGES], empty[STAGES], tfull[2], tempty[2];                         // GEMM ring and accumulators
    uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], q_full, p_ready, pv_done, xchg[4];   // attention item
    uint32_t tmem;
    int abort_flag, T0max, sync_ok;
    alignas(16) float red[128];
    alignas(16) float xch[2][2 * attn::MP];
    alignas(16) float s_q[CONS_WARPS][attn::HD];      // read as float4
};
static_assert(offsetof(Shared, s_q) % 16 == 0 && offsetof(Shared, full) % 8 == 0, "vector and barrier alignment");
constexpr size_t SMEM_BYTES = 1024 + RING_BYTES + sizeof(Shared);
static_assert(SMEM_BYTES <= 227 * 1024, "dynamic shared memory of one CTA");

__device__ __forceinline__ void cons_bar() { asm volatile("bar.sync 1, %0;" ::"n"(CONS_THREADS) : "memory"); }
__device__ __forceinline__ void main_bar() { __syncthreads(); }

// Tracing: with a timeline buffer, CTA 0 stamps the global timer into TRACE_SLOTS words per barrier: [0] its arrival
// at the barrier, [1] its exit, [2..] marks inside the phase that follows (GEMM phases: the activation tiles of
// the ring's first items requested, the first and the last item consumed, the last accumulator stored).
constexpr int TRACE_SLOTS = 8;
__device__ __forceinline__ void trace(const LayersParams& p, int stamp, int slot) {
    if (p.timeline && blockIdx.x == 0) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
        p.timeline[(size_t)stamp * TRACE_SLOTS + slot] = now;
    }
}

// Grid-wide barrier.  Every thread's global writes of the phase before it are visible to every thread of the
// grid after it, to tensor-map (async proxy) loads as well.  false: this CTA or another one gave up.
__device__ __forceinline__ bool grid_sync(const LayersParams& p, Shared& sh, uint32_t& epoch, int& stamp) {
    asm volatile("fence.proxy.async;" ::: "memory");
    main_bar();
    if (threadIdx.x == 0) {
        epoch += gridDim.x;
        const uint32_t target = p.sync_base + epoch;
        bool ok = sh.abort_flag == 0;
        trace(p, stamp, 0);
        if (ok) {
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.sync_counter) : "memory");
            unsigned long long t0 = 0;
            for (uint32_t i = 0;; ++i) {
                uint32_t v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p.sync_counter) : "memory");
                if ((int32_t)(v - target) >= 0) break;
                if ((i & 63u) == 63u) {
                    if (*reinterpret_cast<volatile int*>(p.err) != 0) { ok = false; break; }
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > WAIT_LIMIT_NS) { set_error(p.err, DEV_E_WAIT_TIMEOUT); ok = false; break; }
                }
            }
        }
        if (!ok) sh.abort_flag = 1;
        sh.sync_ok = ok ? 1 : 0;
        trace(p, stamp, 1);
        asm volatile("fence.proxy.async;" ::: "memory");
    }
    ++stamp;
    main_bar();
    return sh.sync_ok != 0;
}

// ---- GEMM roles.  The ring's item counter and the accumulator counter run on across GEMMs and layers.
struct Ring {
    uint32_t it;      // items passed through the ring so far (producer: issued; MMA thread: consumed)
    uint32_t seg;     // accumulators so far (MMA thread and epilogue warps)
    int pre;          // producer: leading items of the next GEMM whose weight unit is already requested
};

__device__ __forceinline__ Range cta_range(const GemmDesc& g, int cta) {
    const long long U = (long long)g.n_tiles * g.KB;
    return make_range(sk_begin(cta, U, g.G), sk_begin(cta + 1, U, g.G), g.KB, g.slots);
}
__device__ __forceinline__ int cta_items(const GemmDesc& g, int cta) {
    const long long U = (long long)g.n_tiles * g.KB;
    return (int)(sk_begin(cta + 1, U, g.G) - sk_begin(cta, U, g.G));
}

// producer thread: request the weight units of the first ring-full of items of GEMM `g` of layer `l`
__device__ __forceinline__ bool prefetch_weights(const LayersParams& p, Shared& sh, unsigned char* ring, Ring& rg, int g, int l,
                                                 uint64_t pol_w) {
    const GemmDesc& gd = p.g[g];
    rg.pre = 0;
    if ((int)blockIdx.x >= gd.G) return true;
    const Range rng = cta_range(gd, blockIdx.x);
    const int n_items = cta_items(gd, blockIdx.x);
    const int n_pre = n_items < STAGES ? n_items : STAGES;
    const unsigned char* base = p.packed + p.pk_layer * l + gd.pk_off;
    int idx = 0;
    for (int i = 0; i < rng.n_seg && idx < n_pre; ++i) {
        const Seg sg = get_seg(rng, i);
        for (int kb = sg.kb0; kb < sg.kb1 && idx < n_pre; ++kb, ++idx) {
            const uint32_t it = rg.it + idx, stage = it % STAGES, par = (it / STAGES) & 1;
            if (!mbar_wait(&sh.empty[stage], par ^ 1, &sh.abort_flag)) return false;
            mbar_expect_tx(&sh.full[stage], STAGE_BYTES);
            bulk_load(ring + stage * STAGE_BYTES, base + ((size_t)sg.tile * gd.KB + kb) * A_BYTES, A_BYTES, &sh.full[stage], pol_w);
        }
    }
    rg.pre = n_pre;
    return true;
}

// producer thread: all items of GEMM `g` of layer `l` (the activation tiles, and the weight units not yet requested)
__device__ __forceinline__ bool produce_gemm(const LayersParams& p, Shared& sh, unsigned char* ring, Ring& rg, int g, int l,
                                             uint64_t pol_w, uint64_t pol_x, int tr) {
    const GemmDesc& gd = p.g[g];
    if ((int)blockIdx.x >= gd.G) return true;
    const Range rng = cta_range(gd, blockIdx.x);
    const unsigned char* base = p.packed + p.pk_layer * l + gd.pk_off;
    int idx = 0;
    for (int i = 0; i < rng.n_seg; ++i) {
        const Seg sg = get_seg(rng, i);
        for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++idx) {
            const uint32_t stage = rg.it % STAGES, par = (rg.it / STAGES) & 1;
            unsigned char* sa = ring + stage * STAGE_BYTES;
            if (idx >= rg.pre) {
                if (!mbar_wait(&sh.empty[stage], par ^ 1, &sh.abort_flag)) return false;
                mbar_expect_tx(&sh.full[stage], STAGE_BYTES);
                bulk_load(sa, base + ((size_t)sg.tile * gd.KB + kb) * A_BYTES, A_BYTES, &sh.full[stage], pol_w);
                }
#pragma unroll
            for (int pl = 0; pl < PLANES; ++pl)
                tma_load_3d_hint(sa + A_BYTES + pl * B_PLANE, &p.map_b[g], kb * BK, 0, pl * p.b_plane_seqs, &sh.full[stage], pol_x);
            ++rg.it;
            if (idx + 1 == rg.pre) trace(p, tr, 2);
        }
    }
    rg.pre = 0;
    return true;
}

// MMA thread
__device__ __forceinline__ bool mma_gemm(const LayersParams& p, Shared& sh, unsigned char* ring, Ring& rg, int g, uint32_t tmem_base, int tr) {
    const GemmDesc& gd = p.g[g];
    if ((int)blockIdx.x >= gd.G) return true;
    const Range rng = cta_range(gd, blockIdx.x);
    for (int i = 0; i < rng.n_seg; ++i, ++rg.seg) {
        const Seg sg = get_seg(rng, i);
        const uint32_t buf = rg.seg & 1;
        if (!mbar_wait(&sh.tempty[buf], ((rg.seg >> 1) & 1) ^ 1, &sh.abort_flag)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + buf * ACC_COLS;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++rg.it) {
            const uint32_t stage = rg.it % STAGES, par = (rg.it / STAGES) & 1;
            if (!mbar_wait(&sh.full[stage], par, &sh.abort_flag)) return false;
            if (i == 0 && kb == sg.kb0) trace(p, tr, 3);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = smem_u32(ring + stage * STAGE_BYTES);
            const uint64_t da = smem_desc(sa, 16), db = smem_desc(sa + A_BYTES, 16);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
                umma(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), IDESC, (kb > sg.kb0 || k > 0) ? 1u : 0u);
            umma_commit(&sh.empty[stage]);
        }
        umma_commit(&sh.tfull[buf]);
    }
    trace(p, tr, 4);
    return true;
}

// epilogue warps 2..5: accumulator -> fp32 partial of the (CTA, slot) piece; false (warp-uniform): a wait ran out
__device__ __forceinline__ bool epilogue_gemm(const LayersParams& p, Shared& sh, Ring& rg, int g, uint32_t tmem_base, int n_rows,
                                              int warp, int lane, int tr) {
    const GemmDesc& gd = p.g[g];
    if ((int)blockIdx.x >= gd.G) return true;
    const Range rng = cta_range(gd, blockIdx.x);
    const int q = warp & 3;                 // tensor-memory lane quarter this warp may read
    const int f = q * 32 + lane;            // feature of the tile owned by this thread
    for (int i = 0; i < rng.n_seg; ++i, ++rg.seg) {
        const Seg sg = get_seg(rng, i);
        const uint32_t buf = rg.seg & 1;
        if (!__all_sync(0xffffffffu, mbar_wait(&sh.tfull[buf], (rg.seg >> 1) & 1, &sh.abort_flag))) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + buf * ACC_COLS + ((uint32_t)(q * 32) << 16);
        uint32_t v[NRS];
#pragma unroll
        for (int c = 0; c < NRS / 16; ++c) tmem_ld16_issue(taddr + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&v[c * 16]));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int c = 0; c < NRS / 16; ++c) {      // + the product with the low-order plane
            uint32_t lo16[16];
            tmem_ld16_issue(taddr + NRS + c * 16, lo16);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 16; ++j) v[c * 16 + j] = __float_as_uint(__fadd_rn(__uint_as_float(v[c * 16 + j]), __uint_as_float(lo16[j])));
        }
        // the accumulator is in registers: hand the tensor-memory buffer back to the MMA thread
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(&sh.tempty[buf]);
        float* part = p.partials + ((size_t)(blockIdx.x * gd.slots + sg.slot) * NRS) * TILE_N + f;
#pragma unroll
        for (int r = 0; r < NRS; ++r)
            if (r < n_rows) __stcg(part + r * TILE_N, __uint_as_float(v[r]));
        if (i == rng.n_seg - 1 && warp == 2 && lane == 0) { trace(p, tr, 5); }
    }
    return true;
}

__device__ __forceinline__ StreamK streamk_of(const LayersParams& p, int g) {
    StreamK k;
    k.partials = p.partials; k.table = p.g[g].table; k.n_tiles = p.g[g].n_tiles; k.KB = p.g[g].KB; k.G = p.g[g].G;
    k.slots = p.g[g].slots; k.rows = NRS; k.seq_rows = NRS;
    return k;
}

__global__ void __launch_bounds__(NUM_THREADS, 1) k_layers_tc(const __grid_constant__ LayersParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Shared& sh = *reinterpret_cast<Shared*>(ring + RING_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int cw = warp - 2;                // consumer warp index (warps 2..13)

    if (threadIdx.x == 0) {
        for (int i = 0; i < 4; ++i) prefetch_tensormap(&p.map_b[i]);
        prefetch_tensormap(&p.map_q);
        prefetch_tensormap(&p.map_k);
        prefetch_tensormap(&p.map_v);
        for (int i = 0; i < STAGES; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&sh.tfull[i], 1); mbar_init(&sh.tempty[i], 128); }
        sh.abort_flag = 0;
        sh.sync_ok = 1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem)), "r"(attn::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem;

    // the block this step runs (row table written by the step before)
    const SeqState* st = p.st;
    const int n_rows = st->active ? (st->n_rows < NRS ? st->n_rows : NRS) : 0;
    const int L = st->L;

    Ring rg;
    rg.it = 0; rg.seg = 0; rg.pre = 0;
    uint32_t epoch = 0;
    int stamp = 0;
    const bool producer = warp == 0 && lane == 0, mma = warp == 1 && lane == 0;
    uint64_t pol_w = 0, pol_x = 0;
    if (producer) {
        pol_w = l2_policy_evict_first();
        pol_x = l2_policy_evict_last();
        if (!prefetch_weights(p, sh, ring, rg, G_QKV, 0, pol_w)) { set_error(p.err, DEV_E_WAIT_TIMEOUT); sh.abort_flag = 1; }
    }

    // one GEMM phase; `next_g` >= 0: afterwards the producer requests the first weight units of that GEMM (of layer next_l)
    auto gemm_phase = [&](int g, int l, int next_g, int next_l) {
        if (producer) {
            bool ok = produce_gemm(p, sh, ring, rg, g, l, pol_w, pol_x, stamp - 1);
            if (ok && next_g >= 0) ok = prefetch_weights(p, sh, ring, rg, next_g, next_l, pol_w);
            if (!ok) { set_error(p.err, DEV_E_WAIT_TIMEOUT); sh.abort_flag = 1; }
        } else if (mma) {
            if (!mma_gemm(p, sh, ring, rg, g, tmem_base, stamp - 1)) { set_error(p.err, DEV_E_WAIT_TIMEOUT); sh.abort_flag = 1; }
        } else if (warp >= 2 && warp < 6) {
            if (!epilogue_gemm(p, sh, rg, g, tmem_base, n_rows, warp, lane, stamp - 1) && lane == 0) { set_error(p.err, DEV_E_WAIT_TIMEOUT); sh.abort_flag = 1; }
        }
    };
    // residual add (partials of GEMM `g_src`, -1: none) + RMSNorm with gain `gain`: row `cta`
    auto norm_phase = [&](int g_src, const void* gain) {
        if (warp < 2 || cta >= n_rows) return;
        StreamK sk = streamk_of(p, g_src < 0 ? 0 : g_src);
        if (g_src < 0) sk.partials = nullptr;
        const __nv_bfloat16* gw = reinterpret_cast<const __nv_bfloat16*>(gain);
        NormFirst<__nv_bfloat16> pf;
        norm_prefetch(pf, sk, gw, p.d, cw, lane);
        resid_norm_row<__nv_bfloat16, CONS_WARPS>(p.hres + (size_t)cta * p.d, sk, cta, gw, p.xn + (size_t)cta * p.d, p.xn_lo + (size_t)cta * p.d,
                                                  p.d, p.rms_eps, nullptr, sh.red, pf, cw, lane, [] { cons_bar(); });
    };

    attn::BulkShared bsm;
    bsm.buf = ring;
    bsm.k_full = sh.k_full; bsm.k_empty = sh.k_empty; bsm.v_full = sh.v_full; bsm.v_empty = sh.v_empty; bsm.s_full = sh.s_full; bsm.q_full = &sh.q_full; bsm.p_ready = &sh.p_ready;
    bsm.pv_done = &sh.pv_done; bsm.xchg = sh.xchg; bsm.s_xchg = &sh.xch[0][0]; bsm.s_abort = &sh.abort_flag;
    attn::BulkMaps bmp;
    bmp.q = &p.map_q; bmp.k = &p.map_k; bmp.v = &p.map_v; bmp.group = p.group; bmp.rows_per_tile = p.rows_per_tile;
    AttnArgs aa;
    aa.q = p.qbuf; aa.out = p.attn_out; aa.out_lo = p.attn_out_lo; aa.part_o = p.part_o; aa.part_ml = p.part_ml; aa.st = st; aa.anc = nullptr; aa.depth = nullptr;
    aa.rows_cap = NRS; aa.cache_in_flight = 0; aa.n_rows_fixed = 0; aa.L_fixed = 0;
    aa.Hq = p.Hq; aa.Hkv = p.Hkv; aa.h = attn::HD; aa.cap = p.cap; aa.split_len = p.split_len; aa.n_split_max = p.n_split_max; aa.dcap = p.dcap;
    aa.scale_log2 = p.scale_log2; aa.err = p.err;
    const int n_heads_qkv = p.Hq + 2 * p.Hkv;
    const int n_row_tiles = (n_rows + p.rows_per_tile - 1) / p.rows_per_tile;
    const int n_split_cap = (L + p.split_len - 1) / p.split_len;      // no row's T0 lies beyond L

    bool ok = true;
    for (int l = 0; l < p.n_layers && ok; ++l) {
        char* kc = p.kcache + p.layer_kv_stride * l;
        char* vc = p.vcache + p.layer_kv_stride * l;
        // ---- 1. residual add of the previous layer's down projection + attention norm
        norm_phase(l == 0 ? -1 : G_DOWN, p.norm_attn[l]);
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 2. QKV projection (its first weight units were requested during the phases before)
        gemm_phase(G_QKV, l, -1, 0);
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 3. partial sums -> (QK-norm) -> RoPE -> query buffer, K/V to cache slot L + row
        if (warp >= 2) {
            QkvArgs qa;
            qa.q_out = p.qbuf; qa.kcache = kc; qa.vcache = vc;
            qa.q_norm = p.qk_norm ? p.q_norm[l] : nullptr; qa.k_norm = p.qk_norm ? p.k_norm[l] : nullptr;
            qa.rope_cos = p.rope_cos; qa.rope_sin = p.rope_sin; qa.Hq = p.Hq; qa.Hkv = p.Hkv; qa.cap = p.cap; qa.qk_norm = p.qk_norm;
            qa.rms_eps = p.rms_eps;
            const StreamK sk = streamk_of(p, G_QKV);
            const int total = n_rows * n_heads_qkv;
            for (int t = cta * CONS_WARPS + cw; t < total; t += G * CONS_WARPS) {
                const int r = t / n_heads_qkv, hs = t % n_heads_qkv;
                QkvPre<attn::HD> pf;
                qkv_prefetch<attn::HD>(pf, qa, sk, hs, L + st->row_depth[r], lane);
                qkv_finish_task<attn::HD>(pf, qa, sk, 0, r, r, L + r, hs, lane);
            }
        }
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 4. attention over the cache below each row's T0: items (split, KV head, row tile) on the tensor cores
        {
            const int n_items = n_split_cap * p.Hkv * n_row_tiles;
            for (int idx = cta; idx < n_items && ok; idx += G) {
                attn::BulkItem it;
                it.split = idx % n_split_cap;
                const int y = idx / n_split_cap;
                it.kvh = y % p.Hkv;
                const int rtile = y / p.Hkv;
                it.seq = 0; it.n_rows = n_rows; it.L = L;
                it.row0 = rtile * p.rows_per_tile;
                if (warp == 2) {
                    int t0 = 0;
                    for (int r = it.row0 + lane; r < it.row0 + p.rows_per_tile && r < n_rows; r += 32)
                        t0 = max(t0, attn::tail_start_tc(L + st->row_depth[r], p.dcap));
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) t0 = max(t0, __shfl_xor_sync(0xffffffffu, t0, o));
                    if (lane == 0) sh.T0max = t0;
                }
                if (threadIdx.x == 0) attn::bulk_init_barriers(bsm);
                main_bar();
                const int T0max = sh.T0max;
                it.beg = it.split * p.split_len;
                if (it.beg < T0max) {       // block-uniform
                    const int end = min(it.beg + p.split_len, T0max);
                    it.n_chunks = (end - it.beg + attn::CK - 1) / attn::CK;
                    it.kv_row0 = l * p.kv_rows_layer + p.kv_row_seq + it.kvh * p.cap;
                    attn::bulk_item_roles<false>(bmp, aa, it, bsm, tmem_base, warp, lane);
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                }
                main_bar();
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                ok = sh.abort_flag == 0;
            }
        }
        if (!ok || !(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 5. tail (end of the cache + in-flight ancestors) and merge with the split partials; meanwhile the
        //         producer requests the first weight units of the O projection (the ring is free again)
        if (producer) {
            if (!prefetch_weights(p, sh, ring, rg, G_O, l, pol_w)) { set_error(p.err, DEV_E_WAIT_TIMEOUT); sh.abort_flag = 1; }
        } else if (warp >= 2) {
            aa.kc = kc; aa.vc = vc;
            const int total = n_rows * p.Hq;
            for (int t = cta * CONS_WARPS + cw; t < total; t += G * CONS_WARPS) {
                attn::PairCtx c;
                c.r = t / p.Hq; c.head = t % p.Hq; c.seq = 0; c.L = L;
                c.depth = st->row_depth[c.r]; c.lo = st->row_anc[c.r][0]; c.hi = st->row_anc[c.r][1];
                attn::FirstPartials<8> fp;
                attn::request_partials<8>(fp, aa, c, lane);      // in flight while the tail is computed
                attn::TailAcc ta;
                attn::tail_pair<16, 16>(ta, aa, c, sh.s_q[cw], lane);
                attn::merge_pair<8>(fp, ta, aa, c, lane);
            }
        }
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 6. O projection
        gemm_phase(G_O, l, G_GU, l);
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 7. residual add + FFN norm
        norm_phase(G_O, p.norm_ffn[l]);
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 8. gate/up projection
        gemm_phase(G_GU, l, G_DOWN, l);
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 9. SiLU(gate) * up
        if (warp >= 2) {
            const StreamK sk = streamk_of(p, G_GU);
            const int groups = p.F / 8;
            const long long total = (long long)n_rows * groups;
            for (long long t = (long long)cta * CONS_THREADS + (threadIdx.x - 64); t < total; t += (long long)G * CONS_THREADS) {
                const int r = (int)(t / groups), j0 = (int)(t % groups) * 8;
                swiglu_task(sk, sk_entry(sk, j0 / 64), r, p.act + (size_t)r * p.F, p.act_lo + (size_t)r * p.F, j0, p.F);
            }
        }
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
        // ---- 10. down projection (summed by the next layer's norm, or by the kernel after this one)
        gemm_phase(G_DOWN, l, l + 1 < p.n_layers ? G_QKV : -1, l + 1);
        if (!(ok = grid_sync(p, sh, epoch, stamp))) break;
    }

    // ---------------- teardown (every thread arrives here)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (sh.abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);   // let copies in flight land before shared memory goes away
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(attn::TMEM_COLS) : "memory");
    }
}

}  // namespace

struct LayersTc {
    LayersParams p;
    int grid = 0;
};

int layers_tc_syncs_per_layer() { return 10; }
int layers_tc_trace_slots() { return TRACE_SLOTS; }

bool layers_tc_supported(const LayersTcDesc& d) {
    if (d.h != attn::HD || !attn_tc_supported(d.h, d.Hq, d.Hkv)) return false;
    if (d.d > 128 * TILE_N || d.d % 8 || d.F % 8) return false;
    for (int i = 0; i < 4; ++i)
        if (!d.gemm[i]) return false;
    return true;
}

int layers_tc_create(LayersTc** out, const LayersTcDesc& d) {
    if (!out || !layers_tc_supported(d)) return -1;
    EncodeFn enc = get_encode();
    if (!enc) return -1;
    LayersTc* t = new (std::nothrow) LayersTc();
    if (!t) return -1;
    memset(&t->p, 0, sizeof(t->p));
    LayersParams& p = t->p;
    int grid = 0;
    for (int i = 0; i < 4; ++i) {
        TcGemmGeom gg;
        tc_gemm_geometry(d.gemm[i], &gg);
        if (gg.nrs != NRS || gg.planes != PLANES || !gg.packed || !gg.table) { delete t; return -1; }
        p.b_plane_seqs = gg.plane_seqs;
        p.g[i].n_tiles = gg.n_tiles; p.g[i].KB = gg.KB; p.g[i].G = gg.grid; p.g[i].slots = gg.slots; p.g[i].table = gg.table;
        p.g[i].pk_off = (unsigned long long)(gg.packed - reinterpret_cast<const unsigned char*>(d.packed));
        p.map_b[i] = gg.map_b;
        p.partials = gg.partials;
        grid = gg.grid > grid ? gg.grid : grid;
    }
    if (grid < d.n_sm) grid = d.n_sm;       // consumers and attention items use every SM
    if (grid < NRS) { delete t; return -1; } // one CTA per row in the norm phases
    t->grid = grid;
    p.packed = reinterpret_cast<const unsigned char*>(d.packed);
    p.pk_layer = d.pk_layer;
    p.hres = d.hres;
    p.xn = reinterpret_cast<__nv_bfloat16*>(d.xn); p.qbuf = reinterpret_cast<__nv_bfloat16*>(d.qbuf);
    p.attn_out = reinterpret_cast<__nv_bfloat16*>(d.attn_out); p.act = reinterpret_cast<__nv_bfloat16*>(d.act);
    p.xn_lo = reinterpret_cast<__nv_bfloat16*>(d.xn_lo); p.attn_out_lo = reinterpret_cast<__nv_bfloat16*>(d.attn_out_lo);
    p.act_lo = reinterpret_cast<__nv_bfloat16*>(d.act_lo);
    if (!p.xn_lo || !p.attn_out_lo || !p.act_lo) { delete t; return -1; }
    p.layer_kv_stride = d.layer_kv_stride;
    p.norm_attn = d.norm_attn; p.norm_ffn = d.norm_ffn; p.q_norm = d.q_norm; p.k_norm = d.k_norm;
    p.rope_cos = d.rope_cos; p.rope_sin = d.rope_sin;
    p.n_layers = d.n_layers; p.d = d.d; p.Hq = d.Hq; p.Hkv = d.Hkv; p.F = d.F; p.cap = d.cap; p.qk_norm = d.qk_norm; p.rms_eps = d.rms_eps;
    p.part_o = d.part_o; p.part_ml = d.part_ml;
    p.split_len = d.split_len; p.n_split_max = d.n_split_max; p.dcap = d.dcap;
    p.group = d.Hq / d.Hkv; p.rows_per_tile = attn::MP / p.group;
    p.kv_rows_layer = d.batch * d.Hkv * d.cap;
    p.scale_log2 = d.scale_log2;
    p.sync_counter = d.sync_counter; p.err = d.err;
    const cuuint32_t estr3[3] = {1, 1, 1};
    {
        cuuint64_t dims[3] = {(cuuint64_t)attn::HD, (cuuint64_t)d.Hq, (cuuint64_t)d.batch * RT};
        cuuint64_t strides[2] = {(cuuint64_t)attn::HD * 2, (cuuint64_t)d.Hq * attn::HD * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)p.group, (cuuint32_t)p.rows_per_tile};
        if (enc(&p.map_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, d.qbuf, dims, strides, box, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { delete t; return -1; }
    }
    for (int i = 0; i < 2; ++i) {
        cuuint64_t dims[2] = {(cuuint64_t)attn::HD, (cuuint64_t)d.n_layers * d.batch * d.Hkv * d.cap};
        cuuint64_t strides[1] = {(cuuint64_t)attn::HD * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)attn::CK};
        if (enc(i ? &p.map_v : &p.map_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, i ? d.vcache : d.kcache, dims, strides, box, estr3,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { delete t; return -1; }
    }
    *out = t;
    return 0;
}

void layers_tc_destroy(LayersTc* t) { delete t; }

int layers_tc_grid(const LayersTc* t) { return t ? t->grid : 0; }

// One launch = all layers for the sequence `seq` (state st, its slice of the cache).  sync_base: the value the
// barrier counter has when the kernel starts (the caller adds layers_tc_arrivals() per launch).
unsigned int layers_tc_arrivals(const LayersTc* t) { return t ? (unsigned int)(t->grid * layers_tc_syncs_per_layer() * t->p.n_layers) : 0u; }

int layers_tc_launch(LayersTc* t, const SeqState* st, int seq, void* kcache_seq, void* vcache_seq, unsigned int sync_base,
                     unsigned long long* timeline, cudaStream_t s) {
    if (!t || !st) return ESP_E_ARG;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(k_layers_tc), (int)SMEM_BYTES)) return ESP_E_CUDA;
    LayersParams p = t->p;
    p.st = st;
    p.kcache = reinterpret_cast<char*>(kcache_seq);
    p.vcache = reinterpret_cast<char*>(vcache_seq);
    p.kv_row_seq = seq * p.Hkv * p.cap;
    p.sync_base = sync_base;
    p.timeline = timeline;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(t->grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;      // every CTA resident at once: the grid barriers need it
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_layers_tc, p) == cudaSuccess ? ESP_OK : ESP_E_CUDA;
}

}  // namespace esp
