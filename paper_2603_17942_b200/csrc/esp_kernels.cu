// CUDA-core kernels of the ESP step: row assembly, RMSNorm, the reference
// (CUDA-core) small-M GEMM, position-canonical tree attention (split partials,
// tail + merge), Top-K' merge, and the single-block tree kernel (verify walk,
// KV compaction, mask update, Algorithm 1 + pruner, next row table).
#include <mutex>
#include <utility>
#include <vector>

#include "esp_epilogue.cuh"
#include "esp_consumers.cuh"
#include "esp_launch.h"

namespace esp {

// ------------------------------------------------------------------ per-device caches of the launch helpers
namespace {
std::mutex g_dev_mutex;
std::vector<std::pair<const void*, int>> g_smem_done;   // (function, device) pairs whose limit has been raised
int g_sm_count[64];
}  // namespace
int ensure_dynamic_smem(const void* func, int bytes) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    for (const auto& e : g_smem_done)
        if (e.first == func && e.second == dev) return 0;
    if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return -1;
    g_smem_done.emplace_back(func, dev);
    return 0;
}
int current_sm_count() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (g_sm_count[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
        g_sm_count[dev] = n;
    }
    return g_sm_count[dev];
}

// ------------------------------------------------------------------ small helpers
__global__ void k_rope_table(float* cs, float* sn, int n_pos, int h, float base) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int half = h / 2;
    if (i >= n_pos * half) return;
    int pos = i / half, j = i % half;
    double inv = pow((double)base, -2.0 * (double)j / (double)h);
    double ang = (double)pos * inv;
    cs[i] = (float)cos(ang);
    sn[i] = (float)sin(ang);
}

// Mask initialisation at prefill, m [slots][d].  mode 0: every slot = (1/t) sum_j E[x_j] (Eq. mask_init_mean; fp32
// running sum in prompt order).  mode 1 ("Last K"): slot i = embedding of the i-th of the last `slots` prompt tokens.
template <typename T>
__global__ void k_mask_init(const T* embed, const int32_t* prompt, int t, int d, float* m, int slots, int mode) {
    int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    if (mode == 1) {
        for (int i = 0; i < slots; ++i) {
            int src = t - slots + i;
            if (src < 0) src = 0;
            m[(size_t)i * d + j] = to_f32(embed[(size_t)prompt[src] * d + j]);
        }
        return;
    }
    float acc = 0.f;
    for (int i = 0; i < t; ++i) acc = acc + to_f32(embed[(size_t)prompt[i] * d + j]);
    const float mean = acc / (float)t;
    for (int i = 0; i < slots; ++i) m[(size_t)i * d + j] = mean;
}

// Input rows of the block: E[token] for tree nodes; probe j of a chain gets mask vector j (rows after the
// tree nodes hold the chains back to back, k rows each).
template <typename T>
__global__ void k_assemble(const SeqState* states, const T* embed, const float* mvec, float* hres, int d, int mask_slots) {
    // let the next kernel start its own preamble (for a GEMM: the first weight tiles) while this one runs; it still
    // waits for this kernel to complete before it touches anything this kernel or its predecessors write
    if (threadIdx.x == 0) pdl_launch_dependents();
    pdl_wait();
    int seq = blockIdx.y, r = blockIdx.x;
    const SeqState* st = states + seq;
    if (!st->active || r >= st->n_rows) return;
    float* out = hres + (size_t)(seq * RT + r) * d;
    int tok = st->row_token[r];
    // four elements per thread and step (d is a multiple of 8), independent loads in flight
    if (tok >= 0) {
        const T* src = embed + (size_t)tok * d;
#pragma unroll 4
        for (int j = threadIdx.x * 4; j < d; j += blockDim.x * 4) {
            float4 v;
            if constexpr (sizeof(T) == 2) {
                const uint2 raw = *reinterpret_cast<const uint2*>(src + j);
                const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&raw.x), hi = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
                v = make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
            } else {
                v = *reinterpret_cast<const float4*>(src + j);
            }
            *reinterpret_cast<float4*>(out + j) = v;
        }
    } else {
        const float* src = mvec + ((size_t)seq * mask_slots + (r - st->n_nodes) % mask_slots) * d;
#pragma unroll 4
        for (int j = threadIdx.x * 4; j < d; j += blockDim.x * 4) *reinterpret_cast<float4*>(out + j) = *reinterpret_cast<const float4*>(src + j);
    }
}

// y = x * rsqrt(mean(x^2)+eps) * g, one block per row
template <typename T>
__global__ void __launch_bounds__(256) k_rmsnorm(const SeqState* states, const float* x, const T* g, T* y, int d, float eps,
                                                float* copy_out) {
    // let the next kernel start its own preamble (for a GEMM: the first weight tiles) while this one runs; it still
    // waits for this kernel to complete before it touches anything this kernel or its predecessors write
    if (threadIdx.x == 0) pdl_launch_dependents();
    pdl_wait();
    int seq = blockIdx.y, r = blockIdx.x;
    const SeqState* st = states + seq;
    if (!st->active || r >= st->n_rows) return;
    const float* xr = x + (size_t)(seq * RT + r) * d;
    __shared__ float red[8];
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += 256) { float v = xr[j]; ss += v * v; }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    float rinv = 1.0f / sqrtf(tot / (float)d + eps);
    T* yr = y + (size_t)(seq * RT + r) * d;
    for (int j = threadIdx.x; j < d; j += 256) yr[j] = from_f32<T>(xr[j] * rinv * to_f32(g[j]));
    if (copy_out)
        for (int j = threadIdx.x; j < d; j += 256) copy_out[(size_t)(seq * RT + r) * d + j] = xr[j];
}

// Consumer of a split GEMM (O or down projection) fused with the residual add and the next RMSNorm:
//   hres[r] += sum over the tile's contributors, in CTA order, of their fp32 partials;  y = rmsnorm(hres[r]) * g.
// One block per row (resid_norm_row); with sk.partials == NULL it is a plain RMSNorm of hres.  The sum order
// depends only on the GEMM's shape, never on the number of rows in the block.
template <typename T>
__global__ void __launch_bounds__(1024) k_resid_norm(const SeqState* states, float* hres, StreamK sk, const T* g, T* y, T* y_lo, int d,
                                                    float eps, float* copy_out) {
    // let the next kernel start its own preamble (for a GEMM: the first weight tiles) while this one runs; it still
    // waits for this kernel to complete before it touches anything this kernel or its predecessors write
    if (threadIdx.x == 0) pdl_launch_dependents();
    // fetched before the wait: the tile's contributor entry and the norm weights of this warp's first group
    // (neither changes after initialisation), so that only the partials are loaded behind the wait
    __shared__ float red[128];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    NormFirst<T> pf;
    norm_prefetch(pf, sk, g, d, warp, lane);
    const int seq = blockIdx.y, r = blockIdx.x;
    const SeqState* st = states + seq;
    const bool idle = !st->active || r >= st->n_rows;     // the row table was written by an earlier step
    pdl_wait();
    if (idle) return;
    const size_t row = (size_t)(seq * RT + r) * d;
    resid_norm_row<T, 32>(hres + row, sk, seq * sk.seq_rows + r, g, y + row, y_lo ? y_lo + row : nullptr, d, eps,
                          copy_out ? copy_out + row : nullptr, red, pf, warp, lane, [] { __syncthreads(); });
}

// Consumer of the split QKV GEMM: sums the partials of one (row, head) in CTA order, then what follows
// the projection in the decoder layer -- per-head RMSNorm on q and k (Qwen3), rotary embedding at the
// row's position L + depth, q to the query buffer, k and v to cache slot L + row.  One warp per (row, head),
// a lane owns HD/32 consecutive features; the rotate-half partner (i, i + HD/2) sits 16 lanes away.
template <int HD>
__global__ void __launch_bounds__(128) k_qkv_finish(EpiArgs a, StreamK sk) {
    // let the next kernel start its own preamble (for a GEMM: the first weight tiles) while this one runs; it still
    // waits for this kernel to complete before it touches anything this kernel or its predecessors write
    if (threadIdx.x == 0) pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hs = blockIdx.x * 4 + warp, r = blockIdx.y, seq = blockIdx.z;   // seq: sequence within this launch
    // Fetched before the wait, so that only the partials are loaded behind it: the row table (written by an earlier
    // step), the tile's contributor entry, the rotary factors of the row's position and the norm weights
    const SeqState* st = a.st ? a.st + seq : nullptr;
    const int n_rows = st ? (st->active ? st->n_rows : 0) : a.rows_fixed;
    const bool work = r < n_rows && hs < a.Hq + 2 * a.Hkv;
    const int L = st ? st->L : 0;
    QkvArgs qa;
    qa.q_out = a.q_out; qa.kcache = a.kcache; qa.vcache = a.vcache; qa.q_norm = a.q_norm; qa.k_norm = a.k_norm;
    qa.rope_cos = a.rope_cos; qa.rope_sin = a.rope_sin; qa.Hq = a.Hq; qa.Hkv = a.Hkv; qa.cap = a.cap; qa.qk_norm = a.qk_norm;
    qa.rms_eps = a.rms_eps;
    QkvPre<HD> pf;
    if (work) qkv_prefetch<HD>(pf, qa, sk, hs, L + (st ? st->row_depth[r] : r), lane);
    pdl_wait();
    if (!work) return;
    qkv_finish_task<HD>(pf, qa, sk, seq, seq * sk.seq_rows + r, seq * RT + r, L + r, hs, lane);
}

// Consumer of the split gate/up GEMM: a tile holds 64 gate features (columns 0..63) and the matching 64 up
// features (columns 64..127); sums both over the tile's contributors in CTA order and stores silu(gate) * up.
__global__ void __launch_bounds__(256) k_swiglu_finish(const SeqState* states, int rows_fixed, StreamK sk, __nv_bfloat16* act,
                                                      __nv_bfloat16* act_lo, int F) {
    // let the next kernel start its own preamble (for a GEMM: the first weight tiles) while this one runs; it still
    // waits for this kernel to complete before it touches anything this kernel or its predecessors write
    if (threadIdx.x == 0) pdl_launch_dependents();
    // eight features per thread: half the threads, so that the next GEMM's CTA finds registers free beside this
    // kernel's CTAs and can start its weight stream while they run
    const int j0 = (blockIdx.x * 256 + threadIdx.x) * 8;
    SkEntry en;      // fixed since the plan was built: fetched before the wait (the eight features share a tile)
    if (j0 < F) en = sk_entry(sk, j0 / 64);
    const int r = blockIdx.y, seq = blockIdx.z;
    const int n_rows = states ? (states[seq].active ? states[seq].n_rows : 0) : rows_fixed;   // written by an earlier step
    pdl_wait();
    if (r >= n_rows || j0 >= F) return;
    swiglu_task(sk, en, seq * sk.seq_rows + r, act + (size_t)(seq * RT + r) * F, act_lo ? act_lo + (size_t)(seq * RT + r) * F : nullptr, j0, F);
}

// ------------------------------------------------------------------ CUDA-core GEMM
// y[row][n] = sum_k x[row][k] * w[n][k], k ascending, one thread per output feature of a
// 128-feature tile and all RT rows of one sequence.  Used for fp32 models and as the on-GPU
// cross-check of the tcgen05 kernel.  Tile -> weight rows mapping is the same as there:
// up to three stacked matrices (q|k|v), or gate/up halves interleaved per tile.
struct SimtGemmArgs {
    const void* w[3];   // stacked matrices (rows_w[i] rows each); SWIGLU: w[0]=gate, w[1]=up
    int32_t rows_w[3];
    const void* x;      // [batch*RT][K]
    int32_t K;
};

template <typename T, int EPI>
__global__ void __launch_bounds__(128) k_gemm_simt(SimtGemmArgs g, EpiArgs a) {
    extern __shared__ float smem[];
    float* s_acc = smem;                       // RT * ACC_LD
    float* s_aux = s_acc + RT * ACC_LD;        // RT * 4
    float* s_x = s_aux + RT * 4;               // RT * 32
    float* s_w = s_x + RT * 32;                // 128 * 33
    pdl_wait();
    const int tile = blockIdx.x, seq = blockIdx.y, f = threadIdx.x;
    if (a.st && !a.st[seq].active) return;
    const int n_rows = a.st ? a.st[seq].n_rows : a.rows_fixed;
    const T* x = reinterpret_cast<const T*>(g.x) + (size_t)seq * RT * g.K;
    // weight row of feature i of this tile (nullptr if outside)
    auto wrow = [&](int i) -> const T* {
        if (EPI == EPI_SWIGLU) {
            int feat = tile * 64 + (i & 63);
            if (feat >= g.rows_w[0]) return nullptr;
            return reinterpret_cast<const T*>(g.w[i >> 6]) + (size_t)feat * g.K;
        }
        int feat = tile * TILE_N + i;
        for (int m = 0; m < 3; ++m) {
            if (feat < g.rows_w[m]) return reinterpret_cast<const T*>(g.w[m]) + (size_t)feat * g.K;
            feat -= g.rows_w[m];
        }
        return nullptr;
    };
    float acc[RT];
#pragma unroll
    for (int r = 0; r < RT; ++r) acc[r] = 0.f;
    for (int k0 = 0; k0 < g.K; k0 += 32) {
        for (int i = f; i < RT * 32; i += 128) {
            int r = i >> 5, c = i & 31;
            s_x[i] = (r < n_rows && k0 + c < g.K) ? to_f32(x[(size_t)r * g.K + k0 + c]) : 0.f;
        }
        for (int i = 0; i < 32; ++i) {
            int row = (f >> 5) + 4 * i, c = f & 31;
            const T* wr = wrow(row);
            s_w[row * 33 + c] = (wr && k0 + c < g.K) ? to_f32(wr[k0 + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int c = 0; c < 32; ++c) {
            float w = s_w[f * 33 + c];
#pragma unroll
            for (int r = 0; r < RT; ++r) acc[r] = fmaf(s_x[r * 32 + c], w, acc[r]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < RT; ++r) s_acc[r * ACC_LD + f] = acc[r];
    __syncthreads();
    run_epilogue<T, EPI>(s_acc, s_aux, tile, seq, a, f, 1);
}

template <typename T>
void launch_gemm_simt_t(int epi, int n_tiles, int batch, const SimtGemmArgs& g, const EpiArgs& a, cudaStream_t s, bool pdl) {
    size_t smem = sizeof(float) * (RT * ACC_LD + RT * 4 + RT * 32 + 128 * 33);
    dim3 grid(n_tiles, batch);
#define ESP_SIMT_CASE(E)                                                                                  \
    case E:                                                                                               \
        cudaFuncSetAttribute(k_gemm_simt<T, E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
        launch_k(k_gemm_simt<T, E>, grid, dim3(128), smem, s, pdl, g, a);                                 \
        break;
    switch (epi) {
        ESP_SIMT_CASE(EPI_STORE_F32)
        ESP_SIMT_CASE(EPI_QKV)
        ESP_SIMT_CASE(EPI_RESID)
        ESP_SIMT_CASE(EPI_SWIGLU)
        ESP_SIMT_CASE(EPI_LOGITS)
    }
#undef ESP_SIMT_CASE
}

void launch_gemm_simt(int dtype, int epi, int n_tiles, int batch, const void* const w[3], const int32_t rows_w[3],
                      const void* x, int K, const EpiArgs& a, cudaStream_t s, bool pdl) {
    SimtGemmArgs g;
    for (int i = 0; i < 3; ++i) { g.w[i] = w[i]; g.rows_w[i] = rows_w[i]; }
    g.x = x;
    g.K = K;
    if (dtype == 0) launch_gemm_simt_t<float>(epi, n_tiles, batch, g, a, s, pdl);
    else launch_gemm_simt_t<__nv_bfloat16>(epi, n_tiles, batch, g, a, s, pdl);
}

// ------------------------------------------------------------------ attention (position-canonical)
// Key list of a row at position P = L + depth: positions 0..P.  Positions below
// T0 = max(0, floor((P - dcap)/16)*16) are summed by the chunked "bulk" path in splits of
// split_len positions aligned to position 0; positions T0..P (cache tail + the row's in-flight
// ancestors, found through its ancestor bitmask in row order = position order) by the tail.
// Every reduction order depends on absolute positions only, so a token verified inside a tree
// block gets bit-identical results to the same token decoded alone.
__device__ __forceinline__ int tail_start(int P, int dcap) {
    int t = P - dcap;
    return t <= 0 ? 0 : (t / 16) * 16;
}

// index of the n-th (0-based) set bit of a 128-bit mask
__device__ __forceinline__ int nth_set_bit(unsigned long long lo, unsigned long long hi, int n) {
    int c = __popcll(lo);
    unsigned long long m = lo;
    int base = 0;
    if (n >= c) { n -= c; m = hi; base = 64; }
    for (int i = 0; i < n; ++i) m &= m - 1;
    return m ? base + __ffsll((long long)m) - 1 : -1;
}


__device__ __forceinline__ void attn_row_info(const AttnArgs& a, int seq, int r, int& n_rows, int& L, int& depth,
                                              unsigned long long& lo, unsigned long long& hi) {
    if (a.st) {
        const SeqState* st = a.st + seq;
        n_rows = st->active ? st->n_rows : 0;
        L = st->L;
        depth = r < RT ? st->row_depth[r] : 0;
        lo = r < RT ? st->row_anc[r][0] : 0;
        hi = r < RT ? st->row_anc[r][1] : 0;
    } else {
        n_rows = a.n_rows_fixed;
        L = a.L_fixed;
        depth = a.depth[seq * RT + r];
        lo = a.anc[(size_t)(seq * RT + r) * 2];
        hi = a.anc[(size_t)(seq * RT + r) * 2 + 1];
    }
}

// One chunk of up to 32 keys for one (row, head) handled by one warp: lane j owns key j.
// Returns the chunk's own (max, sum, weighted values) relative to its own max, in the log2 domain.
template <typename T, int HD>
__device__ __forceinline__ void warp_chunk(const float* s_q, const T* kbase, const T* vbase, int slot, bool valid,
                                           float scale_log2, float& cm, float& cl, float (&co)[HD / 32]) {
    const int lane = threadIdx.x & 31;
    float s = -INFINITY;
    if (valid) {
        const T* kr = kbase + (size_t)slot * HD;
        float acc = 0.f;
#pragma unroll 8
        for (int d = 0; d < HD; ++d) acc = fmaf(s_q[d], to_f32(kr[d]), acc);
        s = acc * scale_log2;
    }
    cm = warp_max(s);
    float p = valid ? exp2f(s - cm) : 0.f;
    cl = warp_sum(p);
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) co[i] = 0.f;
    for (int j = 0; j < 32; ++j) {
        float pj = __shfl_sync(0xffffffffu, p, j);
        int sj = __shfl_sync(0xffffffffu, slot, j);
        if (pj != 0.f) {
            const T* vr = vbase + (size_t)sj * HD;
#pragma unroll
            for (int i = 0; i < HD / 32; ++i) co[i] = fmaf(pj, to_f32(vr[lane + 32 * i]), co[i]);
        }
    }
}

template <int N>
__device__ __forceinline__ void merge_partial(float& m, float& l, float (&o)[N], float cm, float cl, const float (&co)[N]) {
    float mn = fmaxf(m, cm);
    float a = exp2f(m - mn), b = exp2f(cm - mn);
    l = l * a + cl * b;
#pragma unroll
    for (int i = 0; i < N; ++i) o[i] = o[i] * a + co[i] * b;
    m = mn;
}

// Bulk, CUDA-core version: one warp per (row, head, split).  grid = (ceil(RT/4), Hq, n_split*batch).
template <typename T, int HD>
__global__ void __launch_bounds__(128) k_attn_bulk_simt(AttnArgs a, int n_split_launch) {
    __shared__ float s_qall[4][HD];
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 4 + warp, head = blockIdx.y;
    const int split = blockIdx.z % n_split_launch, seq = blockIdx.z / n_split_launch;
    int n_rows, L, depth;
    unsigned long long lo, hi;
    attn_row_info(a, seq, r < RT ? r : 0, n_rows, L, depth, lo, hi);
    if (r >= n_rows) return;
    const int T0 = tail_start(L + depth, a.dcap);
    const int beg = split * a.split_len, end = min(beg + a.split_len, T0);
    if (beg >= end) return;
    const int kvh = head / (a.Hq / a.Hkv);
    const T* q = reinterpret_cast<const T*>(a.q) + ((size_t)(seq * RT + r) * a.Hq + head) * HD;
    float* s_q = s_qall[warp];
    for (int d = lane; d < HD; d += 32) s_q[d] = to_f32(q[d]);
    __syncwarp();
    const T* kb = reinterpret_cast<const T*>(a.kc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    const T* vb = reinterpret_cast<const T*>(a.vc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    float m = -INFINITY, l = 0.f, o[HD / 32];
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) o[i] = 0.f;
    for (int p0 = beg; p0 < end; p0 += 32) {
        float cm, cl, co[HD / 32];
        int pos = p0 + lane;
        warp_chunk<T, HD>(s_q, kb, vb, pos, pos < end, a.scale_log2, cm, cl, co);
        merge_partial(m, l, o, cm, cl, co);
    }
    size_t idx = ((size_t)(seq * RT + r) * a.Hq + head) * a.n_split_max + split;
    if (lane == 0) a.part_ml[idx] = make_float2(m, l);
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) a.part_o[idx * HD + lane + 32 * i] = o[i];
}

// Tail + merge: one warp per (row, head).  grid = (ceil(RT/4), Hq, batch).
template <typename T, int HD>
__global__ void __launch_bounds__(128) k_attn_tail_merge(AttnArgs a) {
    __shared__ float s_qall[4][HD];
    // let the next kernel start its own preamble (for a GEMM: the first weight tiles) while this one runs; it still
    // waits for this kernel to complete before it touches anything this kernel or its predecessors write
    if (threadIdx.x == 0) pdl_launch_dependents();
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 4 + warp, head = blockIdx.y, seq = blockIdx.z;
    int n_rows, L, depth;
    unsigned long long lo, hi;
    attn_row_info(a, seq, r < RT ? r : 0, n_rows, L, depth, lo, hi);
    if (r >= n_rows) return;
    const int P = L + depth;
    const int T0 = tail_start(P, a.dcap);
    const int kvh = head / (a.Hq / a.Hkv);
    const T* q = reinterpret_cast<const T*>(a.q) + ((size_t)(seq * RT + r) * a.Hq + head) * HD;
    float* s_q = s_qall[warp];
    for (int d = lane; d < HD; d += 32) s_q[d] = to_f32(q[d]);
    __syncwarp();
    const T* kb = reinterpret_cast<const T*>(a.kc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    const T* vb = reinterpret_cast<const T*>(a.vc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    float m = -INFINITY, l = 0.f, o[HD / 32];
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) o[i] = 0.f;
    // bulk partials in split order
    const int n_sp = (T0 + a.split_len - 1) / a.split_len;
    const size_t base = ((size_t)(seq * RT + r) * a.Hq + head) * a.n_split_max;
    for (int s = 0; s < n_sp; ++s) {
        float2 ml = a.part_ml[base + s];
        float co[HD / 32];
#pragma unroll
        for (int i = 0; i < HD / 32; ++i) co[i] = a.part_o[(base + s) * HD + lane + 32 * i];
        merge_partial(m, l, o, ml.x, ml.y, co);
    }
    // tail: positions T0..P in order
    const int n_tail = P - T0 + 1;
    for (int t0 = 0; t0 < n_tail; t0 += 32) {
        int t = t0 + lane;
        bool valid = t < n_tail;
        int slot = 0;
        if (valid) {
            int pos = T0 + t;
            if (pos < L) slot = pos;
            else {
                int b = nth_set_bit(lo, hi, pos - L);
                if (b < 0) { set_error(a.err, DEV_E_INDEX); valid = false; }
                else slot = L + b;
            }
        }
        float cm, cl, co[HD / 32];
        warp_chunk<T, HD>(s_q, kb, vb, slot, valid, a.scale_log2, cm, cl, co);
        merge_partial(m, l, o, cm, cl, co);
    }
    T* out = reinterpret_cast<T*>(a.out) + ((size_t)(seq * RT + r) * a.Hq + head) * HD;
    const float inv = 1.0f / l;
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) out[lane + 32 * i] = from_f32<T>(o[i] * inv);
    if constexpr (sizeof(T) == 2) {
        if (a.out_lo) {      // low-order plane for an O projection that reads the output as hi + lo
            T* out_lo = reinterpret_cast<T*>(a.out_lo) + ((size_t)(seq * RT + r) * a.Hq + head) * HD;
#pragma unroll
            for (int i = 0; i < HD / 32; ++i) {
                T hi, lo2;
                split_bf16(o[i] * inv, hi, lo2);
                out_lo[lane + 32 * i] = lo2;
            }
        }
    }
}

template <typename T, int HD>
static void launch_attn_simt_t(const AttnArgs& a, int batch, int n_split_launch, bool bulk_too, cudaStream_t s, bool pdl) {
    dim3 g1((RT + 3) / 4, a.Hq, n_split_launch * batch);
    if (bulk_too && n_split_launch > 0) launch_k(k_attn_bulk_simt<T, HD>, g1, dim3(128), 0, s, pdl, a, n_split_launch);
    dim3 g2((RT + 3) / 4, a.Hq, batch);
    launch_k(k_attn_tail_merge<T, HD>, g2, dim3(128), 0, s, pdl, a);
}

int launch_attn_simt(int dtype, const AttnArgs& a, int batch, int n_split_launch, bool bulk_too, cudaStream_t s, bool pdl) {
#define ESP_ATTN_CASE(TT, H) launch_attn_simt_t<TT, H>(a, batch, n_split_launch, bulk_too, s, pdl); return 0;
    if (dtype == 0) {
        if (a.h == 32) { ESP_ATTN_CASE(float, 32) }
        if (a.h == 64) { ESP_ATTN_CASE(float, 64) }
        if (a.h == 128) { ESP_ATTN_CASE(float, 128) }
    } else {
        if (a.h == 32) { ESP_ATTN_CASE(__nv_bfloat16, 32) }
        if (a.h == 64) { ESP_ATTN_CASE(__nv_bfloat16, 64) }
        if (a.h == 128) { ESP_ATTN_CASE(__nv_bfloat16, 128) }
    }
#undef ESP_ATTN_CASE
    return -1;
}

// ------------------------------------------------------------------ Top-K' merge over vocabulary tiles
// One block per row: global Top-K' (value desc, id asc) of the per-tile lists, plus
// lse = max + log(sum exp) merged over tiles in a fixed order.  The row's per-tile lists are staged in
// shared memory (when they fit) so the K' selection rounds touch no global memory.
constexpr int TOPK_THREADS = 256;
constexpr int TOPK_MAXT = 8;   // tiles per thread (n_tiles <= 2048)
__global__ void __launch_bounds__(TOPK_THREADS) k_topk_merge(const SeqState* states, const Cand* cand, const float2* cand_ms,
                                                             int n_tiles, int KP, int batch, Cand* topk, float* lse, int stage,
                                                             uint32_t* cand_floor) {
    extern __shared__ __align__(16) unsigned char tk_smem[];
    Cand* s_c = reinterpret_cast<Cand*>(tk_smem);
    __shared__ float s_v[TOPK_THREADS];
    __shared__ int s_i[TOPK_THREADS];
    if (threadIdx.x == 0) pdl_launch_dependents();
    pdl_wait();
    const int seq = blockIdx.y, r = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const SeqState* st = states + seq;
    if (!st->active || r >= st->n_rows) return;
    const int Mtot = batch * RT, grow = seq * RT + r;
    const bool probe = r >= st->n_nodes;
    const int kp = probe ? KP : 1;
    if (stage) {
        for (int i = tid; i < n_tiles * kp; i += TOPK_THREADS) {
            const int t = i / kp, q = i - t * kp;
            s_c[i] = cand[((size_t)t * Mtot + grow) * KP + q];
        }
        __syncthreads();
    }
    auto entry = [&](int t, int q) -> Cand { return stage ? s_c[t * kp + q] : cand[((size_t)t * Mtot + grow) * KP + q]; };
    // Two levels, both by (value desc, id asc).  Level 1: each warp merges the sorted lists of its tiles (tile t
    // belongs to thread t mod 256) into its own top kp -- a round is the lane-local best head, then two warp-wide
    // integer reductions (largest order-preserving key, smallest id among its holders); no block barrier.
    // Level 2: warp 0 merges the 8 warp lists the same way, one list per lane.
    __shared__ Cand s_w[TOPK_THREADS / 32][KP_MAX];
    unsigned char cur[TOPK_MAXT];
#pragma unroll
    for (int i = 0; i < TOPK_MAXT; ++i) cur[i] = 0;
    for (int j = 0; j < kp; ++j) {
        float bv = -INFINITY;
        int bi = 0x7fffffff, bt = -1;
#pragma unroll
        for (int i = 0; i < TOPK_MAXT; ++i) {
            const int t = tid + TOPK_THREADS * i;
            if (t < n_tiles && cur[i] < kp) {
                const Cand c = entry(t, cur[i]);
                if (c.id >= 0 && cand_before(c.val, c.id, bv, bi)) { bv = c.val; bi = c.id; bt = i; }
            }
        }
        const uint32_t key = bt >= 0 ? float_order_key(bv) : 0u;
        const uint32_t wkey = __reduce_max_sync(0xffffffffu, key);
        const uint32_t wid = __reduce_min_sync(0xffffffffu, (bt >= 0 && key == wkey) ? (uint32_t)bi : 0xffffffffu);
        if (bt >= 0 && key == wkey && (uint32_t)bi == wid) {   // token ids are unique across tiles: one owner
#pragma unroll
            for (int i = 0; i < TOPK_MAXT; ++i) if (i == bt) cur[i]++;
            s_w[warp][j].val = bv;
            s_w[warp][j].id = bi;
        }
        if (wkey == 0u && lane == 0) { s_w[warp][j].val = -INFINITY; s_w[warp][j].id = -1; }
    }
    __syncthreads();
    if (warp == 0) {
        int c2 = 0;     // this lane's cursor into warp list `lane`
        for (int j = 0; j < kp; ++j) {
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            bool have = false;
            if (lane < TOPK_THREADS / 32 && c2 < kp) {
                const Cand c = s_w[lane][c2];
                if (c.id >= 0) { bv = c.val; bi = c.id; have = true; }
            }
            const uint32_t key = have ? float_order_key(bv) : 0u;
            const uint32_t wkey = __reduce_max_sync(0xffffffffu, key);
            const uint32_t wid = __reduce_min_sync(0xffffffffu, (have && key == wkey) ? (uint32_t)bi : 0xffffffffu);
            if (have && key == wkey && (uint32_t)bi == wid) {
                ++c2;
                topk[(size_t)grow * KP_MAX + j].val = bv;
                topk[(size_t)grow * KP_MAX + j].id = bi;
            }
            if (wkey == 0u && lane == 0) { topk[(size_t)grow * KP_MAX + j].val = -INFINITY; topk[(size_t)grow * KP_MAX + j].id = -1; }
        }
    }
    __syncthreads();
    if (probe) {
        // thread-strided partial merges in tile order, then a fixed tree over threads
        float m = -INFINITY, sm = 0.f;
        for (int t = tid; t < n_tiles; t += TOPK_THREADS) {
            const float2 ms = cand_ms[(size_t)t * Mtot + grow];
            const float mn = fmaxf(m, ms.x);
            sm = sm * expf(m - mn) + ms.y * expf(ms.x - mn);
            m = mn;
        }
        float* s_s = reinterpret_cast<float*>(s_i);
        s_v[tid] = m;
        s_s[tid] = sm;
        __syncthreads();
        for (int o = TOPK_THREADS / 2; o > 0; o >>= 1) {
            if (tid < o) {
                const float m1 = s_v[tid], m2 = s_v[tid + o];
                const float s1 = s_s[tid], s2 = s_s[tid + o];
                const float mn = fmaxf(m1, m2);
                const float sn = (m1 == -INFINITY ? 0.f : s1 * expf(m1 - mn)) + (m2 == -INFINITY ? 0.f : s2 * expf(m2 - mn));
                s_v[tid] = mn;
                s_s[tid] = sn;
            }
            __syncthreads();
        }
        if (tid == 0) lse[grow] = s_v[0] + logf(s_s[0]);
        if (tid == 0 && cand_floor) cand_floor[grow] = 0;     // nothing is known about the next forward's logits
    }
}

void launch_topk_merge(const SeqState* st, const Cand* cand, const float2* cand_ms, int n_tiles, int KP, int batch,
                       Cand* topk, float* lse, cudaStream_t s, bool pdl, int rows_cap, uint32_t* cand_floor) {
    dim3 grid(rows_cap, batch);
    size_t smem = (size_t)n_tiles * KP * sizeof(Cand);
    int stage = smem <= 160 * 1024 ? 1 : 0;
    if (!stage) smem = 0;
    static size_t attr_bytes = 0;
    if (smem > attr_bytes) {
        cudaFuncSetAttribute(k_topk_merge, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attr_bytes = smem;
    }
    launch_k(k_topk_merge, grid, dim3(TOPK_THREADS), smem, s, pdl, st, cand, cand_ms, n_tiles, KP, batch, topk, lse, stage, cand_floor);
}

// ------------------------------------------------------------------ sampling noise, stand-alone (for checking)
__global__ void k_gumbel_noise(uint32_t key0, uint32_t key1, uint32_t position, int n, float* out) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n) out[v] = gumbel_noise(key0, key1, position, (uint32_t)v);
}
void launch_gumbel_noise(uint32_t key0, uint32_t key1, uint32_t position, int n, float* out, cudaStream_t s) {
    k_gumbel_noise<<<(n + 255) / 256, 256, 0, s>>>(key0, key1, position, n, out);
}

// ------------------------------------------------------------------ row-table builders
__device__ void write_probe_rows(SeqState* st, int N, int k, int first_anchor, int n_anchor_rows) {
    // probe j (1-based) of the a-th anchored node sits at row N + a*k + (j-1)
    for (int i = threadIdx.x; i < n_anchor_rows * k; i += blockDim.x) {
        int aidx = i / k, j = i % k + 1;
        int u = first_anchor + aidx;
        int row = N + aidx * k + (j - 1);
        st->row_token[row] = -1;
        st->row_parent[row] = j == 1 ? u : row - 1;
        st->row_depth[row] = st->row_depth[u] + j;
        unsigned long long lo = st->row_anc[u][0], hi = st->row_anc[u][1];
        for (int jj = 0; jj < j; ++jj) {
            int b = N + aidx * k + jj;
            if (b < 64) lo |= 1ull << b; else hi |= 1ull << (b - 64);
        }
        st->row_anc[row][0] = lo;
        st->row_anc[row][1] = hi;
        st->row_logp[row] = 0.f;
    }
}

// Prefill chunk: rows are n consecutive prompt tokens (a chain); the last chunk appends k probes
// behind the last prompt token (Figure 1 middle).
__global__ void k_setup_chain(SeqState* states, int seq, const int32_t* prompt_dev, int off, int n, int last, int k) {
    SeqState* st = states + seq;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        st->row_token[i] = prompt_dev[off + i];
        st->row_parent[i] = i - 1;
        st->row_depth[i] = i;
        unsigned long long lo = i >= 63 ? ~0ull : ((1ull << (i + 1)) - 1);
        unsigned long long hi = i < 64 ? 0ull : ((1ull << (i - 63)) - 1);
        st->row_anc[i][0] = lo;
        st->row_anc[i][1] = hi;
        st->row_logp[i] = 0.f;
    }
    __syncthreads();
    if (last && k > 0) write_probe_rows(st, n, k, n - 1, 1);
    if (threadIdx.x == 0) {
        st->n_nodes = n;
        st->n_rows = n + (last ? k : 0);
        st->mode = last ? 2 : 1;
        st->active = 1;
        if (off == 0) st->L = 0;
    }
}

// Caller-provided tree (test hook): tokens/parents in breadth-first order.
__global__ void k_set_tree(SeqState* states, int seq, const int32_t* tokens, const int32_t* parents, int n, int k,
                           int n_anchor, int* err) {
    SeqState* st = states + seq;
    if (threadIdx.x == 0) {
        for (int i = 0; i < n; ++i) {
            int p = parents[i];
            if (i == 0 ? p != -1 : (p < 0 || p >= i)) { set_error(err, DEV_E_INDEX); p = i == 0 ? -1 : 0; }
            st->row_token[i] = tokens[i];
            st->row_parent[i] = p;
            st->row_depth[i] = i == 0 ? 0 : st->row_depth[p] + 1;
            unsigned long long lo = i == 0 ? 0 : st->row_anc[p][0], hi = i == 0 ? 0 : st->row_anc[p][1];
            if (i < 64) lo |= 1ull << i; else hi |= 1ull << (i - 64);
            st->row_anc[i][0] = lo;
            st->row_anc[i][1] = hi;
            st->row_logp[i] = 0.f;
        }
        st->n_nodes = n;
    }
    __syncthreads();
    int nA = k > 0 ? (n_anchor == 0 ? n : min(n_anchor, n)) : 0;
    write_probe_rows(st, n, k, 0, nA);
    if (threadIdx.x == 0) { st->n_rows = n + nA * k; st->mode = 0; st->forced = 1; }
}

// ------------------------------------------------------------------ the single-block tree kernel
// verify walk -> KV compaction -> mask update -> Algorithm 1 + pruner -> next row table.

// Total order of created nodes as one integer: (logP descending, depth ascending, creation index ascending);
// a smaller key comes first.  -0.0 and +0.0 compare equal as floats, so both map to the key of +0.0.
__device__ __forceinline__ unsigned long long node_key(float lp, int depth, int idx) {
    unsigned u = __float_as_uint(lp == 0.f ? 0.f : lp);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);   // monotone: larger float -> larger u
    return ((unsigned long long)(~u) << 32) | ((unsigned long long)depth << 16) | (unsigned long long)idx;
}

template <typename T>
__global__ void __launch_bounds__(1024) k_tree_step(TreeArgs A) {
    extern __shared__ unsigned char smem_raw[];
    int* c_tok = reinterpret_cast<int*>(smem_raw);
    int* c_par = c_tok + MAX_CAND;
    int* c_dep = c_par + MAX_CAND;
    float* c_lp = reinterpret_cast<float*>(c_dep + MAX_CAND);
    int* c_rank = reinterpret_cast<int*>(c_lp + MAX_CAND);
    __shared__ int s_path[PROBES_MAX + 2], s_out[PROBES_MAX + 2];
    __shared__ int s_na, s_ustar, s_delta, s_nexp, s_ncreated, s_abort;
    __shared__ int s_exp[RT], s_sel[RT], s_new[RT];
    __shared__ int s_rtok[RT], s_rpar[RT], s_rdep[RT], s_arg[RT];   // this step's row table and per-row argmax
    __shared__ int s_cnt[3], s_nsurv;
    __shared__ int s_keep[PROBES_MAX * RT], s_nkeep;                  // per depth, the B-1 best nodes: the only ones the final pick can take
    __shared__ Cand s_list[PROBES_MAX][KP_MAX];                       // Top-K' lists of the probes the next tree uses
    __shared__ float s_lse[PROBES_MAX];
    unsigned long long* c_key = reinterpret_cast<unsigned long long*>(c_rank + MAX_CAND);   // total-order keys
    unsigned long long* c_sort = c_key + MAX_CAND;                                           // scratch of the sorts

    pdl_wait();
    const Dims& D = A.D;
    const int seq = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    SeqState* st = A.states + seq;
    // where this launch's record goes; every sequence, active or not, counts the handle's decode steps
    const unsigned long long rec_no = st->rec;
    int32_t* rec = A.out_ring + ((size_t)(A.is_step ? (int)(rec_no % NREC) : NREC) * D.batch + seq) * RING;
    __syncthreads();      // every thread has read the counter
    if (A.is_step && tid == 0) st->rec = rec_no + 1;
    if (!st->active) {
        if (tid == 0) rec[0] = 0;
        return;
    }
    const int mode = st->mode;
    const int N0 = st->n_nodes, L0 = st->L;
    const int grow0 = seq * RT;

    if (mode == 1) {  // prefill chunk: every row is a prompt token and is already in place
        if (tid == 0) st->L = L0 + N0;
        return;
    }
    for (int r = tid; r < N0; r += nt) {
        s_rtok[r] = st->row_token[r];
        s_rpar[r] = st->row_parent[r];
        s_rdep[r] = st->row_depth[r];
        s_arg[r] = A.topk[(size_t)(grow0 + r) * KP_MAX].id;
    }
    __syncthreads();

    // ---- verification (Section 2): follow the model's own next token through the tree
    if (tid == 0) {
        int a = 0, cur, n_emit = 0;
        s_abort = 0;
        if (mode == 2) {
            cur = N0 - 1;  // last prompt token; nothing to verify, its argmax is the first generated token
            s_path[0] = cur;
            s_out[n_emit++] = s_arg[cur];
            s_ustar = cur;
            s_delta = 0;
        } else {
            cur = 0;
            s_path[0] = 0;
            for (;;) {
                int y = s_arg[cur];
                s_out[n_emit++] = y;
                int nxt = -1;
                for (int c = cur + 1; c < N0; ++c)
                    if (s_rpar[c] == cur && s_rtok[c] == y) { nxt = c; break; }
                if (nxt < 0 || n_emit > PROBES_MAX) break;
                cur = nxt;
                s_path[++a] = cur;
            }
            // deepest anchored node on the accepted path
            int nA = D.k > 0 ? (D.n_anchor == 0 ? N0 : min(D.n_anchor, N0)) : 0;
            int us = 0;
            for (int j = 0; j <= a; ++j) if (s_path[j] < nA) us = s_path[j];
            s_ustar = us;
            s_delta = a - s_rdep[us];
        }
        s_na = a;
        st->n_out = n_emit;
        for (int j = 0; j < n_emit; ++j) st->out_tokens[j] = s_out[j];
        rec[0] = n_emit;
        rec[1] = mode == 2 ? L0 + N0 : L0 + a + 1;
        for (int j = 0; j < n_emit; ++j) rec[2 + j] = s_out[j];
        if (mode == 0) {
            const int rows = st->n_rows;
            st->rows_hist[rows <= 16 ? 0 : (rows <= 32 ? 1 : (rows <= 64 ? 2 : 3))] += 1;
            st->steps += 1;
            st->emitted += n_emit;
            st->accept_hist[a < PROBES_MAX ? a : PROBES_MAX] += 1;
        }
    }
    __syncthreads();
    const int a_acc = s_na;
    const int n_emit = mode == 2 ? 1 : a_acc + 1;

    // ---- KV compaction: cache slot L+j <- row p_j for the accepted path (row 0 is already at slot L).
    // Sources sit at or above their destination, so increasing j with a barrier in between is safe.
    if (mode == 0) {
        const int vec_per_row = D.h * (int)sizeof(T) / 16;
        const size_t layer_stride = (size_t)D.batch * D.Hkv * D.cap * D.h;
        const int per_j = D.n_layers * D.Hkv * 2 * vec_per_row;
        for (int j = 1; j <= a_acc; ++j) {
            const int src = L0 + s_path[j], dst = L0 + j;
            if (src != dst) {
                for (int i = tid; i < per_j; i += nt) {
                    int v = i % vec_per_row, rest = i / vec_per_row;
                    int kv = rest & 1;
                    rest >>= 1;
                    int hh = rest % D.Hkv, l = rest / D.Hkv;
                    T* basep = reinterpret_cast<T*>(kv ? A.vcache : A.kcache) + (size_t)l * layer_stride +
                               ((size_t)seq * D.Hkv + hh) * D.cap * D.h;
                    const uint4* s4 = reinterpret_cast<const uint4*>(basep + (size_t)src * D.h) + v;
                    uint4* d4 = reinterpret_cast<uint4*>(basep + (size_t)dst * D.h) + v;
                    *d4 = *s4;
                }
            }
            __syncthreads();
        }
    }
    const int Lnew = mode == 2 ? L0 + N0 : L0 + a_acc + 1;

    // ---- mask update, Eq. (mask_update_mean): m <- m + lambda (e - m)
    {
        const T* E = reinterpret_cast<const T*>(A.embed);
        float* m = A.mvec + (size_t)seq * D.mask_slots * D.d;
        // four consecutive elements per thread; every load of a pass is issued before the first store
        const int e0 = D.ema_per_token ? 0 : n_emit - 1;
        for (int j = tid * 4; j < D.d; j += nt * 4) {
            float ev[PROBES_MAX + 2][4];
            float4 mv[PROBES_MAX];
            for (int e = e0; e < n_emit; ++e)
#pragma unroll
                for (int i = 0; i < 4; ++i) ev[e][i] = j + i < D.d ? to_f32(E[(size_t)s_out[e] * D.d + j + i]) : 0.f;
            const bool vec = j + 4 <= D.d;
#pragma unroll
            for (int slot = 0; slot < PROBES_MAX; ++slot) {
                if (slot < D.mask_slots) {
                    float* ms = m + (size_t)slot * D.d + j;
                    mv[slot] = vec ? *reinterpret_cast<const float4*>(ms)
                                   : make_float4(ms[0], j + 1 < D.d ? ms[1] : 0.f, j + 2 < D.d ? ms[2] : 0.f, 0.f);
                }
            }
#pragma unroll
            for (int slot = 0; slot < PROBES_MAX; ++slot) {      // every mask vector follows the same update
                if (slot < D.mask_slots) {
                    float x[4] = {mv[slot].x, mv[slot].y, mv[slot].z, mv[slot].w};
                    for (int e = e0; e < n_emit; ++e)
#pragma unroll
                        for (int i = 0; i < 4; ++i) x[i] = __fadd_rn(x[i], __fmul_rn(D.lambda, __fsub_rn(ev[e][i], x[i])));
                    float* ms = m + (size_t)slot * D.d + j;
                    if (vec) *reinterpret_cast<float4*>(ms) = make_float4(x[0], x[1], x[2], x[3]);
                    else for (int i = 0; i < 4 && j + i < D.d; ++i) ms[i] = x[i];
                }
            }
        }
    }

    // ---- next tree (Algorithm 1 with the pruner).  Depth i draws from probe delta+i of u*.
    const int root_tok = s_out[n_emit - 1];
    const int ustar = s_ustar, delta = s_delta;
    const int Dd = D.k - delta > 0 ? D.k - delta : 0;
    if (tid == 0) {
        c_tok[0] = root_tok; c_par[0] = -1; c_dep[0] = 0; c_lp[0] = 0.f;
        s_exp[0] = 0; s_nexp = 1; s_ncreated = 1; s_nkeep = 0;
    }
    // the probe lists the tree draws from, staged once
    for (int w = tid; w < Dd * KP_MAX; w += nt) {
        const int i = w / KP_MAX + 1, q = w % KP_MAX;
        const int prow = mode == 2 ? N0 + (i - 1) : N0 + ustar * D.k + (delta + i - 1);
        s_list[i - 1][q] = A.topk[(size_t)(grow0 + prow) * KP_MAX + q];
        if (q == 0) s_lse[i - 1] = A.lse[grow0 + prow];
    }
    __syncthreads();
    for (int i = 1; i <= Dd; ++i) {
        // Algorithm 1 draws min(K, B-i) candidates per expanded node; a static tree its fixed width for this depth
        const int pool = D.static_w[0] > 0 ? D.static_w[i - 1] : min(D.K, D.B - i);
        if (pool <= 0) break;
        const Cand* list = s_list[i - 1];
        const float lse_i = s_lse[i - 1];
        const int base = s_ncreated, n_exp = s_nexp;
        const int n_new = n_exp * pool;
        if (base + n_new > MAX_CAND) { if (tid == 0) { set_error(A.err, DEV_E_TREE_OVERFLOW); s_abort = 1; } }
        __syncthreads();
        if (s_abort) break;
        for (int w = tid; w < n_new; w += nt) {
            const int e = w / pool, j = w % pool;
            const int p = s_exp[e];
            const int ptok = c_tok[p];
            int seen = 0, q = 0;
            for (; q < D.KP; ++q) {
                int t = list[q].id;
                if (D.prune_parent && t == ptok) continue;
                if (D.prune_root && t == root_tok) continue;
                if (seen == j) break;
                ++seen;
            }
            const int c = base + w;
            if (q < D.KP && list[q].id >= 0) {
                c_tok[c] = list[q].id;
                c_lp[c] = __fadd_rn(c_lp[p], __fsub_rn(list[q].val, lse_i));
            } else {  // list exhausted (cannot happen when K' = K + pruner flags): never selectable
                c_tok[c] = -1;
                c_lp[c] = -INFINITY;
            }
            c_par[c] = p;
            c_dep[c] = i;
            c_key[c] = node_key(c_lp[c], i, c);
        }
        __syncthreads();
        const int width = D.W == 0 ? D.B - i : min(D.W, D.B - i);
        // Ranks of the new nodes among themselves (same depth: logP desc, creation asc) matter only below
        // R = max(width, B-1).  With many new nodes, first find by bisection on the keys' high words (the logP
        // part) the smallest bound that at least R keys do not exceed; only the nodes within it are ranked.
        const int R = min(max(width, D.B - 1), RT);
        const int n_kept = min(min(D.B - 1, RT), n_new), keep0 = s_nkeep;
        int* surv = reinterpret_cast<int*>(c_sort);     // creation indices of the nodes that may rank below R
        int n_surv = n_new;
        if (n_new > 4 * R) {
            unsigned hk[MAX_CAND / 1024];               // high words of this thread's keys (n_new <= MAX_CAND)
            bool hv[MAX_CAND / 1024];
#pragma unroll
            for (int q = 0; q < MAX_CAND / 1024; ++q) {
                const int w = tid + q * nt;
                hv[q] = w < n_new;
                hk[q] = hv[q] ? (unsigned)(c_key[base + w] >> 32) : 0u;
            }
            if (tid == 0) { s_cnt[0] = 0; s_cnt[1] = 0; s_cnt[2] = 0; s_nsurv = 0; }
            __syncthreads();
            unsigned lo = 0u, hi = 0xffffffffu;         // count(high word <= hi) >= R throughout
            for (int it = 0; lo < hi; ++it) {
                const unsigned mid = lo + ((hi - lo) >> 1);
                if (tid == 0) s_cnt[(it + 1) % 3] = 0;  // last read two barriers ago
                int mine = 0;
#pragma unroll
                for (int q = 0; q < MAX_CAND / 1024; ++q) mine += (hv[q] && hk[q] <= mid) ? 1 : 0;
                mine = __reduce_add_sync(0xffffffffu, mine);
                if ((tid & 31) == 0 && mine) atomicAdd(&s_cnt[it % 3], mine);
                __syncthreads();
                if (s_cnt[it % 3] >= R) hi = mid; else lo = mid + 1;
            }
#pragma unroll
            for (int q = 0; q < MAX_CAND / 1024; ++q)
                if (hv[q] && hk[q] <= lo) surv[atomicAdd(&s_nsurv, 1)] = base + tid + q * nt;
            __syncthreads();
            n_surv = s_nsurv;
        } else {
            for (int w = tid; w < n_new; w += nt) surv[w] = base + w;
            __syncthreads();
        }
        for (int w = tid; w < n_surv; w += nt) {
            const int c = surv[w];
            const unsigned long long key = c_key[c];
            int rank = 0;
            for (int o = 0; o < n_surv; ++o) rank += c_key[surv[o]] < key ? 1 : 0;
            if (rank < width && c_tok[c] >= 0) s_exp[rank] = c;
            // a node with B-1 or more nodes of its own depth before it cannot be among the B-1 best overall
            if (rank < n_kept) s_keep[keep0 + rank] = c;
        }
        __syncthreads();
        if (tid == 0) { s_ncreated = base + n_new; s_nexp = min(width, n_new); s_nkeep = keep0 + n_kept; }
        __syncthreads();
    }
    // final selection: root + the B-1 best created nodes by (logP desc, depth asc, creation asc)
    // (ranked among the kept nodes only: every node that precedes one of the B-1 best is itself kept)
    const int n_keep = s_nkeep;
    for (int r = tid; r < RT; r += nt) s_sel[r] = -1;
    __syncthreads();
    for (int w = tid; w < n_keep; w += nt) {
        const int c = s_keep[w];
        const unsigned long long key = c_key[c];
        int rank = 0;
        for (int o = 0; o < n_keep; ++o) rank += c_key[s_keep[o]] < key ? 1 : 0;
        c_rank[c] = rank;
        if (rank < D.B - 1 && c_tok[c] >= 0 && rank < RT) s_sel[rank] = c;
    }
    __syncthreads();
    int n_sel = min(D.B - 1, n_keep);
    // (entries with token -1 rank last because their logP is -inf; drop them)
    if (tid == 0) {
        int n = 0;
        while (n < n_sel && s_sel[n] >= 0) ++n;
        s_nexp = n;
    }
    __syncthreads();
    n_sel = s_nexp;
    // breadth-first row order: by depth, ties by selection rank
    for (int r = tid; r < n_sel; r += nt) {
        const int c = s_sel[r], dp = c_dep[c];
        int idx = 1;
        for (int o = 0; o < n_sel; ++o) {
            const int d2 = c_dep[s_sel[o]];
            idx += (d2 < dp || (d2 == dp && o < r)) ? 1 : 0;
        }
        s_new[r] = idx;
        c_rank[c] = idx;  // creation index -> new row index
    }
    if (tid == 0) c_rank[0] = 0;
    __syncthreads();
    const int N = n_sel + 1;
    for (int r = tid; r < n_sel; r += nt) {
        const int c = s_sel[r], row = s_new[r];
        st->row_token[row] = c_tok[c];
        st->row_parent[row] = c_rank[c_par[c]];
        st->row_depth[row] = c_dep[c];
        st->row_logp[row] = c_lp[c];
        // ancestor-or-self mask by walking up the creation-time parents
        unsigned long long lo = 0, hi = 0;
        for (int x = c; x >= 0; x = c_par[x]) {
            int b = c_rank[x];
            if (b < 64) lo |= 1ull << b; else hi |= 1ull << (b - 64);
        }
        st->row_anc[row][0] = lo;
        st->row_anc[row][1] = hi;
    }
    if (tid == 0) {
        st->row_token[0] = root_tok; st->row_parent[0] = -1; st->row_depth[0] = 0; st->row_logp[0] = 0.f;
        st->row_anc[0][0] = 1ull; st->row_anc[0][1] = 0ull;
    }
    __syncthreads();
    const int nA = D.k > 0 ? (D.n_anchor == 0 ? N : min(D.n_anchor, N)) : 0;
    write_probe_rows(st, N, D.k, 0, nA);
    if (tid == 0) {
        st->n_nodes = N;
        st->n_rows = N + nA * D.k;
        st->L = Lnew;
        st->mode = 0;
        st->forced = 0;
        if (Lnew + RT > D.cap) set_error(A.err, DEV_E_CAPACITY);
    }
}

void launch_tree_step(int dtype, const TreeArgs& A, cudaStream_t s, bool pdl) {
    size_t smem = (size_t)MAX_CAND * 36;
    if (dtype == 0) {
        ensure_dynamic_smem(reinterpret_cast<const void*>(k_tree_step<float>), (int)smem);
        launch_k(k_tree_step<float>, dim3(A.D.batch), dim3(1024), smem, s, pdl, A);
    } else {
        ensure_dynamic_smem(reinterpret_cast<const void*>(k_tree_step<__nv_bfloat16>), (int)smem);
        launch_k(k_tree_step<__nv_bfloat16>, dim3(A.D.batch), dim3(1024), smem, s, pdl, A);
    }
}

// ------------------------------------------------------------------ thin launch wrappers
void launch_rope_table(float* cs, float* sn, int n_pos, int h, float base, cudaStream_t s) {
    int n = n_pos * (h / 2);
    k_rope_table<<<(n + 255) / 256, 256, 0, s>>>(cs, sn, n_pos, h, base);
}
void launch_mask_init(int dtype, const void* embed, const int32_t* prompt, int t, int d, float* m, int slots, int mode, cudaStream_t s) {
    if (dtype == 0) k_mask_init<float><<<(d + 127) / 128, 128, 0, s>>>((const float*)embed, prompt, t, d, m, slots, mode);
    else k_mask_init<__nv_bfloat16><<<(d + 127) / 128, 128, 0, s>>>((const __nv_bfloat16*)embed, prompt, t, d, m, slots, mode);
}
void launch_assemble(int dtype, const SeqState* st, const void* embed, const float* mvec, float* hres, int d, int mask_slots,
                     int batch, cudaStream_t s, bool pdl, int rows_cap) {
    dim3 grid(rows_cap, batch);
    if (dtype == 0) launch_k(k_assemble<float>, grid, dim3(128), 0, s, pdl, st, (const float*)embed, mvec, hres, d, mask_slots);
    else launch_k(k_assemble<__nv_bfloat16>, grid, dim3(128), 0, s, pdl, st, (const __nv_bfloat16*)embed, mvec, hres, d, mask_slots);
}
void launch_rmsnorm(int dtype, const SeqState* st, const float* x, const void* g, void* y, int d, float eps, int batch,
                    float* copy_out, cudaStream_t s, bool pdl) {
    dim3 grid(RT, batch);
    if (dtype == 0) launch_k(k_rmsnorm<float>, grid, dim3(256), 0, s, pdl, st, x, (const float*)g, (float*)y, d, eps, copy_out);
    else launch_k(k_rmsnorm<__nv_bfloat16>, grid, dim3(256), 0, s, pdl, st, x, (const __nv_bfloat16*)g, (__nv_bfloat16*)y, d, eps, copy_out);
}
void launch_resid_norm(const SeqState* st, float* hres, const StreamK& sk, const void* g, void* y, void* y_lo, int d, float eps,
                       float* copy_out, int nq, cudaStream_t s, bool pdl, int rows_cap) {
    launch_k(k_resid_norm<__nv_bfloat16>, dim3(rows_cap, nq), dim3(1024), 0, s, pdl, st, hres, sk, (const __nv_bfloat16*)g,
             (__nv_bfloat16*)y, (__nv_bfloat16*)y_lo, d, eps, copy_out);
}
void launch_swiglu_finish(const SeqState* st, const StreamK& sk, void* act, void* act_lo, int F, int nq, cudaStream_t s, bool pdl, int rows_cap) {
    launch_k(k_swiglu_finish, dim3((F / 8 + 255) / 256, rows_cap, nq), dim3(256), 0, s, pdl, st, 0, sk, (__nv_bfloat16*)act,
             (__nv_bfloat16*)act_lo, F);
}
int launch_qkv_finish(const EpiArgs& a, const StreamK& sk, int nq, cudaStream_t s, bool pdl, int rows_cap) {
    const int n_heads = a.Hq + 2 * a.Hkv;
    dim3 grid((n_heads + 3) / 4, rows_cap, nq);
    if (a.h == 128) launch_k(k_qkv_finish<128>, grid, dim3(128), 0, s, pdl, a, sk);
    else if (a.h == 64) launch_k(k_qkv_finish<64>, grid, dim3(128), 0, s, pdl, a, sk);
    else if (a.h == 32) launch_k(k_qkv_finish<32>, grid, dim3(128), 0, s, pdl, a, sk);
    else return -1;
    return 0;
}
void launch_setup_chain(SeqState* st, int seq, const int32_t* prompt_dev, int off, int n, int last, int k, cudaStream_t s) {
    k_setup_chain<<<1, 128, 0, s>>>(st, seq, prompt_dev, off, n, last, k);
}
void launch_set_tree(SeqState* st, int seq, const int32_t* tokens, const int32_t* parents, int n, int k, int n_anchor,
                     int* err, cudaStream_t s) {
    k_set_tree<<<1, 128, 0, s>>>(st, seq, tokens, parents, n, k, n_anchor, err);
}

}  // namespace esp
