// Shared declarations of the ESP B200 library: device state layout, launch
// parameters and small device helpers.  Everything here is device/product
// code; the CPU oracle shares none of it.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/esp.h"

namespace esp {

constexpr int RT = ESP_MAX_ROWS;        // rows of one block per sequence
constexpr int KP_MAX = ESP_MAX_KPRIME;  // Top-K' entries kept per row
constexpr int PROBES_MAX = ESP_MAX_PROBES;
constexpr int TILE_N = 128;             // output features per GEMM tile
constexpr int MAX_CAND = 4096;          // nodes Algorithm 1 may create in one step
constexpr int PREFILL_CHUNK = ESP_PREFILL_CHUNK;   // prompt rows per prefill block
constexpr int DCAP_STEP = 16;           // tail cap of decode steps (>= 2k)
constexpr int DCAP_PREFILL = 16;        // tail cap of prefill blocks: their earlier rows are cache positions already
constexpr int RING = ESP_MAX_PROBES + 4; // per-sequence result record: n_out, L, tokens
// Result records: a decode step writes every sequence's record into slot (steps so far) % NREC, so that steps
// enqueued without a read in between keep their results; the prefill uses slot NREC.  [NREC + 1][batch][RING].
constexpr int NREC = ESP_MAX_UNREAD_STEPS;

// device error codes (first one recorded wins)
enum : int {
    DEV_OK = 0,
    DEV_E_WAIT_TIMEOUT = 1,   // a bounded mbarrier wait ran out
    DEV_E_INDEX = 2,          // an index left its range
    DEV_E_TREE_OVERFLOW = 3,  // Algorithm 1 would create more than MAX_CAND nodes
    DEV_E_CAPACITY = 4        // KV cache would overflow
};

// Per-sequence device state.  The row table describes the block the next
// forward pass runs: tree nodes first (breadth-first, parent < child), then
// the mask-probe rows (Figure 3 of the paper: all mask rows at the end).
struct SeqState {
    int32_t L;         // cached positions
    int32_t n_nodes;   // N, tree nodes incl. root
    int32_t n_rows;    // N + probe rows
    int32_t mode;      // 0 decode step, 1 prefill chunk (not last), 2 last prefill chunk
    int32_t active;    // takes part in the next forward pass
    int32_t ready;     // prefilled
    int32_t n_out;     // tokens emitted by the last step
    int32_t out_tokens[PROBES_MAX + 2];
    int32_t forced;    // next tree was set by the caller (informational)
    int32_t row_token[RT];   // -1 for probe rows
    int32_t row_parent[RT];  // parent row (probe j>1: previous probe; probe 1: its anchor)
    int32_t row_depth[RT];   // position of the row minus L
    unsigned long long row_anc[RT][2];  // ancestor-or-self bitmask over rows
    float row_logp[RT];
    unsigned long long steps, emitted;
    unsigned long long accept_hist[PROBES_MAX + 1];
    unsigned long long rec;       // decode steps launched on the handle so far (every sequence counts alike): next record slot
    unsigned long long rows_hist[4];   // decode steps by rows of their block: <= 16, <= 32, <= 64, more
};

struct Cand {  // one Top-K' entry
    float val;
    int32_t id;
};

// Geometry + spec needed by device code.
struct Dims {
    int32_t n_layers, d, Hq, Hkv, h, F, V, qk_norm;
    int32_t cap;        // KV positions allocated per sequence (max_seq_len + RT)
    int32_t batch;
    int32_t split_len;  // attention split length in positions (multiple of 64)
    int32_t n_split_max;
    float rms_eps;
    // speculation
    int32_t k, K, KP, B, W, n_anchor, prune_parent, prune_root, ema_per_token;
    int32_t static_w[PROBES_MAX];   // fixed branch widths per depth; static_w[0] == 0: Algorithm 1
    int32_t mask_slots;             // mask vectors per sequence: max(k, 1)
    float lambda;
    int32_t gemm_rows;              // rows of a block the tensor-core GEMMs carry: 80, or RT for larger blocks
    float inv_temp;                 // 1 / temperature, 0 = greedy matching
    uint32_t seed_lo, seed_hi;      // key of the sampling noise
};

// epilogue selectors of the small-M GEMMs.  EPI_PARTIAL (tensor-core kernel only) finishes nothing: every
// (tile, k-range) segment is stored as an fp32 partial and the kernel that consumes the result sums them.
enum Epi : int { EPI_STORE_F32 = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_SWIGLU = 3, EPI_LOGITS = 4, EPI_PARTIAL = 5 };

// Stream-K partition of a GEMM: the n_tiles*KB (tile, k-block) units are dealt out in equal contiguous
// ranges to G persistent CTAs; CTA c owns units [c*U/G, (c+1)*U/G).  The piece of tile t a CTA computed is
// kept in slot min(t - first tile of the CTA, slots - 1) of that CTA:
// partials[((cta*slots + slot)*rows + row)*TILE_N + feature], rows = seq_rows x the sequences one launch covers
// (row = sequence-in-launch * seq_rows + block row; seq_rows = 80, or RT for blocks of more than 80 rows).
// `table` (device memory, one entry per tile, written once when the GEMM plan is made) lists, in CTA order,
// the cta*slots+slot index of every piece of the tile, so consumer kernels need no partition arithmetic.
struct TileSrc {
    uint16_t n;        // contributors of the tile
    uint16_t idx[15];  // their cta*slots + slot, ascending CTA
};
struct StreamK {
    const float* partials;  // NULL: nothing to sum
    const TileSrc* table;
    int32_t n_tiles, KB, G, slots;
    int32_t rows;           // rows per slot
    int32_t seq_rows;       // rows per sequence within a slot
};
__host__ __device__ __forceinline__ long long sk_begin(long long c, long long U, long long G) { return c * U / G; }
__host__ __device__ __forceinline__ int sk_cta_of_unit(long long u, long long U, long long G) {
    return (int)(((u + 1) * G + U - 1) / U - 1);
}
// contributors of a tile, in the (fixed) order their partials are summed
__host__ __device__ __forceinline__ void sk_contributors(const StreamK& s, int tile, int& c_first, int& c_last) {
    const long long U = (long long)s.n_tiles * s.KB, t0 = (long long)tile * s.KB;
    c_first = sk_cta_of_unit(t0, U, s.G);
    c_last = sk_cta_of_unit(t0 + s.KB - 1, U, s.G);
}
__host__ __device__ __forceinline__ int sk_slot(const StreamK& s, int c, int tile) {
    const long long U = (long long)s.n_tiles * s.KB;
    const int d = tile - (int)(sk_begin(c, U, s.G) / s.KB);
    return d < s.slots - 1 ? d : s.slots - 1;
}
// address of contributor c's partial row of a tile
__device__ __forceinline__ const float* sk_partial(const StreamK& s, int c, int tile, int row) {
    return s.partials + ((size_t)(c * s.slots + sk_slot(s, c, tile)) * s.rows + row) * TILE_N;
}
// Sum over the contributors of `tile`, in CTA order, of the four floats at column f of row r.  The loads of up
// to eight contributors are issued before the first addition (adding the zeros of absent ones changes nothing).
// A tile's table entry does not change after the plan was built: a consumer may fetch it before it waits for the GEMM.
struct SkEntry {
    uint4 e0, e1;
};
__device__ __forceinline__ SkEntry sk_entry(const StreamK& s, int tile) {
    const uint4* e = reinterpret_cast<const uint4*>(s.table + tile);
    SkEntry en;
    en.e0 = __ldg(e);
    en.e1 = __ldg(e + 1);
    return en;
}
__device__ __forceinline__ float4 sk_sum4(const StreamK& s, const SkEntry& en, int r, int f) {
    const uint32_t w[8] = {en.e0.x, en.e0.y, en.e0.z, en.e0.w, en.e1.x, en.e1.y, en.e1.z, en.e1.w};
    const int n = (int)(w[0] & 0xffffu);
    const float* base = s.partials + (size_t)r * TILE_N + f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int cb = 0; cb < 16; cb += 8) {
        if (cb < n) {
            float4 t[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int hw = cb + u + 1;   // halfword holding idx[cb + u]
                t[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (hw < 16 && cb + u < n) {
                    const uint32_t idx = (w[hw >> 1] >> ((hw & 1) * 16)) & 0xffffu;
                    t[u] = __ldcg(reinterpret_cast<const float4*>(base + (size_t)idx * ((size_t)s.rows * TILE_N)));
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { acc.x += t[u].x; acc.y += t[u].y; acc.z += t[u].z; acc.w += t[u].w; }
        }
    }
    return acc;
}

__device__ __forceinline__ float4 sk_sum4(const StreamK& s, int tile, int r, int f) { return sk_sum4(s, sk_entry(s, tile), r, f); }

// Everything an epilogue may need.  One struct for all variants keeps the
// GEMM kernels identical across call sites.
struct EpiArgs {
    int32_t n_out;            // valid output features (ragged last tile is masked)
    const SeqState* st;       // per-sequence state (row counts, L, depths); may be NULL -> rows_fixed
    int32_t rows_fixed;       // used when st == NULL
    int32_t batch;
    // EPI_STORE_F32
    float* y_f32;             // [batch*RT][n_out]
    // EPI_RESID
    float* hres;              // [batch*RT][n_out]
    // EPI_QKV
    void* q_out;              // [batch*RT][Hq*h] T
    void* kcache;             // this layer: [batch][Hkv][cap][h] T
    void* vcache;
    const void* q_norm;       // [h] T or NULL
    const void* k_norm;
    const float* rope_cos;    // [cap][h/2]
    const float* rope_sin;
    int32_t Hq, Hkv, h, cap, qk_norm;
    float rms_eps;
    // EPI_SWIGLU
    void* act_out;            // [batch*RT][F] T
    // EPI_LOGITS
    Cand* cand;               // [n_tiles][batch*RT][KP]
    float2* cand_ms;          // [n_tiles][batch*RT] (max, sum exp)
    int32_t KP;
    int32_t n_tiles;
    float* logits_dump;       // optional [batch*RT][V]
    // optional [batch*RT]: per probe row, a running lower bound of its K'-th largest logit, as an order-preserving
    // unsigned key (0 = nothing known yet).  Tiles add to it; entries below it cannot be in the row's Top-K'.
    uint32_t* cand_floor;
    // sample matching: tree rows pick argmax(logit * samp_inv_temp + Gumbel noise); 0 = greedy matching
    float samp_inv_temp;
    uint32_t samp_key0, samp_key1;
};

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// (value descending, id ascending) strict order used by argmax / Top-K everywhere
__device__ __forceinline__ bool cand_before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

__device__ __forceinline__ void set_error(int* err, int code) {
    if (err) atomicCAS(err, 0, code);
}

// Programmatic dependent launch.  A kernel launched with the attribute may start while its predecessor in
// the stream still runs; pdl_wait() returns once the predecessor has completed and its writes are visible.
// Rule used throughout: before pdl_wait() a kernel touches only immutable inputs (weights) and its own
// shared/tensor memory, and data that kernels before the predecessor wrote only where the predecessor releases
// its dependents after its own wait (the attention kernels; a kernel can only start once all CTAs of the one
// before it have released it or exited).  Both calls are no-ops for a plain launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Raises a kernel's dynamic shared-memory limit once per device (the attribute belongs to the device's copy of the
// function) and tells how many SMs the current device has; both are cached per device, under a lock.
int ensure_dynamic_smem(const void* func, int bytes);     // 0 on success
int current_sm_count();                                   // 0 on failure

// Launch with or without the programmatic-dependent-launch attribute.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                            Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace esp
