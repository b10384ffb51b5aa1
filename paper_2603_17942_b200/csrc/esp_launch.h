// Host-side launch interface between the translation units of the library.
#pragma once

#include "esp_common.cuh"

namespace esp {

struct AttnArgs {
    const void* q;        // [batch][RT][Hq][h]
    const void* kc;       // [batch][Hkv][cap][h]
    const void* vc;
    void* out;            // [batch][RT][Hq][h]
    void* out_lo;         // optional (tensor-core path): low-order bf16 plane of out, out = hi + lo
    float* part_o;        // [batch*RT][Hq][n_split_max][h]
    float2* part_ml;      // [batch*RT][Hq][n_split_max]
    const SeqState* st;   // NULL -> use the explicit fields below
    const unsigned long long* anc;  // [batch][RT][2]
    const int32_t* depth;           // [batch][RT]
    int32_t rows_cap;               // no block of this launch has more rows than this (0: RT); sizes the grids
    int32_t cache_in_flight;        // 1: positions below T0 may have been written by the kernel before this one
                                    // (prefill blocks: a row's earlier rows sit in the cache already)
    int32_t n_rows_fixed, L_fixed;
    int32_t Hq, Hkv, h, cap, split_len, n_split_max, dcap;
    float scale_log2;     // log2(e)/sqrt(h)
    int* err;
};

struct TreeArgs {
    Dims D;
    SeqState* states;
    const Cand* topk;   // [batch*RT][KP_MAX]
    const float* lse;   // [batch*RT]
    float* mvec;        // [batch][mask_slots][d]
    const void* embed;
    void* kcache;       // [n_layers][batch][Hkv][cap][h]
    void* vcache;
    int* err;
    int32_t* out_ring;  // [NREC + 1][batch][RING]: n_out, new L, tokens  (copied to the host by esp_read)
    int32_t is_step;    // 1: a decode step (record slot = steps so far % NREC), 0: a prefill block (slot NREC)
};


void launch_rope_table(float* cs, float* sn, int n_pos, int h, float base, cudaStream_t s);
void launch_gumbel_noise(uint32_t key0, uint32_t key1, uint32_t position, int n, float* out, cudaStream_t s);
void launch_mask_init(int dtype, const void* embed, const int32_t* prompt, int t, int d, float* m, int slots, int mode, cudaStream_t s);
void launch_assemble(int dtype, const SeqState* st, const void* embed, const float* mvec, float* hres, int d, int mask_slots,
                     int batch, cudaStream_t s, bool pdl, int rows_cap = RT);
void launch_rmsnorm(int dtype, const SeqState* st, const float* x, const void* g, void* y, int d, float eps, int batch,
                    float* copy_out, cudaStream_t s, bool pdl);
// consumers of the split (EPI_PARTIAL) tensor-core GEMMs, bf16 models; nq = sequences the GEMM launch covered
// y_lo / act_lo: optional low-order planes (the next GEMM then reads the activation as hi + lo)
void launch_resid_norm(const SeqState* st, float* hres, const StreamK& sk, const void* g, void* y, void* y_lo, int d, float eps,
                       float* copy_out, int nq, cudaStream_t s, bool pdl, int rows_cap = RT);
int launch_qkv_finish(const EpiArgs& a, const StreamK& sk, int nq, cudaStream_t s, bool pdl, int rows_cap = RT);
void launch_swiglu_finish(const SeqState* st, const StreamK& sk, void* act, void* act_lo, int F, int nq, cudaStream_t s, bool pdl, int rows_cap = RT);
void launch_setup_chain(SeqState* st, int seq, const int32_t* prompt_dev, int off, int n, int last, int k, cudaStream_t s);
void launch_set_tree(SeqState* st, int seq, const int32_t* tokens, const int32_t* parents, int n, int k, int n_anchor,
                     int* err, cudaStream_t s);
void launch_topk_merge(const SeqState* st, const Cand* cand, const float2* cand_ms, int n_tiles, int KP, int batch,
                       Cand* topk, float* lse, cudaStream_t s, bool pdl, int rows_cap = RT, uint32_t* cand_floor = nullptr);
void launch_tree_step(int dtype, const TreeArgs& A, cudaStream_t s, bool pdl);

// CUDA-core GEMM (fp32 models; on-GPU cross-check for bf16)
void launch_gemm_simt(int dtype, int epi, int n_tiles, int batch, const void* const w[3], const int32_t rows_w[3],
                      const void* x, int K, const EpiArgs& a, cudaStream_t s, bool pdl);

// position-canonical attention: CUDA-core bulk (+ tail/merge), or tail/merge only when the
// tensor-core bulk kernel already produced the split partials
int launch_attn_simt(int dtype, const AttnArgs& a, int batch, int n_split_launch, bool bulk_too, cudaStream_t s, bool pdl);
// bf16, head_dim 128: tcgen05 bulk kernel over the cache below each row's T0, then tail + merge (esp_attn_tc.cu).
// A plan holds the TMA descriptors of one query buffer and one layer's KV cache.
struct AttnTc;
bool attn_tc_supported(int h, int Hq, int Hkv);

// Length of the cache splits of tree attention: a power of two >= 256 positions, at most 16 splits of max_len.
// A split is one work item per (sequence, KV head, row tile) and leaves one partial per (row, head), so the
// choice trades items for partial traffic.  One sequence keeps the finest split (the items are what fills the
// SMs).  With several sequences the groups alone fill them, and the length is the one a small cost model prefers:
// waves of items over the SMs x (1.45 us per 128-key chunk + 2.6 us per item) + the items' partial traffic.
// It depends on nothing but the handle's capacity, batch and head count, so every row of a handle sees one
// split grid, whatever the block it arrives in.
inline int attn_split_len(int max_len, int batch, int Hkv) {
    int S = 256;
    while ((max_len + S - 1) / S > 16) S *= 2;
    if (batch <= 1) return S;
    const double groups = (double)batch * Hkv * 3;   // 3 row tiles: up to 96 rows x 4 heads of a group
    int best = S;
    double best_t = 0;
    for (int c = S;; c *= 2) {
        const int splits = (max_len + c - 1) / c;
        const double items = splits * groups;
        const double waves = (double)(long long)((items + 147) / 148);
        const double t = waves * ((c / 128) * 1.45 + 2.6) + items * 0.02;
        if (c == S || t < best_t) { best = c; best_t = t; }
        if (splits == 1) break;
    }
    return best;
}
int attn_tc_create(AttnTc** out, const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap);
void attn_tc_destroy(AttnTc* t);
int attn_tc_launch(const AttnTc* t, const AttnArgs& a, int batch, int n_split_launch, cudaStream_t s, bool pdl);
// the same for one call, descriptors built in the call's own frame (no allocation anywhere)
int attn_tc_run(const void* q, const void* kcache, const void* vcache, int batch, int Hq, int Hkv, int cap, const AttnArgs& a,
                int n_split_launch, cudaStream_t s);

// tcgen05 GEMM: a plan holds the TMA descriptors and the stream-K partition of one weight shape
struct TcGemm;
// epi selects the tile -> weight-row mapping and the fused epilogue; with defer the kernel only stores partials
// (EPI_PARTIAL) and the caller runs the matching consumer kernel.  x: activations [x_seqs][RT][K]; nrs = rows of a
// block that take part (80, or RT for blocks of more than 80 rows); a deferred plan may cover up to nq_max
// sequences per launch, so that the weights are streamed once for all of them.  planes = 2 (deferred plans only):
// x holds the activations as hi + lo bf16 pairs, [2][x_seqs][RT][K], and every product is taken with both
int tc_gemm_create(TcGemm** out, int epi, bool defer, const void* const w[3], const int32_t rows_w[3], int K, const void* x,
                   int x_seqs, int nrs, int nq_max, void* partials, size_t partial_bytes, int* counters, int n_sm, int* err, TileSrc* table_dev,
                   int table_entries, void* packed, cudaStream_t stream, int planes = 1);
// bytes of the repacked copy of a weight set (tc_gemm_create's `packed`; NULL there = stream the caller's matrices)
size_t tc_gemm_packed_bytes(int epi, const int32_t rows_w[3], int K);
void tc_gemm_destroy(TcGemm* g);
int tc_gemm_launch(const TcGemm* g, const EpiArgs& a, cudaStream_t s, bool pdl, int nq = 1, int b_seq0 = 0);
StreamK tc_gemm_streamk(const TcGemm* g, int nq = 1);
int tc_wait_selftest(int* err_dev, cudaStream_t s);
int tc_gemm_tiles(const TcGemm* g);
size_t tc_gemm_partial_bytes(int n_sm, int nq = 1, int nrs = 80);
int tc_gemm_max_nq(int nrs = 80, int planes = 1);
int tc_gemm_counter_ints();


// All layers of a step in one persistent cooperative launch (esp_layers_tc.cu): bf16, head_dim 128, blocks of at
// most 80 rows, one sequence per pass.  Same phases, same partition and same bits as the kernels above.
struct LayersTc;
struct LayersTcDesc {
    const TcGemm* gemm[4];         // layer 0's QKV, O, gate/up and down plans (every layer has the same geometry)
    const void* packed;            // layer 0's repacked weights; pk_layer bytes per layer
    size_t pk_layer;
    float* hres;
    void *xn, *qbuf, *attn_out, *act;
    void *xn_lo, *attn_out_lo, *act_lo;   // low-order planes of the GEMM inputs
    void *kcache, *vcache;         // [n_layers][batch][Hkv][cap][h]
    size_t layer_kv_stride;        // bytes
    const void* const* norm_attn;  // device arrays of n_layers device pointers
    const void* const* norm_ffn;
    const void* const* q_norm;
    const void* const* k_norm;
    const float *rope_cos, *rope_sin;
    int32_t n_layers, d, Hq, Hkv, h, F, cap, qk_norm, batch;
    float rms_eps;
    float* part_o;
    float2* part_ml;
    int32_t split_len, n_split_max, dcap;
    float scale_log2;
    unsigned int* sync_counter;    // zero when the plan is made; the kernel counts it up
    int* err;
    int32_t n_sm;
};
bool layers_tc_supported(const LayersTcDesc& d);
int layers_tc_create(LayersTc** out, const LayersTcDesc& d);
void layers_tc_destroy(LayersTc* t);
int layers_tc_grid(const LayersTc* t);
int layers_tc_syncs_per_layer();
int layers_tc_trace_slots();   // time stamps per barrier in the timeline
unsigned int layers_tc_arrivals(const LayersTc* t);   // what one launch adds to the barrier counter
// seq: the sequence's index in the cache; sync_base: the counter's value when the kernel starts;
// timeline: optional [n_layers * layers_tc_syncs_per_layer()] device words, CTA 0's global timer after every barrier
int layers_tc_launch(LayersTc* t, const SeqState* st, int seq, void* kcache_seq, void* vcache_seq, unsigned int sync_base,
                     unsigned long long* timeline, cudaStream_t s);

}  // namespace esp
