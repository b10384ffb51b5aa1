// C ABI of the ESP B200 library: configuration checks, workspace carving,
// prefill, the decode-and-verify step and the stand-alone operators.
#include <math.h>
#include <mutex>
#include <new>
#include <string.h>
#include <vector>

#include "esp_launch.h"

using namespace esp;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carve {
    size_t off = 0;
    char* base = nullptr;
    template <typename T> T* take(size_t n) {
        off = align_up(off, 256);
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

struct Buffers {
    void *kcache, *vcache;
    float* hres;
    void *xn, *qbuf, *attn_out, *act;       // bf16 models: xn, attn_out and act hold two planes (hi, then lo)
    void *xn_lo, *attn_out_lo, *act_lo;      // the low-order planes (NULL for fp32 models)
    float* part_o;
    float2* part_ml;
    Cand* cand;
    float2* cand_ms;
    uint32_t* cand_floor;
    Cand* topk;
    float* lse;
    float* mvec;
    SeqState* states;
    int* err;
    int32_t* out_ring;
    int32_t* prompt_dev;
    int32_t* tree_dev;
    float *rope_cos, *rope_sin;
    void* gemm_partials;
    int* gemm_counters;
    TileSrc* sk_tables;   // [4][SK_TABLE_TILES]: QKV, O, gate/up, down (every layer has the same partition)
    // weights repacked for streaming (bf16 models, one sequence): per layer [qkv | o | gate/up | down], then the LM head
    char* packed;
    size_t pk_qkv, pk_o, pk_gu, pk_down, pk_lm, pk_layer;
    // the all-layers kernel: per-layer pointer tables [4][n_layers] (attention norm, FFN norm, q norm, k norm),
    // its barrier counter and the time stamps of a profiled step
    const void** layer_ptrs;
    unsigned int* sync_counter;
    unsigned long long* timeline;
};
constexpr int SK_TABLE_TILES = 2048;
// bf16 models: the inputs of the layer GEMMs (RMSNorm output, attention output, SiLU*up) reach the tensor cores as
// pairs hi + lo of bf16 numbers, each product taken with both.  With one plane the logits of a 32-layer model
// sit 2.5e-2 of their range from the fp32 reference (worst of 8.7 M logits), with two 1.5e-2; the keys, values,
// queries and probabilities stay single bf16 numbers (the cache is bf16).
constexpr int ACT_PLANES = 2;


// tree nodes including the root: max_nodes, or 1 + the fixed widths of a static tree
int spec_nodes(const esp_spec_cfg& s) {
    if (s.n_probes > 0 && s.static_widths[0] > 0) {
        int n = 1;
        for (int i = 0; i < s.n_probes && i < PROBES_MAX && s.static_widths[i] > 0; ++i) n += s.static_widths[i];
        return n;
    }
    return s.max_nodes;
}
int spec_topk(const esp_spec_cfg& s) {
    if (s.n_probes > 0 && s.static_widths[0] > 0) {
        int m = 0;
        for (int i = 0; i < s.n_probes && i < PROBES_MAX && s.static_widths[i] > 0; ++i) m = s.static_widths[i] > m ? s.static_widths[i] : m;
        return m;
    }
    return s.topk;
}
int spec_rows(const esp_spec_cfg& s) {
    const int B = spec_nodes(s);
    int nA = s.n_probes > 0 ? (s.n_anchor == 0 ? B : (s.n_anchor < B ? s.n_anchor : B)) : 0;
    return B + s.n_probes * nA;
}

int check_cfg(const esp_model_cfg* m, const esp_spec_cfg* s, Dims* D) {
    if (!m || !s) return ESP_E_ARG;
    if (m->dtype != 0 && m->dtype != 1) return ESP_E_BADCFG;
    if (m->n_layers < 1 || m->d_model < 8 || m->d_ffn < 8 || m->vocab < 2) return ESP_E_BADCFG;
    if (m->head_dim != 32 && m->head_dim != 64 && m->head_dim != 128) return ESP_E_BADCFG;
    if (m->n_kv_heads < 1 || m->n_q_heads % m->n_kv_heads) return ESP_E_BADCFG;
    if ((m->n_q_heads * m->head_dim) % TILE_N || (m->n_kv_heads * m->head_dim) % TILE_N) return ESP_E_BADCFG;
    if (m->d_model % 8 || m->d_ffn % 8) return ESP_E_BADCFG;  // 16-byte rows for TMA and vector loads
    if (m->dtype == 1 && m->d_model > 128 * TILE_N) return ESP_E_BADCFG;   // the norm kernels keep one partial per 128 features
    if (m->vocab > 2048 * TILE_N) return ESP_E_BADCFG;
    if (m->max_batch < 1 || m->max_seq_len < 1) return ESP_E_BADCFG;
    if (s->n_probes < 0 || s->n_probes > PROBES_MAX) return ESP_E_BADCFG;
    if (s->max_nodes < 1) return ESP_E_BADCFG;
    const bool is_static = s->n_probes > 0 && s->static_widths[0] > 0;
    for (int i = 0; i < PROBES_MAX; ++i)
        if (s->static_widths[i] < 0 || (i > 0 && s->static_widths[i] > 0 && s->static_widths[i - 1] == 0)) return ESP_E_BADCFG;
    const int topk = spec_topk(*s), n_nodes = spec_nodes(*s);
    const int KP = topk + (s->prune_parent ? 1 : 0) + (s->prune_root ? 1 : 0);
    if (s->n_probes > 0 && (topk < 1 || KP > KP_MAX || KP > m->vocab)) return ESP_E_BADCFG;
    if (spec_rows(*s) > RT) return ESP_E_BADCFG;
    if (2 * s->n_probes > DCAP_STEP) return ESP_E_BADCFG;
    if (s->expand_width < 0 || s->n_anchor < 0) return ESP_E_BADCFG;
    if (s->mask_init < 0 || s->mask_init > 2) return ESP_E_BADCFG;
    if (!(s->temperature >= 0.f) || s->temperature > 1e6f) return ESP_E_BADCFG;
    // Algorithm 1 must not create more than MAX_CAND nodes
    long created = 1, n_exp = 1;
    for (int i = 1; i <= s->n_probes && !is_static; ++i) {
        long pool = s->topk < s->max_nodes - i ? s->topk : s->max_nodes - i;
        if (pool <= 0) break;
        long n_new = n_exp * pool;
        created += n_new;
        long width = s->expand_width == 0 ? s->max_nodes - i : (s->expand_width < s->max_nodes - i ? s->expand_width : s->max_nodes - i);
        n_exp = width < n_new ? width : n_new;
    }
    if (created > MAX_CAND) return ESP_E_BADCFG;
    if (D) {
        D->n_layers = m->n_layers; D->d = m->d_model; D->Hq = m->n_q_heads; D->Hkv = m->n_kv_heads; D->h = m->head_dim;
        D->F = m->d_ffn; D->V = m->vocab; D->qk_norm = m->qk_norm;
        D->cap = m->max_seq_len + RT;
        D->batch = m->max_batch;
        const int S = attn_split_len(m->max_seq_len, m->max_batch, m->n_kv_heads);
        D->split_len = S;
        D->n_split_max = (m->max_seq_len + RT + S - 1) / S + 1;   // a prefill block's own rows count as cache positions
        D->rms_eps = m->rms_eps;
        D->k = s->n_probes; D->K = topk; D->KP = s->n_probes > 0 ? KP : 1; D->B = n_nodes; D->W = is_static ? 1 : s->expand_width;
        D->mask_slots = s->n_probes > 0 ? s->n_probes : 1;
        for (int i = 0; i < PROBES_MAX; ++i) D->static_w[i] = is_static && i < s->n_probes ? s->static_widths[i] : 0;
        D->n_anchor = s->n_anchor; D->prune_parent = s->prune_parent; D->prune_root = s->prune_root;
        D->ema_per_token = s->ema_per_token; D->lambda = s->lambda;
        // rows of a block the tensor-core GEMMs carry: 80 covers every tree of at most 80 rows and the prefill blocks
        D->gemm_rows = spec_rows(*s) <= 80 ? 80 : RT;
        D->inv_temp = s->temperature > 0.f ? 1.0f / s->temperature : 0.f;
        D->seed_lo = s->seed_lo; D->seed_hi = s->seed_hi;
    }
    return ESP_OK;
}

size_t carve_all(const Dims& D, int dtype, int n_sm, char* base, Buffers* b) {
    Carve c;
    c.base = base;
    const size_t es = dtype ? 2 : 4;
    const size_t Mtot = (size_t)D.batch * RT;
    const size_t kv = (size_t)D.n_layers * D.batch * D.Hkv * D.cap * D.h * es;
    const int n_tiles_v = (D.V + TILE_N - 1) / TILE_N;
    Buffers tmp;
    Buffers& o = b ? *b : tmp;
    o.kcache = c.take<char>(kv);
    o.vcache = c.take<char>(kv);
    o.hres = c.take<float>(Mtot * D.d);
    // activations that feed the tensor-core GEMMs are kept as bf16 pairs hi + lo (ACT_PLANES planes, Mtot rows apart)
    const size_t pl = dtype ? ACT_PLANES : 1;
    o.xn = c.take<char>(pl * Mtot * D.d * es);
    o.qbuf = c.take<char>(Mtot * D.Hq * D.h * es);
    o.attn_out = c.take<char>(pl * Mtot * D.Hq * D.h * es);
    o.act = c.take<char>(pl * Mtot * D.F * es);
    o.xn_lo = o.attn_out_lo = o.act_lo = nullptr;
    if (base && pl == 2) {
        o.xn_lo = reinterpret_cast<char*>(o.xn) + Mtot * D.d * es;
        o.attn_out_lo = reinterpret_cast<char*>(o.attn_out) + Mtot * D.Hq * D.h * es;
        o.act_lo = reinterpret_cast<char*>(o.act) + Mtot * D.F * es;
    }
    o.part_o = c.take<float>(Mtot * D.Hq * D.n_split_max * D.h);
    o.part_ml = c.take<float2>(Mtot * D.Hq * D.n_split_max);
    o.cand = c.take<Cand>((size_t)n_tiles_v * Mtot * D.KP);
    o.cand_ms = c.take<float2>((size_t)n_tiles_v * Mtot);
    o.cand_floor = c.take<uint32_t>(Mtot);
    o.topk = c.take<Cand>(Mtot * KP_MAX);
    o.lse = c.take<float>(Mtot);
    o.mvec = c.take<float>((size_t)D.batch * D.mask_slots * D.d);
    o.states = c.take<SeqState>(D.batch);
    o.err = c.take<int>(4);
    o.out_ring = c.take<int32_t>((size_t)(NREC + 1) * D.batch * RING);
    o.prompt_dev = c.take<int32_t>(D.cap);
    o.tree_dev = c.take<int32_t>(2 * RT);
    o.rope_cos = c.take<float>((size_t)D.cap * (D.h / 2));
    o.rope_sin = c.take<float>((size_t)D.cap * (D.h / 2));
    {
        // the decode steps' passes (several sequences of gemm_rows rows) or one 128-row prefill block, whichever is larger
        const size_t step_b = tc_gemm_partial_bytes(n_sm, D.batch < tc_gemm_max_nq(D.gemm_rows, ACT_PLANES) ? D.batch : tc_gemm_max_nq(D.gemm_rows, ACT_PLANES), D.gemm_rows);
        const size_t pre_b = tc_gemm_partial_bytes(n_sm, 1, RT);
        o.gemm_partials = c.take<char>(step_b > pre_b ? step_b : pre_b);
    }
    o.gemm_counters = c.take<int>(tc_gemm_counter_ints());
    o.sk_tables = c.take<TileSrc>(4 * SK_TABLE_TILES);
    o.layer_ptrs = c.take<const void*>((size_t)4 * D.n_layers);
    o.sync_counter = c.take<unsigned int>(64);
    o.timeline = c.take<unsigned long long>((size_t)layers_tc_trace_slots() * D.n_layers * layers_tc_syncs_per_layer() + 8);
    o.packed = nullptr;
    o.pk_qkv = o.pk_o = o.pk_gu = o.pk_down = o.pk_lm = o.pk_layer = 0;
    if (dtype == 1) {
        const int32_t dq = D.Hq * D.h, dkv = D.Hkv * D.h;
        const int32_t r1[3] = {dq, dkv, dkv}, r2[3] = {D.d, 0, 0}, r3[3] = {D.F, D.F, 0}, r5[3] = {D.V, 0, 0};
        o.pk_qkv = tc_gemm_packed_bytes(EPI_PARTIAL, r1, D.d);
        o.pk_o = tc_gemm_packed_bytes(EPI_PARTIAL, r2, dq);
        o.pk_gu = tc_gemm_packed_bytes(EPI_SWIGLU, r3, D.d);
        o.pk_down = tc_gemm_packed_bytes(EPI_PARTIAL, r2, D.F);
        o.pk_lm = tc_gemm_packed_bytes(EPI_LOGITS, r5, D.d);
        o.pk_layer = o.pk_qkv + o.pk_o + o.pk_gu + o.pk_down;
        o.packed = c.take<char>(o.pk_layer * D.n_layers + o.pk_lm);
    }
    return align_up(c.off, 256);
}

}  // namespace

struct esp_handle {
    esp_model_cfg mc;
    esp_spec_cfg sc;
    Dims D;
    Buffers b;
    cudaStream_t stream;
    int dtype, gemm_impl, n_sm;
    int rows_cap = RT;   // no block (step or prefill) has more rows than this
    const void *embed, *lm_head, *final_norm;
    std::vector<const void*> wq, wk, wv, wo, wg, wu, wd, na, nf, qn, kn;
    std::vector<TcGemm*> p_qkv, p_o, p_gu, p_down;
    // the same GEMMs with 128 rows per block for the prefill, when the decode steps use the 80-row kernels
    std::vector<TcGemm*> p_qkv_w, p_o_w, p_gu_w, p_down_w;
    TcGemm* p_lm_w = nullptr;
    int rows_cap_prefill = RT;
    std::vector<AttnTc*> p_attn;   // per layer, bf16 models with head_dim 128
    TcGemm* p_lm = nullptr;
    LayersTc* p_layers = nullptr;  // all layers in one launch (one sequence per pass, blocks of at most 80 rows)
    bool use_layers = false;       // esp_debug_set_layer_kernel (off by default: measured slower than one kernel per operation)
    unsigned int sync_epoch = 0;   // value of the barrier counter after the launches enqueued so far
    std::vector<int> L_host, ready;
    unsigned long long issued = 0;      // decode steps enqueued on this handle
    unsigned long long consumed = 0;    // ... whose records esp_read has returned
    int32_t* pinned = nullptr;  // [batch][RING] + 4 ints (error words)
    float *dbg_logits = nullptr, *dbg_hidden = nullptr;
    int launches = 0, kernels_per_step = 0;
    size_t layer_kv_stride = 0;  // bytes
    bool prof = false;           // record an event after every kernel group
    bool use_pdl = true;         // programmatic dependent launch between the kernels of a step
    bool use_graph = true;       // replay the step's launch sequence as a CUDA graph
    struct StepGraph { unsigned long long key; cudaGraphExec_t exec; int kernels; };
    std::vector<StepGraph> graphs;
    std::vector<cudaEvent_t> ev;
    std::vector<int> ev_kind;
    size_t ev_used = 0;
};

namespace {

int cuda_ok(cudaError_t e) { return e == cudaSuccess ? ESP_OK : ESP_E_CUDA; }

enum { KIND_MISC = 0, KIND_QKV, KIND_ATTN, KIND_O, KIND_GATEUP, KIND_DOWN, KIND_LMHEAD, KIND_SELECT, KIND_N, KIND_FUSED };

void mark(esp_handle* h, int kind) {
    if (!h->prof) return;
    if (h->ev_used == h->ev.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        h->ev.push_back(e);
        h->ev_kind.push_back(0);
    }
    h->ev_kind[h->ev_used] = kind;
    cudaEventRecord(h->ev[h->ev_used++], h->stream);
}

void* layer_ptr(void* base, size_t stride_bytes, int l) { return reinterpret_cast<char*>(base) + stride_bytes * l; }

// One forward pass covers sequences [s0, s0 + nb): all of them on the CUDA-core path (nb = max_batch), one at a
// time on the tensor-core path (nb = 1; the activation buffers are shared, only the sequence state, the KV
// cache, the mask vectors and the selection results are per sequence).
EpiArgs base_epi(esp_handle* h, int n_out, int s0, int nb) {
    EpiArgs a;
    memset(&a, 0, sizeof(a));
    a.n_out = n_out;
    a.st = h->b.states + s0;
    a.batch = nb;
    a.Hq = h->D.Hq; a.Hkv = h->D.Hkv; a.h = h->D.h; a.cap = h->D.cap; a.qk_norm = h->D.qk_norm;
    a.rms_eps = h->D.rms_eps;
    a.rope_cos = h->b.rope_cos; a.rope_sin = h->b.rope_sin;
    a.KP = h->D.KP;
    a.samp_inv_temp = h->D.inv_temp; a.samp_key0 = h->D.seed_lo; a.samp_key1 = h->D.seed_hi;
    return a;
}

int run_gemm(esp_handle* h, TcGemm* plan, int epi, int n_tiles, const void* const w[3], const int32_t rows_w[3],
             const void* x, int K, const EpiArgs& a, bool tc, bool pdl, int nq = 1, int b_row0 = 0) {
    h->launches++;
    if (tc) return tc_gemm_launch(plan, a, h->stream, pdl, nq, b_row0);
    launch_gemm_simt(h->dtype, epi, n_tiles, h->D.batch, w, rows_w, x, K, a, h->stream, pdl);
    return ESP_OK;
}

// One decoder forward over the block every active sequence of [s0, s0 + nb) has in its row table.
// Tensor-core path (bf16, nb <= 3 sequences whose activation blocks sit RT rows apart): the layer GEMMs stream
// their weights once for all nb sequences and store stream-K partials that the next kernel sums (k_qkv_finish;
// k_resid_norm = residual add + RMSNorm; k_swiglu_finish); the LM head runs once per sequence and finishes
// in-kernel.  CUDA-core path (fp32 models): the same layer with every epilogue fused in the GEMM.
int forward_pass(esp_handle* h, bool with_lm, int dcap, int s0, int nb, bool tc, bool prefill) {
    const Dims& D = h->D;
    Buffers& b = h->b;
    cudaStream_t s = h->stream;
    const int dq = D.Hq * D.h, dkv = D.Hkv * D.h;
    const size_t es = h->dtype ? 2 : 4;
    int Lmax = 0;
    for (int i = s0; i < s0 + nb; ++i) Lmax = h->L_host[i] > Lmax ? h->L_host[i] : Lmax;
    // a prefill block's rows attend to the block's earlier rows through the cache as well
    const int n_split_launch = (Lmax + (prefill ? RT : 0) + D.split_len - 1) / D.split_len;
    const bool pdl = h->use_pdl && !h->prof;
    SeqState* st0 = b.states + s0;
    const size_t kv_seq_off = (size_t)s0 * D.Hkv * D.cap * D.h * es;   // this pass's first sequence inside a layer's cache
    float* mvec0 = b.mvec + (size_t)s0 * D.mask_slots * D.d;
    StreamK pending;   // partials of the last down projection, summed by the next norm
    pending.partials = nullptr; pending.table = nullptr; pending.n_tiles = 0; pending.KB = 1; pending.G = 1; pending.slots = 2; pending.rows = RT; pending.seq_rows = RT;
    mark(h, -1);
    const int rc_rows = prefill ? h->rows_cap_prefill : h->rows_cap;   // no block has more rows: sizes the row dimension of the grids
    const bool wide = prefill && !h->p_qkv_w.empty();                  // 128-row GEMM plans for the prefill blocks
    auto plan = [&](std::vector<TcGemm*>& narrow, std::vector<TcGemm*>& w128, int l) -> TcGemm* { return wide ? w128[l] : narrow[l]; };
    launch_assemble(h->dtype, st0, h->embed, mvec0, b.hres, D.d, D.mask_slots, nb, s, false, rc_rows);
    h->launches++;
    // One sequence, a block of at most 80 rows, bf16: every layer in one persistent launch (same bits as the
    // kernel-per-operation path below, which serves batches, prefill blocks and larger blocks).
    const bool fused = tc && nb == 1 && !prefill && h->p_layers && h->use_layers;
    if (fused) {
        mark(h, KIND_MISC);
        const int rc = layers_tc_launch(h->p_layers, st0, s0, reinterpret_cast<char*>(b.kcache) + kv_seq_off,
                                        reinterpret_cast<char*>(b.vcache) + kv_seq_off, h->sync_epoch, h->prof ? b.timeline : nullptr, s);
        if (rc) return rc;
        h->sync_epoch += layers_tc_arrivals(h->p_layers);
        h->launches++;
        mark(h, KIND_FUSED);
        pending = tc_gemm_streamk(h->p_down[D.n_layers - 1], 1);
    }
    for (int l = 0; l < D.n_layers && !fused; ++l) {
        if (tc) launch_resid_norm(st0, b.hres, pending, h->na[l], b.xn, b.xn_lo, D.d, D.rms_eps, nullptr, nb, s, pdl, rc_rows);
        else launch_rmsnorm(h->dtype, st0, b.hres, h->na[l], b.xn, D.d, D.rms_eps, nb, nullptr, s, pdl);
        h->launches++;
        mark(h, KIND_MISC);
        {
            EpiArgs a = base_epi(h, dq + 2 * dkv, s0, nb);
            a.q_out = b.qbuf;
            a.kcache = reinterpret_cast<char*>(layer_ptr(b.kcache, h->layer_kv_stride, l)) + kv_seq_off;
            a.vcache = reinterpret_cast<char*>(layer_ptr(b.vcache, h->layer_kv_stride, l)) + kv_seq_off;
            a.q_norm = D.qk_norm ? h->qn[l] : nullptr;
            a.k_norm = D.qk_norm ? h->kn[l] : nullptr;
            const void* w[3] = {h->wq[l], h->wk[l], h->wv[l]};
            const int32_t rows[3] = {dq, dkv, dkv};
            int rc = run_gemm(h, tc ? plan(h->p_qkv, h->p_qkv_w, l) : nullptr, EPI_QKV, (dq + 2 * dkv) / TILE_N, w, rows, b.xn, D.d, a, tc, pdl, tc ? nb : 1);
            if (rc) return rc;
            mark(h, KIND_QKV);
            if (tc) {
                if (launch_qkv_finish(a, tc_gemm_streamk(plan(h->p_qkv, h->p_qkv_w, l), nb), nb, s, pdl, rc_rows)) return ESP_E_BADCFG;
                h->launches++;
                mark(h, KIND_MISC);
            }
        }
        {
            AttnArgs a;
            memset(&a, 0, sizeof(a));
            a.q = b.qbuf;
            a.kc = reinterpret_cast<char*>(layer_ptr(b.kcache, h->layer_kv_stride, l)) + kv_seq_off;
            a.vc = reinterpret_cast<char*>(layer_ptr(b.vcache, h->layer_kv_stride, l)) + kv_seq_off;
            a.out = b.attn_out;
            a.out_lo = tc ? b.attn_out_lo : nullptr;
            a.part_o = b.part_o; a.part_ml = b.part_ml;
            a.st = st0;
            a.Hq = D.Hq; a.Hkv = D.Hkv; a.h = D.h; a.cap = D.cap; a.split_len = D.split_len; a.n_split_max = D.n_split_max;
            a.dcap = dcap;
            a.rows_cap = rc_rows;
            a.cache_in_flight = prefill ? 1 : 0;
            a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)D.h));
            a.err = b.err;
            if (tc && !h->p_attn.empty()) {
                if (attn_tc_launch(h->p_attn[(size_t)l * D.batch + s0], a, nb, n_split_launch, s, pdl)) return ESP_E_BADCFG;
                h->launches += n_split_launch > 0 ? 2 : 1;
            } else {
                if (launch_attn_simt(h->dtype, a, nb, n_split_launch, true, s, pdl)) return ESP_E_BADCFG;
                h->launches += n_split_launch > 0 ? 2 : 1;
            }
            mark(h, KIND_ATTN);
        }
        {
            EpiArgs a = base_epi(h, D.d, s0, nb);
            a.hres = b.hres;
            const void* w[3] = {h->wo[l], nullptr, nullptr};
            const int32_t rows[3] = {D.d, 0, 0};
            int rc = run_gemm(h, tc ? plan(h->p_o, h->p_o_w, l) : nullptr, EPI_RESID, (D.d + TILE_N - 1) / TILE_N, w, rows, b.attn_out, dq, a, tc, pdl, tc ? nb : 1);
            if (rc) return rc;
            mark(h, KIND_O);
        }
        if (tc) launch_resid_norm(st0, b.hres, tc_gemm_streamk(plan(h->p_o, h->p_o_w, l), nb), h->nf[l], b.xn, b.xn_lo, D.d, D.rms_eps, nullptr, nb, s, pdl, rc_rows);
        else launch_rmsnorm(h->dtype, st0, b.hres, h->nf[l], b.xn, D.d, D.rms_eps, nb, nullptr, s, pdl);
        h->launches++;
        mark(h, KIND_MISC);
        {
            EpiArgs a = base_epi(h, D.F, s0, nb);
            a.act_out = b.act;
            const void* w[3] = {h->wg[l], h->wu[l], nullptr};
            const int32_t rows[3] = {D.F, D.F, 0};
            int rc = run_gemm(h, tc ? plan(h->p_gu, h->p_gu_w, l) : nullptr, EPI_SWIGLU, (D.F + 63) / 64, w, rows, b.xn, D.d, a, tc, pdl, tc ? nb : 1);
            if (rc) return rc;
            mark(h, KIND_GATEUP);
            if (tc) {
                launch_swiglu_finish(st0, tc_gemm_streamk(plan(h->p_gu, h->p_gu_w, l), nb), b.act, b.act_lo, D.F, nb, s, pdl, rc_rows);
                h->launches++;
                mark(h, KIND_MISC);
            }
        }
        {
            EpiArgs a = base_epi(h, D.d, s0, nb);
            a.hres = b.hres;
            const void* w[3] = {h->wd[l], nullptr, nullptr};
            const int32_t rows[3] = {D.d, 0, 0};
            int rc = run_gemm(h, tc ? plan(h->p_down, h->p_down_w, l) : nullptr, EPI_RESID, (D.d + TILE_N - 1) / TILE_N, w, rows, b.act, D.F, a, tc, pdl, tc ? nb : 1);
            if (rc) return rc;
            if (tc) pending = tc_gemm_streamk(plan(h->p_down, h->p_down_w, l), nb);
            mark(h, KIND_DOWN);
        }
    }
    if (with_lm) {
        float* dbg_hidden = h->dbg_hidden ? h->dbg_hidden + (size_t)s0 * RT * D.d : nullptr;
        if (tc) launch_resid_norm(st0, b.hres, pending, h->final_norm, b.xn, nullptr, D.d, D.rms_eps, dbg_hidden, nb, s, pdl, rc_rows);   // the LM head reads one plane
        else launch_rmsnorm(h->dtype, st0, b.hres, h->final_norm, b.xn, D.d, D.rms_eps, nb, dbg_hidden, s, pdl);
        h->launches++;
        mark(h, KIND_MISC);
        const int n_tiles = (D.V + TILE_N - 1) / TILE_N;
        // tensor-core path: the LM head and its selection run once per sequence (the candidate lists are shared)
        const int n_lm = tc ? nb : 1, per = tc ? 1 : nb;
        for (int q = 0; q < n_lm; ++q) {
            const int sq = s0 + q;
            EpiArgs a = base_epi(h, D.V, sq, per);
            a.cand = b.cand; a.cand_ms = b.cand_ms; a.cand_floor = b.cand_floor; a.n_tiles = n_tiles;
            a.logits_dump = h->dbg_logits ? h->dbg_logits + (size_t)sq * RT * D.V : nullptr;
            const void* w[3] = {h->lm_head, nullptr, nullptr};
            const int32_t rows[3] = {D.V, 0, 0};
            int rc = run_gemm(h, wide ? h->p_lm_w : h->p_lm, EPI_LOGITS, n_tiles, w, rows, b.xn, D.d, a, tc, pdl, 1, q);
            if (rc) return rc;
            mark(h, KIND_LMHEAD);
            launch_topk_merge(b.states + sq, b.cand, b.cand_ms, n_tiles, D.KP, per, b.topk + (size_t)sq * RT * KP_MAX, b.lse + (size_t)sq * RT, s, pdl, rc_rows, b.cand_floor);
            h->launches++;
            mark(h, KIND_SELECT);
        }
    }
    return cuda_ok(cudaGetLastError());
}

// Forward over the sequences that take part: `only_seq` (prefill) or every prefilled sequence (a step).
int forward(esp_handle* h, bool with_lm, int dcap, int only_seq) {
    const bool tc = h->dtype == 1 && h->gemm_impl == 0 && h->p_lm != nullptr;
    const bool prefill = only_seq >= 0;
    if (!tc) return forward_pass(h, with_lm, dcap, 0, h->D.batch, false, prefill);
    if (only_seq >= 0) return forward_pass(h, with_lm, dcap, only_seq, 1, true, true);
    // consecutive sequences share a pass (and a weight stream); sequences that are not ready are inactive in it
    const int per_pass = tc_gemm_max_nq(h->D.gemm_rows, ACT_PLANES);
    for (int s0 = 0; s0 < h->D.batch; s0 += per_pass) {
        const int nb = h->D.batch - s0 < per_pass ? h->D.batch - s0 : per_pass;
        bool any = false;
        for (int i = s0; i < s0 + nb; ++i) any = any || h->ready[i];
        if (!any) continue;
        const int rc = forward_pass(h, with_lm, dcap, s0, nb, true, false);
        if (rc) return rc;
    }
    return ESP_OK;
}

int tree_step(esp_handle* h, bool is_step) {
    TreeArgs A;
    A.is_step = is_step ? 1 : 0;
    A.D = h->D;
    A.states = h->b.states;
    A.topk = h->b.topk;
    A.lse = h->b.lse;
    A.mvec = h->b.mvec;
    A.embed = h->embed;
    A.kcache = h->b.kcache;
    A.vcache = h->b.vcache;
    A.err = h->b.err;
    A.out_ring = h->b.out_ring;
    launch_tree_step(h->dtype, A, h->stream, h->use_pdl && !h->prof);
    h->launches++;
    mark(h, KIND_SELECT);
    return cuda_ok(cudaGetLastError());
}

void drop_graphs(esp_handle* h) {
    for (auto& g : h->graphs) cudaGraphExecDestroy(g.exec);
    h->graphs.clear();
}

__global__ void k_select(SeqState* st, int batch, int seq_only) {
    int i = threadIdx.x;
    if (i < batch) st[i].active = seq_only < 0 ? st[i].ready : (i == seq_only);
}
__global__ void k_mark_ready(SeqState* st, int seq) { st[seq].ready = 1; }

// Copies the records of slot `slot` (all sequences) and the error word to pinned memory; synchronises.
int read_ring(esp_handle* h, int slot) {
    const int n = h->D.batch * RING;
    if (cudaMemcpyAsync(h->pinned, h->b.out_ring + (size_t)slot * n, sizeof(int32_t) * n, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return ESP_E_CUDA;
    if (cudaMemcpyAsync(h->pinned + n, h->b.err, sizeof(int), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return ESP_E_CUDA;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return ESP_E_CUDA;
    return h->pinned[n] ? ESP_E_DEVICE : ESP_OK;
}

}  // namespace

extern "C" {

int esp_workspace_bytes(const esp_model_cfg* model, const esp_spec_cfg* spec, size_t* bytes_out) {
    if (!bytes_out) return ESP_E_ARG;
    Dims D;
    int rc = check_cfg(model, spec, &D);
    if (rc) return rc;
    *bytes_out = carve_all(D, model->dtype, 148, nullptr, nullptr);
    return ESP_OK;
}

int esp_init(const esp_model_cfg* model, const esp_spec_cfg* spec, const esp_weights* w, void* workspace,
             size_t workspace_bytes, void* cuda_stream, esp_handle** handle_out) {
    if (!handle_out || !w || !workspace) return ESP_E_ARG;
    Dims D;
    int rc = check_cfg(model, spec, &D);
    if (rc) return rc;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return ESP_E_WORKSPACE;
    size_t need = carve_all(D, model->dtype, 148, nullptr, nullptr);
    if (workspace_bytes < need) return ESP_E_WORKSPACE;
    if (!w->embed || !w->lm_head || !w->final_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up ||
        !w->w_down || !w->norm_attn || !w->norm_ffn)
        return ESP_E_ARG;
    if (model->qk_norm && (!w->q_norm || !w->k_norm)) return ESP_E_ARG;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ESP_E_CUDA;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return ESP_E_CUDA;
    if (n_sm > 148) n_sm = 148;
    esp_handle* h = new (std::nothrow) esp_handle();
    if (!h) return ESP_E_ARG;
    h->mc = *model; h->sc = *spec; h->D = D;
    h->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    h->dtype = model->dtype;
    h->gemm_impl = model->dtype == 0 ? 1 : 0;
    h->n_sm = n_sm;
    {
        const int step_rows = spec_rows(*spec), pre_rows = PREFILL_CHUNK + spec->n_probes;
        h->rows_cap = step_rows > RT ? RT : step_rows;
        h->rows_cap_prefill = pre_rows > RT ? RT : pre_rows;
    }
    carve_all(D, model->dtype, 148, reinterpret_cast<char*>(workspace), &h->b);
    h->embed = w->embed; h->lm_head = w->lm_head; h->final_norm = w->final_norm;
    for (int l = 0; l < D.n_layers; ++l) {
        h->wq.push_back(w->wq[l]); h->wk.push_back(w->wk[l]); h->wv.push_back(w->wv[l]); h->wo.push_back(w->wo[l]);
        h->wg.push_back(w->w_gate[l]); h->wu.push_back(w->w_up[l]); h->wd.push_back(w->w_down[l]);
        h->na.push_back(w->norm_attn[l]); h->nf.push_back(w->norm_ffn[l]);
        h->qn.push_back(model->qk_norm ? w->q_norm[l] : nullptr); h->kn.push_back(model->qk_norm ? w->k_norm[l] : nullptr);
    }
    h->L_host.assign(D.batch, 0);
    h->ready.assign(D.batch, 0);
    h->layer_kv_stride = (size_t)D.batch * D.Hkv * D.cap * D.h * (model->dtype ? 2 : 4);
    if (cudaMemsetAsync(workspace, 0, need, h->stream) != cudaSuccess) { delete h; return ESP_E_CUDA; }
    if (cudaHostAlloc(reinterpret_cast<void**>(&h->pinned), sizeof(int32_t) * (D.batch * RING + 4), cudaHostAllocDefault) != cudaSuccess) {
        delete h;
        return ESP_E_CUDA;
    }
    launch_rope_table(h->b.rope_cos, h->b.rope_sin, D.cap, D.h, model->rope_base, h->stream);
    if (model->dtype == 1 && attn_tc_supported(D.h, D.Hq, D.Hkv)) {
        const size_t seq_bytes = (size_t)D.Hkv * D.cap * D.h * 2;
        for (int l = 0; l < D.n_layers; ++l) {
            for (int i = 0; i < D.batch; ++i) {      // a pass starting at sequence i: the layer's cache from there on, the shared q buffer
                AttnTc* t = nullptr;
                char* kc = reinterpret_cast<char*>(layer_ptr(h->b.kcache, h->layer_kv_stride, l)) + seq_bytes * i;
                char* vc = reinterpret_cast<char*>(layer_ptr(h->b.vcache, h->layer_kv_stride, l)) + seq_bytes * i;
                if (attn_tc_create(&t, h->b.qbuf, kc, vc, D.batch - i, D.Hq, D.Hkv, D.cap)) { esp_free(h); return ESP_E_CUDA; }
                h->p_attn.push_back(t);
            }
        }
    }
    if (model->dtype == 1) {
        const int dq = D.Hq * D.h, dkv = D.Hkv * D.h;
        const int nrs = D.gemm_rows;
        const int nq_max = D.batch < tc_gemm_max_nq(nrs, ACT_PLANES) ? D.batch : tc_gemm_max_nq(nrs, ACT_PLANES);   // sequences sharing a weight stream
        bool ok = true;
        for (int l = 0; l < D.n_layers && ok; ++l) {
            TcGemm* p = nullptr;
            char* pk = h->b.packed + h->b.pk_layer * l;
            const void* w1[3] = {h->wq[l], h->wk[l], h->wv[l]};
            const int32_t r1[3] = {dq, dkv, dkv};
            ok = ok && !tc_gemm_create(&p, EPI_PARTIAL, true, w1, r1, D.d, h->b.xn, D.batch, nrs, nq_max, h->b.gemm_partials, tc_gemm_partial_bytes(148, nq_max, nrs), h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 0 * SK_TABLE_TILES, SK_TABLE_TILES, pk, h->stream, ACT_PLANES);
            h->p_qkv.push_back(p);
            const void* w2[3] = {h->wo[l], nullptr, nullptr};
            const int32_t r2[3] = {D.d, 0, 0};
            p = nullptr;
            ok = ok && !tc_gemm_create(&p, EPI_PARTIAL, true, w2, r2, dq, h->b.attn_out, D.batch, nrs, nq_max, h->b.gemm_partials, tc_gemm_partial_bytes(148, nq_max, nrs), h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 1 * SK_TABLE_TILES, SK_TABLE_TILES, pk + h->b.pk_qkv, h->stream, ACT_PLANES);
            h->p_o.push_back(p);
            const void* w3[3] = {h->wg[l], h->wu[l], nullptr};
            const int32_t r3[3] = {D.F, D.F, 0};
            p = nullptr;
            ok = ok && !tc_gemm_create(&p, EPI_SWIGLU, true, w3, r3, D.d, h->b.xn, D.batch, nrs, nq_max, h->b.gemm_partials, tc_gemm_partial_bytes(148, nq_max, nrs), h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 2 * SK_TABLE_TILES, SK_TABLE_TILES, pk + h->b.pk_qkv + h->b.pk_o, h->stream, ACT_PLANES);
            h->p_gu.push_back(p);
            const void* w4[3] = {h->wd[l], nullptr, nullptr};
            const int32_t r4[3] = {D.d, 0, 0};
            p = nullptr;
            ok = ok && !tc_gemm_create(&p, EPI_PARTIAL, true, w4, r4, D.F, h->b.act, D.batch, nrs, nq_max, h->b.gemm_partials, tc_gemm_partial_bytes(148, nq_max, nrs), h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 3 * SK_TABLE_TILES, SK_TABLE_TILES, pk + h->b.pk_qkv + h->b.pk_o + h->b.pk_gu, h->stream, ACT_PLANES);
            h->p_down.push_back(p);
        }
        const void* w5[3] = {h->lm_head, nullptr, nullptr};
        const int32_t r5[3] = {D.V, 0, 0};
        ok = ok && !tc_gemm_create(&h->p_lm, EPI_LOGITS, false, w5, r5, D.d, h->b.xn, D.batch, nrs, 1, h->b.gemm_partials, tc_gemm_partial_bytes(148, nq_max, nrs), h->b.gemm_counters, n_sm, h->b.err, nullptr, 0, h->b.packed + h->b.pk_layer * D.n_layers, h->stream);
        if (ok && nrs != RT) {
            // the prefill runs 120-row blocks: the same weights (already repacked) behind 128-row GEMM plans
            const size_t pbytes = tc_gemm_partial_bytes(148, 1, RT);
            for (int l = 0; l < D.n_layers && ok; ++l) {
                TcGemm* p = nullptr;
                char* pk = h->b.packed + h->b.pk_layer * l;
                const void* w1[3] = {h->wq[l], h->wk[l], h->wv[l]};
                const int32_t r1[3] = {dq, dkv, dkv};
                ok = ok && !tc_gemm_create(&p, EPI_PARTIAL, true, w1, r1, D.d, h->b.xn, D.batch, RT, 1, h->b.gemm_partials, pbytes, h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 0 * SK_TABLE_TILES, SK_TABLE_TILES, pk, h->stream, ACT_PLANES);
                h->p_qkv_w.push_back(p);
                const void* w2[3] = {h->wo[l], nullptr, nullptr};
                const int32_t r2[3] = {D.d, 0, 0};
                p = nullptr;
                ok = ok && !tc_gemm_create(&p, EPI_PARTIAL, true, w2, r2, dq, h->b.attn_out, D.batch, RT, 1, h->b.gemm_partials, pbytes, h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 1 * SK_TABLE_TILES, SK_TABLE_TILES, pk + h->b.pk_qkv, h->stream, ACT_PLANES);
                h->p_o_w.push_back(p);
                const void* w3[3] = {h->wg[l], h->wu[l], nullptr};
                const int32_t r3[3] = {D.F, D.F, 0};
                p = nullptr;
                ok = ok && !tc_gemm_create(&p, EPI_SWIGLU, true, w3, r3, D.d, h->b.xn, D.batch, RT, 1, h->b.gemm_partials, pbytes, h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 2 * SK_TABLE_TILES, SK_TABLE_TILES, pk + h->b.pk_qkv + h->b.pk_o, h->stream, ACT_PLANES);
                h->p_gu_w.push_back(p);
                const void* w4[3] = {h->wd[l], nullptr, nullptr};
                const int32_t r4[3] = {D.d, 0, 0};
                p = nullptr;
                ok = ok && !tc_gemm_create(&p, EPI_PARTIAL, true, w4, r4, D.F, h->b.act, D.batch, RT, 1, h->b.gemm_partials, pbytes, h->b.gemm_counters, n_sm, h->b.err, h->b.sk_tables + 3 * SK_TABLE_TILES, SK_TABLE_TILES, pk + h->b.pk_qkv + h->b.pk_o + h->b.pk_gu, h->stream, ACT_PLANES);
                h->p_down_w.push_back(p);
            }
            ok = ok && !tc_gemm_create(&h->p_lm_w, EPI_LOGITS, false, w5, r5, D.d, h->b.xn, D.batch, RT, 1, h->b.gemm_partials, pbytes, h->b.gemm_counters, n_sm, h->b.err, nullptr, 0, h->b.packed + h->b.pk_layer * D.n_layers, h->stream);
        }
        if (!ok) { esp_free(h); return ESP_E_CUDA; }
        // the all-layers kernel: per-layer pointer tables and the plan
        if (nrs == 80 && D.batch == 1) {
            std::vector<const void*> tab((size_t)4 * D.n_layers, nullptr);
            for (int l = 0; l < D.n_layers; ++l) {
                tab[0 * D.n_layers + l] = h->na[l]; tab[1 * D.n_layers + l] = h->nf[l];
                tab[2 * D.n_layers + l] = h->qn[l]; tab[3 * D.n_layers + l] = h->kn[l];
            }
            if (cudaMemcpyAsync(h->b.layer_ptrs, tab.data(), sizeof(void*) * tab.size(), cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
                cudaStreamSynchronize(h->stream) != cudaSuccess) { esp_free(h); return ESP_E_CUDA; }
            LayersTcDesc ld;
            memset(&ld, 0, sizeof(ld));
            ld.gemm[0] = h->p_qkv[0]; ld.gemm[1] = h->p_o[0]; ld.gemm[2] = h->p_gu[0]; ld.gemm[3] = h->p_down[0];
            ld.packed = h->b.packed; ld.pk_layer = h->b.pk_layer;
            ld.hres = h->b.hres; ld.xn = h->b.xn; ld.qbuf = h->b.qbuf; ld.attn_out = h->b.attn_out; ld.act = h->b.act;
            ld.xn_lo = h->b.xn_lo; ld.attn_out_lo = h->b.attn_out_lo; ld.act_lo = h->b.act_lo;
            ld.kcache = h->b.kcache; ld.vcache = h->b.vcache; ld.layer_kv_stride = h->layer_kv_stride;
            ld.norm_attn = h->b.layer_ptrs; ld.norm_ffn = h->b.layer_ptrs + D.n_layers;
            ld.q_norm = h->b.layer_ptrs + 2 * D.n_layers; ld.k_norm = h->b.layer_ptrs + 3 * D.n_layers;
            ld.rope_cos = h->b.rope_cos; ld.rope_sin = h->b.rope_sin;
            ld.n_layers = D.n_layers; ld.d = D.d; ld.Hq = D.Hq; ld.Hkv = D.Hkv; ld.h = D.h; ld.F = D.F; ld.cap = D.cap;
            ld.qk_norm = D.qk_norm; ld.batch = D.batch; ld.rms_eps = D.rms_eps;
            ld.part_o = h->b.part_o; ld.part_ml = h->b.part_ml;
            ld.split_len = D.split_len; ld.n_split_max = D.n_split_max; ld.dcap = DCAP_STEP;
            ld.scale_log2 = (float)(1.4426950408889634 / sqrt((double)D.h));
            ld.sync_counter = h->b.sync_counter; ld.err = h->b.err; ld.n_sm = n_sm;
            if (layers_tc_supported(ld) && layers_tc_create(&h->p_layers, ld)) { esp_free(h); return ESP_E_CUDA; }
        }
    }
    if (cudaStreamSynchronize(h->stream) != cudaSuccess || cudaGetLastError() != cudaSuccess) { esp_free(h); return ESP_E_CUDA; }
    *handle_out = h;
    return ESP_OK;
}

int esp_prefill(esp_handle* h, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t* first_token_out) {
    if (!h || !prompt) return ESP_E_ARG;
    if (seq < 0 || seq >= h->D.batch) return ESP_E_ARG;
    if (n_prompt < 1 || n_prompt > h->mc.max_seq_len) return ESP_E_PROMPT;
    for (int i = 0; i < n_prompt; ++i)
        if (prompt[i] < 0 || prompt[i] >= h->D.V) return ESP_E_PROMPT;
    cudaStream_t s = h->stream;
    if (cudaMemcpyAsync(h->b.prompt_dev, prompt, sizeof(int32_t) * n_prompt, cudaMemcpyHostToDevice, s) != cudaSuccess) return ESP_E_CUDA;
    if (h->sc.mask_init != 2)   // 2: the caller's vectors (esp_set_mask) stay
        launch_mask_init(h->dtype, h->embed, h->b.prompt_dev, n_prompt, h->D.d, h->b.mvec + (size_t)seq * h->D.mask_slots * h->D.d,
                         h->D.mask_slots, h->sc.mask_init, s);
    k_select<<<1, 32, 0, s>>>(h->b.states, h->D.batch, seq);
    std::vector<int> saved = h->L_host;
    for (int i = 0; i < h->D.batch; ++i) h->L_host[i] = 0;
    for (int off = 0; off < n_prompt; off += PREFILL_CHUNK) {
        const int cn = n_prompt - off < PREFILL_CHUNK ? n_prompt - off : PREFILL_CHUNK;
        const int last = off + cn == n_prompt;
        launch_setup_chain(h->b.states, seq, h->b.prompt_dev, off, cn, last, h->D.k, s);
        h->L_host[seq] = off;
        int rc = forward(h, last, DCAP_PREFILL, seq);
        if (!rc) rc = tree_step(h, false);
        if (rc) {
            // the other sequences keep their lengths; this one has to be prefilled again before it can step
            k_select<<<1, 32, 0, s>>>(h->b.states, h->D.batch, -1);
            h->L_host = saved;
            h->L_host[seq] = 0;
            h->ready[seq] = 0;
            return rc;
        }
    }
    k_mark_ready<<<1, 1, 0, s>>>(h->b.states, seq);
    k_select<<<1, 32, 0, s>>>(h->b.states, h->D.batch, -1);
    int rc = read_ring(h, NREC);
    h->L_host = saved;
    h->L_host[seq] = n_prompt;
    h->ready[seq] = 1;
    if (rc) return rc;
    if (first_token_out) *first_token_out = h->pinned[seq * RING + 2];
    return ESP_OK;
}

int esp_step_async(esp_handle* h) {
    if (!h) return ESP_E_ARG;
    bool any = false;
    int Lmax = 0;
    for (int i = 0; i < h->D.batch; ++i) {
        if (!h->ready[i]) continue;
        any = true;
        if (h->L_host[i] + h->D.k + 1 + RT > h->D.cap) return ESP_E_FULL;
        Lmax = h->L_host[i] > Lmax ? h->L_host[i] : Lmax;
    }
    if (!any) return ESP_E_STATE;
    if (h->issued - h->consumed >= (unsigned long long)NREC) return ESP_E_STATE;   // every record slot holds an unread step
    int rc = ESP_OK;
    bool done = false;
    // (the all-layers kernel makes a step a handful of launches, and its barrier counter's start value is a launch
    // parameter: such steps are launched directly)
    const bool fused_step = h->p_layers && h->use_layers && h->D.batch == 1 && h->gemm_impl == 0;
    if (h->use_graph && !h->prof && !fused_step) {
        // The launch sequence of a step depends on the host only through the number of attention splits;
        // every other quantity (L, row counts, the tree) is read from device state by the kernels.
        // (key: which sequences take part and how many cache splits each one's attention launches)
        unsigned long long key = 1469598103934665603ull;
        for (int i = 0; i < h->D.batch; ++i) {
            const unsigned long long v = h->ready[i] ? 1ull + (unsigned long long)((h->L_host[i] + h->D.split_len - 1) / h->D.split_len) : 0ull;
            key = (key ^ v) * 1099511628211ull;
        }
        esp_handle::StepGraph* g = nullptr;
        for (auto& e : h->graphs)
            if (e.key == key) g = &e;
        if (!g) {
            cudaGraph_t graph = nullptr;
            cudaGraphExec_t exec = nullptr;
            const int before = h->launches;
            bool ok = cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
            if (ok) {
                int r1 = forward(h, true, DCAP_STEP, -1);
                int r2 = r1 ? r1 : tree_step(h, true);
                ok = cudaStreamEndCapture(h->stream, &graph) == cudaSuccess && !r2 && graph;
            }
            if (ok) ok = cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess;
            if (graph) cudaGraphDestroy(graph);
            if (ok) {
                h->graphs.push_back({key, exec, h->launches - before});
                g = &h->graphs.back();
            } else {
                cudaGetLastError();      // capture is not available here: launch directly from now on
                h->use_graph = false;
            }
        }
        if (g) {
            if (cudaGraphLaunch(g->exec, h->stream) != cudaSuccess) return ESP_E_CUDA;
            h->kernels_per_step = g->kernels;
            done = true;
        }
    }
    if (!done) {
        const int before = h->launches;
        rc = forward(h, true, DCAP_STEP, -1);
        if (rc) return rc;
        rc = tree_step(h, true);
        h->kernels_per_step = h->launches - before;
    }
    if (rc) return rc;
    ++h->issued;
    // until the result is read the host only knows an upper bound of each cache length
    for (int i = 0; i < h->D.batch; ++i)
        if (h->ready[i]) h->L_host[i] += h->D.k + 1;
    return rc;
}

int esp_read(esp_handle* h, int32_t* tokens_out, int32_t* n_out) {
    if (!h) return ESP_E_ARG;
    if (h->consumed == h->issued) {           // nothing unread: only the device status
        if (n_out)
            for (int i = 0; i < h->D.batch; ++i) n_out[i] = 0;
        if (cudaStreamSynchronize(h->stream) != cudaSuccess) return ESP_E_CUDA;
        int e = 0;
        if (cudaMemcpy(&e, h->b.err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
        return e ? ESP_E_DEVICE : ESP_OK;
    }
    int rc = read_ring(h, (int)(h->consumed % NREC));
    ++h->consumed;
    const int unread = (int)(h->issued - h->consumed);
    for (int i = 0; i < h->D.batch; ++i) {
        const int32_t* r = h->pinned + i * RING;
        if (!h->ready[i] || r[0] <= 0) { if (n_out) n_out[i] = 0; continue; }   // took no part in that step
        h->L_host[i] = r[1] + unread * (h->D.k + 1);     // steps still unread can each add at most k + 1 positions
        if (n_out) n_out[i] = r[0];
        if (tokens_out)
            for (int j = 0; j < r[0] && j <= PROBES_MAX; ++j) tokens_out[i * (PROBES_MAX + 1) + j] = r[2 + j];
    }
    return rc;
}

int esp_step(esp_handle* h, int32_t* tokens_out, int32_t* n_out) {
    int rc = esp_step_async(h);
    if (rc) return rc;
    return esp_read(h, tokens_out, n_out);
}

int esp_set_mask(esp_handle* h, int32_t seq, const float* mask) {
    if (!h || !mask) return ESP_E_ARG;
    if (seq < 0 || seq >= h->D.batch) return ESP_E_ARG;
    if (h->sc.n_probes < 1) return ESP_E_STATE;
    const size_t n = (size_t)h->D.mask_slots * h->D.d;
    if (cudaMemcpyAsync(h->b.mvec + (size_t)seq * n, mask, sizeof(float) * n, cudaMemcpyHostToDevice, h->stream) != cudaSuccess) return ESP_E_CUDA;
    return cuda_ok(cudaStreamSynchronize(h->stream));
}

int esp_set_tree(esp_handle* h, int32_t seq, const int32_t* tokens, const int32_t* parents, int32_t n) {
    if (!h || !tokens || !parents) return ESP_E_ARG;
    if (seq < 0 || seq >= h->D.batch || !h->ready[seq]) return ESP_E_STATE;
    const int k = h->D.k;
    const int nA = k > 0 ? (h->D.n_anchor == 0 ? n : (h->D.n_anchor < n ? h->D.n_anchor : n)) : 0;
    if (n < 1 || n + nA * k > h->rows_cap) return ESP_E_ARG;   // the kernels are sized for the configured block
    std::vector<int> depth(n, 0);
    for (int i = 0; i < n; ++i) {
        if (tokens[i] < 0 || tokens[i] >= h->D.V) return ESP_E_ARG;
        if (i == 0 ? parents[i] != -1 : (parents[i] < 0 || parents[i] >= i)) return ESP_E_ARG;
        if (i) depth[i] = depth[parents[i]] + 1;
        if (depth[i] + k > DCAP_STEP || depth[i] > PROBES_MAX) return ESP_E_ARG;
    }
    cudaStream_t s = h->stream;
    if (cudaMemcpyAsync(h->b.tree_dev, tokens, sizeof(int32_t) * n, cudaMemcpyHostToDevice, s) != cudaSuccess) return ESP_E_CUDA;
    if (cudaMemcpyAsync(h->b.tree_dev + RT, parents, sizeof(int32_t) * n, cudaMemcpyHostToDevice, s) != cudaSuccess) return ESP_E_CUDA;
    launch_set_tree(h->b.states, seq, h->b.tree_dev, h->b.tree_dev + RT, n, k, h->D.n_anchor, h->b.err, s);
    return cuda_ok(cudaStreamSynchronize(s));
}

int esp_debug_state(esp_handle* h, int32_t seq, int32_t* row_token, int32_t* row_parent, int32_t* row_depth,
                    int32_t* n_nodes, int32_t* n_rows, int32_t* L, int32_t* topk_ids, float* topk_vals, float* lse,
                    float* mask_vec) {
    if (!h || seq < 0 || seq >= h->D.batch) return ESP_E_ARG;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return ESP_E_CUDA;
    SeqState st;
    if (cudaMemcpy(&st, h->b.states + seq, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
    if (row_token) memcpy(row_token, st.row_token, sizeof(st.row_token));
    if (row_parent) memcpy(row_parent, st.row_parent, sizeof(st.row_parent));
    if (row_depth) memcpy(row_depth, st.row_depth, sizeof(st.row_depth));
    if (n_nodes) *n_nodes = st.n_nodes;
    if (n_rows) *n_rows = st.n_rows;
    if (L) *L = st.L;
    if (topk_ids || topk_vals) {
        std::vector<Cand> c((size_t)RT * KP_MAX);
        if (cudaMemcpy(c.data(), h->b.topk + (size_t)seq * RT * KP_MAX, sizeof(Cand) * c.size(), cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
        for (size_t i = 0; i < c.size(); ++i) {
            if (topk_ids) topk_ids[i] = c[i].id;
            if (topk_vals) topk_vals[i] = c[i].val;
        }
    }
    if (lse && cudaMemcpy(lse, h->b.lse + (size_t)seq * RT, sizeof(float) * RT, cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
    const size_t mbytes = sizeof(float) * h->D.mask_slots * h->D.d;
    if (mask_vec && cudaMemcpy(mask_vec, h->b.mvec + (size_t)seq * h->D.mask_slots * h->D.d, mbytes, cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
    return ESP_OK;
}

int esp_debug_capture(esp_handle* h, float* logits, float* hidden) {
    if (!h) return ESP_E_ARG;
    h->dbg_logits = logits;
    h->dbg_hidden = hidden;
    drop_graphs(h);
    return ESP_OK;
}

int esp_debug_set_gemm(esp_handle* h, int32_t impl) {
    if (!h || (impl != 0 && impl != 1)) return ESP_E_ARG;
    if (h->dtype == 0 && impl == 0) return ESP_E_BADCFG;
    if (impl == 0 && !h->p_lm) return ESP_E_BADCFG;
    h->gemm_impl = impl;
    drop_graphs(h);
    return ESP_OK;
}

int esp_debug_set_layer_kernel(esp_handle* h, int32_t mode) {
    if (!h || (mode != 0 && mode != 1)) return ESP_E_ARG;
    if (mode == 0 && !h->p_layers) return ESP_E_BADCFG;
    h->use_layers = mode == 0;
    drop_graphs(h);
    return ESP_OK;
}

int esp_debug_layer_timeline(esp_handle* h, uint64_t* stamps_ns, int32_t capacity, int32_t* n_out) {
    if (!h || !stamps_ns || !n_out || capacity < 0) return ESP_E_ARG;
    if (!h->p_layers) return ESP_E_BADCFG;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return ESP_E_CUDA;
    const int n = layers_tc_trace_slots() * h->D.n_layers * layers_tc_syncs_per_layer();
    *n_out = n;
    const int m = n < capacity ? n : capacity;
    if (m > 0 && cudaMemcpy(stamps_ns, h->b.timeline, sizeof(uint64_t) * m, cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
    return ESP_OK;
}

int esp_step_profiled(esp_handle* h, float* ms_by_kind, int32_t* tokens_out, int32_t* n_out) {
    if (!h || !ms_by_kind) return ESP_E_ARG;
    h->prof = true;
    h->ev_used = 0;
    int rc = esp_step_async(h);
    h->prof = false;
    if (rc) return rc;
    rc = esp_read(h, tokens_out, n_out);
    for (int i = 0; i < KIND_N; ++i) ms_by_kind[i] = 0.f;
    for (size_t i = 1; i < h->ev_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, h->ev[i - 1], h->ev[i]) != cudaSuccess) return ESP_E_CUDA;
        const int kind = h->ev_kind[i];
        if (kind >= 0 && kind < KIND_N) ms_by_kind[kind] += ms;
        if (kind == KIND_FUSED) {
            // inside the all-layers kernel: the global timer after each grid barrier, ten phases per layer
            // (norm, QKV, q/k/v finish, attention bulk, tail + merge, O, norm, gate/up, SiLU*up, down)
            static const int kind_of_phase[10] = {KIND_MISC, KIND_QKV, KIND_MISC, KIND_ATTN, KIND_ATTN, KIND_O, KIND_MISC, KIND_GATEUP, KIND_MISC, KIND_DOWN};
            const int n = h->D.n_layers * layers_tc_syncs_per_layer();
            const int ts = layers_tc_trace_slots();
            std::vector<unsigned long long> tl((size_t)ts * n);
            if (cudaMemcpy(tl.data(), h->b.timeline, sizeof(unsigned long long) * ts * n, cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
            double inside = 0.0;
            for (int j = 1; j < n; ++j) {
                const double d_ms = (double)(tl[(size_t)ts * j + 1] - tl[(size_t)ts * (j - 1) + 1]) * 1e-6;   // barrier exit to barrier exit
                ms_by_kind[kind_of_phase[j % 10]] += (float)d_ms;
                inside += d_ms;
            }
            if (ms > inside) ms_by_kind[KIND_MISC] += (float)(ms - inside);   // launch, set-up and the first norm
        }
    }
    return rc;
}

int esp_get_stats(esp_handle* h, esp_stats* out) {
    if (!h || !out) return ESP_E_ARG;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return ESP_E_CUDA;
    memset(out, 0, sizeof(*out));
    for (int i = 0; i < h->D.batch; ++i) {
        SeqState st;
        if (cudaMemcpy(&st, h->b.states + i, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
        out->steps += (int64_t)st.steps;
        out->emitted += (int64_t)st.emitted;
        for (int a = 0; a <= PROBES_MAX; ++a) out->accept_hist[a] += (int64_t)st.accept_hist[a];
        for (int a = 0; a < 4; ++a) out->rows_hist[a] += (int64_t)st.rows_hist[a];
    }
    int e = 0;
    if (cudaMemcpy(&e, h->b.err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ESP_E_CUDA;
    out->device_error = e;
    out->kernels_per_step = h->kernels_per_step;
    return ESP_OK;
}

int esp_debug_wait_selftest(void* scratch, void* cuda_stream, int32_t* device_status_out) {
    if (!scratch || !device_status_out) return ESP_E_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    int* err = reinterpret_cast<int*>(scratch);
    if (cudaMemsetAsync(err, 0, 256, s) != cudaSuccess) return ESP_E_CUDA;
    if (tc_wait_selftest(err, s)) return ESP_E_CUDA;
    int e = 0;
    if (cudaMemcpyAsync(&e, err, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ESP_E_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ESP_E_CUDA;
    *device_status_out = e;
    return ESP_OK;
}

int esp_debug_gumbel(uint32_t seed_lo, uint32_t seed_hi, uint32_t position, int32_t n_tokens, float* noise_out,
                     void* cuda_stream) {
    if (!noise_out || n_tokens < 0) return ESP_E_ARG;
    if (n_tokens == 0) return ESP_OK;
    launch_gumbel_noise(seed_lo, seed_hi, position, n_tokens, noise_out, reinterpret_cast<cudaStream_t>(cuda_stream));
    return cuda_ok(cudaGetLastError());
}

void esp_free(esp_handle* h) {
    if (!h) return;
    for (auto* p : h->p_qkv) tc_gemm_destroy(p);
    for (auto* p : h->p_o) tc_gemm_destroy(p);
    for (auto* p : h->p_gu) tc_gemm_destroy(p);
    for (auto* p : h->p_down) tc_gemm_destroy(p);
    tc_gemm_destroy(h->p_lm);
    for (auto* p : h->p_qkv_w) tc_gemm_destroy(p);
    for (auto* p : h->p_o_w) tc_gemm_destroy(p);
    for (auto* p : h->p_gu_w) tc_gemm_destroy(p);
    for (auto* p : h->p_down_w) tc_gemm_destroy(p);
    tc_gemm_destroy(h->p_lm_w);
    layers_tc_destroy(h->p_layers);
    for (auto* t : h->p_attn) attn_tc_destroy(t);
    if (h->pinned) cudaFreeHost(h->pinned);
    drop_graphs(h);
    for (auto e : h->ev) cudaEventDestroy(e);
    delete h;
}

// ------------------------------------------------------------------ stand-alone operators
int esp_tree_attention_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim, int32_t cap, size_t* bytes_out) {
    if (!bytes_out || batch < 1 || n_q_heads < 1 || cap < RT) return ESP_E_ARG;
    const int S = attn_split_len(cap - RT, 1, 1);   // the finest split of this capacity: covers every batch
    const size_t ns = ((size_t)cap + S - 1) / S + 1;
    const size_t rows = (size_t)batch * RT * n_q_heads * ns;
    *bytes_out = align_up(rows * head_dim * sizeof(float), 256) + align_up(rows * sizeof(float2), 256) + 256;
    return ESP_OK;
}

// scratch layout: [error word, 256 bytes][split partials: weighted values][split partials: (max, sum)]
int esp_tree_attention(int32_t dtype, int32_t batch, int32_t n_rows, int32_t L, int32_t cap, int32_t n_q_heads,
                       int32_t n_kv_heads, int32_t head_dim, int32_t dcap, const void* q, const void* kcache,
                       const void* vcache, const uint64_t* anc, const int32_t* depth, void* out, void* scratch,
                       size_t scratch_bytes, void* cuda_stream) {
    if (!q || !kcache || !vcache || !anc || !depth || !out || !scratch) return ESP_E_ARG;
    if (dtype != 0 && dtype != 1) return ESP_E_BADCFG;
    if (head_dim != 32 && head_dim != 64 && head_dim != 128) return ESP_E_BADCFG;
    if (n_kv_heads < 1 || n_q_heads % n_kv_heads || batch < 1) return ESP_E_BADCFG;
    if (n_rows < 1 || n_rows > RT || L < 0 || L + RT > cap || dcap < 16 || dcap % 16) return ESP_E_ARG;
    size_t need = 0;
    esp_tree_attention_scratch_bytes(batch, n_q_heads, head_dim, cap, &need);
    if (scratch_bytes < need || reinterpret_cast<uintptr_t>(scratch) % 256) return ESP_E_WORKSPACE;
    const int S = attn_split_len(cap - RT, batch, n_kv_heads);
    const size_t ns = ((size_t)cap + S - 1) / S + 1;
    const size_t rows = (size_t)batch * RT * n_q_heads * ns;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    char* sc = reinterpret_cast<char*>(scratch);
    // the error word starts at zero (the scratch may hold an earlier call's bytes); the partials are written before they are read
    if (cudaMemsetAsync(sc, 0, 256, s) != cudaSuccess) return ESP_E_CUDA;
    AttnArgs a;
    memset(&a, 0, sizeof(a));
    a.q = q; a.kc = kcache; a.vc = vcache; a.out = out;
    a.part_o = reinterpret_cast<float*>(sc + 256);
    a.part_ml = reinterpret_cast<float2*>(sc + 256 + align_up(rows * head_dim * sizeof(float), 256));
    a.st = nullptr;
    a.anc = reinterpret_cast<const unsigned long long*>(anc);
    a.depth = depth;
    a.n_rows_fixed = n_rows; a.L_fixed = L;
    a.rows_cap = n_rows;      // sizes the grids: no block has more rows
    a.Hq = n_q_heads; a.Hkv = n_kv_heads; a.h = head_dim; a.cap = cap; a.split_len = S; a.n_split_max = (int)ns; a.dcap = dcap;
    a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)head_dim));
    a.err = reinterpret_cast<int*>(sc);
    const int n_split_launch = (L + S - 1) / S;
    const bool mma = dtype == 1 && attn_tc_supported(head_dim, n_q_heads, n_kv_heads);
    if (mma) {
        if (attn_tc_run(q, kcache, vcache, batch, n_q_heads, n_kv_heads, cap, a, n_split_launch, s)) return ESP_E_BADCFG;
    } else if (launch_attn_simt(dtype, a, batch, n_split_launch, true, s, false)) {
        return ESP_E_BADCFG;
    }
    return cuda_ok(cudaGetLastError());
}

// ---- the same operator with its scratch inside the library: nothing is allocated by anyone
// File-scope device array; every GPU that loads the library keeps one copy until the process ends.  In host
// code the name below is only a handle for cudaGetSymbolAddress, never a pointer a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[ESP_STATIC_SCRATCH_BYTES];

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
void* g_static_ptr[STATIC_MAX_DEVICES];   // device address of g_static_scratch, per device, 0 until looked up
std::mutex g_static_mutex;

// Device address of the array on the current device (looked up once per device, with that device current).
int static_scratch_ptr(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return ESP_E_CUDA;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return ESP_E_BADCFG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ESP_E_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return ESP_OK;
}
}  // namespace

int esp_tree_attention_static(int32_t dtype, int32_t batch, int32_t n_rows, int32_t L, int32_t cap, int32_t n_q_heads,
                              int32_t n_kv_heads, int32_t head_dim, int32_t dcap, const void* q, const void* kcache,
                              const void* vcache, const uint64_t* anc, const int32_t* depth, void* out,
                              void* cuda_stream) {
    size_t need = 0;
    int rc = esp_tree_attention_scratch_bytes(batch, n_q_heads, head_dim, cap, &need);
    if (rc) return rc;
    if (need > (size_t)ESP_STATIC_SCRATCH_BYTES) return ESP_E_WORKSPACE;   // shape beyond the built-in array
    void* scratch = nullptr;
    rc = static_scratch_ptr(&scratch);
    if (rc) return rc;
    return esp_tree_attention(dtype, batch, n_rows, L, cap, n_q_heads, n_kv_heads, head_dim, dcap, q, kcache, vcache, anc,
                              depth, out, scratch, need, cuda_stream);
}

int esp_tree_attention_status(const void* scratch, void* cuda_stream, int32_t* device_status_out) {
    const void* src = scratch;
    if (!src) {
        void* p = nullptr;
        const int rc = static_scratch_ptr(&p);
        if (rc) return rc;
        src = p;
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    int e = 0;
    if (cudaMemcpyAsync(&e, src, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ESP_E_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ESP_E_CUDA;
    if (device_status_out) *device_status_out = e;
    return e ? ESP_E_DEVICE : ESP_OK;
}

int esp_gemm_scratch_bytes(size_t* bytes_out) {
    if (!bytes_out) return ESP_E_ARG;
    *bytes_out = align_up(tc_gemm_partial_bytes(148, 1, RT), 256) + align_up(sizeof(int) * tc_gemm_counter_ints(), 256) + 256;
    return ESP_OK;
}

int esp_gemm_bf16(int32_t impl, int32_t rows, int32_t n_out, int32_t k_in, const void* x, const void* w, float* y,
                  void* scratch, size_t scratch_bytes, void* cuda_stream) {
    if (!x || !w || !y || !scratch) return ESP_E_ARG;
    if (rows < 1 || rows > RT || n_out < 1 || k_in < 8 || k_in % 8) return ESP_E_ARG;
    size_t need = 0;
    esp_gemm_scratch_bytes(&need);
    if (scratch_bytes < need || reinterpret_cast<uintptr_t>(scratch) % 256) return ESP_E_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    EpiArgs a;
    memset(&a, 0, sizeof(a));
    a.n_out = n_out; a.st = nullptr; a.rows_fixed = rows; a.batch = 1; a.y_f32 = y;
    const void* wv[3] = {w, nullptr, nullptr};
    const int32_t rw[3] = {n_out, 0, 0};
    const int n_tiles = (n_out + TILE_N - 1) / TILE_N;
    if (impl == 1) {
        launch_gemm_simt(1, EPI_STORE_F32, n_tiles, 1, wv, rw, x, k_in, a, s, false);
        return cuda_ok(cudaGetLastError());
    }
    if (impl != 0) return ESP_E_ARG;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return ESP_E_CUDA;
    if (n_sm > 148) n_sm = 148;
    char* sc = reinterpret_cast<char*>(scratch);
    int* counters = reinterpret_cast<int*>(sc + align_up(tc_gemm_partial_bytes(148, 1, RT), 256));
    int* err = reinterpret_cast<int*>(sc + need - 256);
    if (cudaMemsetAsync(counters, 0, sizeof(int) * tc_gemm_counter_ints() , s) != cudaSuccess) return ESP_E_CUDA;
    if (cudaMemsetAsync(err, 0, 256, s) != cudaSuccess) return ESP_E_CUDA;
    TcGemm* plan = nullptr;
    if (tc_gemm_create(&plan, EPI_STORE_F32, false, wv, rw, k_in, x, 1, rows <= 80 ? 80 : RT, 1, sc, tc_gemm_partial_bytes(148, 1, RT), counters, n_sm, err, nullptr, 0, nullptr, s)) return ESP_E_CUDA;
    int rc = tc_gemm_launch(plan, a, s, false);
    int e = 0;
    if (!rc && cudaMemcpyAsync(&e, err, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) rc = ESP_E_CUDA;
    if (!rc && cudaStreamSynchronize(s) != cudaSuccess) rc = ESP_E_CUDA;
    tc_gemm_destroy(plan);
    if (!rc && e) rc = ESP_E_DEVICE;
    return rc;
}

}  // extern "C"
