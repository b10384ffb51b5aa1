/*
 * esp.h -- C ABI of the B200 (sm_100a) implementation of the ESP
 * (Embedding-Space Probing) decode-and-verify step.
 *
 * One handle owns one model replica on one GPU.  Every device buffer
 * (weights, workspace) is allocated by the caller and outlives the handle;
 * the library allocates and frees no device memory.  All work is enqueued on
 * the CUDA stream given to esp_init.  Every call returns ESP_OK (0) or a
 * negative ESP_E_* code; nothing throws, aborts or exits.  Device-side
 * problems (a bounded wait that ran out, an index outside its range) set an
 * error word that esp_read / esp_step / esp_get_stats report as
 * ESP_E_DEVICE.
 *
 * Pointers are marked [host] or [device].  Matrices are row-major
 * [out_features][in_features]; dtype 0 = fp32, 1 = bf16 (weights,
 * activations fed to matrix products and the KV cache share the dtype;
 * accumulation, normalisation, softmax, the residual stream, the mask vector
 * and all selection logic are fp32).
 */
#ifndef ESP_B200_H
#define ESP_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    ESP_OK = 0,
    ESP_E_BADCFG = -1,    /* unsupported or inconsistent configuration */
    ESP_E_WORKSPACE = -2, /* workspace missing, misaligned or too small */
    ESP_E_PROMPT = -3,    /* prompt empty, too long, or token id out of range */
    ESP_E_FULL = -4,      /* the sequence has no room left for another block */
    ESP_E_DEVICE = -5,    /* device error word set (see esp_stats.device_error) */
    ESP_E_CUDA = -6,      /* a CUDA runtime/driver call failed */
    ESP_E_STATE = -7,     /* call out of order (e.g. step before prefill) */
    ESP_E_ARG = -8        /* NULL or out-of-range argument */
};

#define ESP_MAX_ROWS 128  /* rows of one block per sequence: tree nodes + mask probes */
#define ESP_MAX_PROBES 8  /* k */
#define ESP_MAX_KPRIME 32 /* Top-K entries kept per probe, K + pruner refills */
#define ESP_MAX_UNREAD_STEPS 1024 /* decode steps esp_step_async may enqueue before their results are read */
#define ESP_PREFILL_CHUNK 120 /* prompt rows esp_prefill runs per block (the last block adds the k mask rows) */

/* The frozen decoder f_theta (Section 2; LLaMA3 / Qwen3 shapes, Section 4 "Models"). */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t dtype;           /* 0 = fp32 (CUDA-core path), 1 = bf16 (tcgen05 path) */
    int32_t tied_embeddings; /* informational; lm_head may simply alias embed */
    int32_t qk_norm;         /* per-head RMSNorm on q and k before RoPE (Qwen3) */
    float rope_base, rms_eps;
    int32_t max_seq_len;     /* cached positions per sequence (prompt + generated) */
    int32_t max_batch;       /* independent sequences sharing one forward pass */
} esp_model_cfg;

/* Speculation hyper-parameters (Section 3.3-3.5, Section 4 "Block Complexity", "Mask token design"). */
typedef struct {
    int32_t n_probes;      /* k mask tokens per anchored node; 0 = plain greedy decoding */
    int32_t topk;          /* K candidates per probe (Algorithm 1's pool is min(K, B-i)) */
    int32_t max_nodes;     /* B tree nodes including the last accepted token */
    int32_t expand_width;  /* nodes per depth that get children: 1 = Top-1 expansion, 0 = all */
    int32_t n_anchor;      /* nodes (tree order) carrying a probe chain; 0 = every node (paper) */
    int32_t prune_parent;  /* Section 3.5: drop a candidate equal to its parent's token */
    int32_t prune_root;    /* also drop a candidate equal to the last generated token */
    int32_t ema_per_token; /* mask update per emitted token (1) or once per step (0) */
    float lambda;          /* mask update rate, Eq. (mask_update_mean); 0.1 in the paper */
    /* Static tree (Section 4.2, "[K_1, .., K_k]"): when static_widths[0] > 0 the tree is not grown by
     * Algorithm 1; instead the Top-1 node of depth i-1 gets the first static_widths[i-1] candidates of
     * probe i (after the pruner), for as many depths as there are non-zero widths.  topk, max_nodes and
     * expand_width are then ignored (the tree has 1 + sum of widths nodes). */
    int32_t static_widths[ESP_MAX_PROBES];
    /* How esp_prefill sets the k mask vectors (Section 3.1; Section 4 "Different mask embedding designs"):
     * 0 = all k to the mean of the prompt embeddings (Eq. mask_init_mean, the paper's method);
     * 1 = "Last K": mask i gets the embedding of the i-th of the last k prompt tokens;
     * 2 = given by the caller with esp_set_mask before esp_prefill (the "Sample" N(mu, sigma^2 I) and the
     *     mu + n*sigma initialisations: the caller draws or builds the vectors).
     * Every mask vector then follows the same update, Eq. (mask_update_mean). */
    int32_t mask_init;
    /* Matching rule of the verification (Section 4: greedy matching at temperature 0, "sample matching"
     * otherwise).  temperature = 0: a node's next token is the arg-max of its logits.  temperature > 0: it is
     * a draw from softmax(logits / temperature), taken as argmax_v(logits[v] / temperature + g(seed, t, v))
     * with t the absolute position of the drawn token and g standard Gumbel noise from Philox4x32-10 on
     * counter (v, t, 0, 0), key (seed_lo, seed_hi): the stream equals plain autoregressive sampling with the
     * same seed, token by token.  Drafts (probe rows) are always the Top-K of the probe logits. */
    float temperature;
    uint32_t seed_lo, seed_hi;
} esp_spec_cfg;

/* Model weights. [device] matrices; the per-layer members are [host] arrays of
 * n_layers [device] pointers.  q_norm / k_norm may be NULL unless qk_norm. */
typedef struct {
    const void* embed;      /* [vocab][d_model] */
    const void* lm_head;    /* [vocab][d_model]; may equal embed */
    const void* final_norm; /* [d_model] */
    const void* const* wq;  /* [n_q_heads*head_dim][d_model] */
    const void* const* wk;  /* [n_kv_heads*head_dim][d_model] */
    const void* const* wv;  /* [n_kv_heads*head_dim][d_model] */
    const void* const* wo;  /* [d_model][n_q_heads*head_dim] */
    const void* const* w_gate; /* [d_ffn][d_model] */
    const void* const* w_up;   /* [d_ffn][d_model] */
    const void* const* w_down; /* [d_model][d_ffn] */
    const void* const* norm_attn; /* [d_model] */
    const void* const* norm_ffn;  /* [d_model] */
    const void* const* q_norm;    /* [head_dim] */
    const void* const* k_norm;    /* [head_dim] */
} esp_weights;

typedef struct {
    int64_t steps;          /* decode-and-verify calls so far (all sequences) */
    int64_t emitted;        /* tokens emitted by those calls (bonus tokens included) */
    int64_t accept_hist[ESP_MAX_PROBES + 1]; /* [a] = steps that accepted a draft tokens */
    int32_t device_error;   /* 0, or the first device-side error code recorded */
    int32_t kernels_per_step; /* kernel launches one esp_step enqueues */
    int64_t rows_hist[4];   /* decode steps by block size (tree nodes + mask rows): <= 16, <= 32, <= 64, more rows */
} esp_stats;

typedef struct esp_handle esp_handle;

/* Bytes of [device] workspace esp_init needs (KV cache for max_batch sequences of
 * max_seq_len + ESP_MAX_ROWS positions, activations, split-K and attention
 * partials, per-sequence state and -- for bf16 models -- a copy of
 * every layer matrix and of the LM head repacked into the 16 KB blocks the GEMM
 * main loop streams, i.e. about the size of the model again).
 * ESP_E_BADCFG if the configuration is unsupported. */
int esp_workspace_bytes(const esp_model_cfg* model, const esp_spec_cfg* spec, size_t* bytes_out);

/* Create a handle.  `workspace` [device] must be 256-byte aligned and at least
 * esp_workspace_bytes large; it is zeroed here.  `cuda_stream` is a cudaStream_t
 * (NULL = default stream).  Builds the rotary table, the TMA descriptors and the repacked
 * weight copy (the caller's matrices are still read by the CUDA-core path and the embedding
 * gather, so they must stay alive).
 * The frozen model is the f_theta of Section 2. */
int esp_init(const esp_model_cfg* model, const esp_spec_cfg* spec, const esp_weights* weights, void* workspace,
             size_t workspace_bytes, void* cuda_stream, esp_handle** handle_out);

/* Prefill of sequence `seq` (Figure 1 middle; Section 3.3: generation only).
 * prompt [host] n_prompt ids.  Sets the mask vector to the mean prompt
 * embedding (Eq. mask_init_mean), runs the prompt in causal blocks with the
 * k mask rows appended to the last one, caches the prompt rows, emits the
 * first token (written to *first_token_out [host], may be NULL), applies the
 * mask update and builds the first draft tree (Algorithm 1).  Synchronises. */
int esp_prefill(esp_handle* h, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t* first_token_out);

/* One decode-and-verify step for every prefilled sequence (Figure 1 right):
 * forward over [last accepted token, draft-tree nodes, mask probes] under the
 * tree mask, argmax (or the sampled token, see esp_spec_cfg.temperature) / Top-K' +
 * log-sum-exp, lossless verification (Section 2),
 * KV compaction of the accepted path, mask update (Eq. mask_update_mean) and
 * the next tree (Algorithm 1 + pruner).  esp_step = esp_step_async + esp_read.
 * tokens_out [host] [max_batch][ESP_MAX_PROBES+1], n_out [host] [max_batch].
 * esp_step_async only enqueues the step; nothing of it depends on the host, so several may be enqueued back to
 * back.  Every step leaves its result in a record of its own and esp_read returns the OLDEST unread step (0 tokens
 * for a sequence that took no part in it; with nothing unread it reports 0 tokens for every sequence and the
 * device status).  At most ESP_MAX_UNREAD_STEPS steps may be unread: one more esp_step_async returns ESP_E_STATE.
 * While steps are unread the host knows each cache length only as an upper bound (k + 1 positions per unread
 * step): ESP_E_FULL may then come that many positions early, and the attention launches are sized for the bound
 * (splits without work return at once); results do not depend on it. */
int esp_step(esp_handle* h, int32_t* tokens_out, int32_t* n_out);
int esp_step_async(esp_handle* h);
int esp_read(esp_handle* h, int32_t* tokens_out, int32_t* n_out);

/* Mask vectors of sequence `seq` given by the caller (mask_init = 2): mask [host] [n_probes][d_model] fp32.
 * Call before esp_prefill of that sequence (a later call replaces the current vectors).  Synchronises. */
int esp_set_mask(esp_handle* h, int32_t seq, const float* mask);

/* Test hook: replace the draft tree of sequence `seq` for the next step.
 * tokens/parents [host] n nodes in breadth-first order (parents[0] = -1,
 * parents[i] < i); node 0 must carry the current root token.  Has no
 * counterpart in the paper; it exists to drive acceptance lengths that
 * random-init models never produce.  The tree with its probe rows must fit the
 * block the handle was configured for (the spec's rows), else ESP_E_ARG. */
int esp_set_tree(esp_handle* h, int32_t seq, const int32_t* tokens, const int32_t* parents, int32_t n);

/* Debug/parity access to device state of sequence `seq`, copied to [host] buffers (any may be NULL):
 *   row_token/row_parent/row_depth [ESP_MAX_ROWS], n_nodes, n_rows, L of the block the NEXT step will run;
 *   topk_ids/topk_vals [ESP_MAX_ROWS][ESP_MAX_KPRIME], lse [ESP_MAX_ROWS] from the LAST forward;
 *   mask_vec [max(n_probes, 1)][d_model].  Synchronises. */
int esp_debug_state(esp_handle* h, int32_t seq, int32_t* row_token, int32_t* row_parent, int32_t* row_depth,
                    int32_t* n_nodes, int32_t* n_rows, int32_t* L, int32_t* topk_ids, float* topk_vals, float* lse,
                    float* mask_vec);

/* Debug/parity: when `logits` [device] fp32 [max_batch*ESP_MAX_ROWS][vocab] is non-NULL, every later forward also
 * stores the full logits there (the product path never materialises them).  `hidden` [device] fp32
 * [max_batch*ESP_MAX_ROWS][d_model], if non-NULL, receives the residual stream after the last layer. */
int esp_debug_capture(esp_handle* h, float* logits, float* hidden);

/* Selects the matrix-product implementation for bf16 models: 0 = tcgen05 tensor-core kernels (default),
 * 1 = CUDA-core reference kernels (same epilogues; for A/B checks on the GPU).  fp32 models always use 1. */
int esp_debug_set_gemm(esp_handle* h, int32_t impl);

/* Selects how the decoder layers of a step are launched for bf16 models with head_dim 128, max_batch 1 and blocks
 * of at most 80 rows: 1 = one kernel per operation, chained by programmatic dependent launch (default; what
 * batches, prefill blocks and larger blocks always use), 0 = all layers in one persistent cooperative kernel (the
 * weight ring keeps running across the operations of a layer, grid-wide barriers with bounded waits between
 * them).  Both run the same arithmetic in the same order and give the same bits.  Mode 0 is kept for A/B
 * checks and tracing (esp_debug_layer_timeline): on a B200 its step is slower, because every phase between two
 * GEMMs pays two grid barriers plus its own chain of L2 round trips with 14 warps per SM, where the chained
 * kernels overlap neighbouring launches.  No counterpart in the paper.
 * ESP_E_BADCFG if mode 0 is not available for the handle's configuration. */
int esp_debug_set_layer_kernel(esp_handle* h, int32_t mode);

/* Measurement hook (no counterpart in the paper): one esp_step with a CUDA event recorded on the handle's
 * stream after every kernel group; ms_by_kind [host] [8] receives the device time per group in this order:
 * 0 row assembly, RMSNorm and the kernels that sum GEMM partials (residual add + norm, RoPE + cache write,
 * SiLU*up), 1 QKV GEMM, 2 tree attention, 3 O GEMM, 4 gate/up GEMM, 5 down GEMM, 6 LM-head GEMM with fused
 * selection, 7 Top-K' merge + tree kernel.  The kernels run back to back without overlap in this mode, so the
 * groups add up to more than an unprofiled step.  When all layers run in one kernel (esp_debug_set_layer_kernel
 * mode 0) that kernel's share is split by the global-timer stamps its first CTA takes after every grid barrier.
 * tokens_out / n_out as esp_step. */
int esp_step_profiled(esp_handle* h, float* ms_by_kind, int32_t* tokens_out, int32_t* n_out);

/* Tracing (no counterpart in the paper): the time stamps of the last esp_step_profiled whose layers ran in one
 * kernel.  stamps_ns [host] [capacity] receives the GPU's global timer (ns) as read by that kernel's first CTA:
 * eight words per grid barrier -- [0] its arrival at the barrier, [1] its exit, and inside the phase that
 * follows, when that is a GEMM, [2] the activation tiles of the ring's first items requested, [3] the first
 * item consumed by the tensor cores, [4] the last one issued, [5] the last accumulator stored ([6], [7] and the
 * words of other phases are unused and hold stale values) -- ten barriers per layer, one behind each phase in
 * the order: attention norm, QKV GEMM, q/k/v finish, attention over the cache, attention tail + merge, O GEMM,
 * FFN norm, gate/up GEMM, SiLU*up, down GEMM.  *n_out [host] = words per step (n_layers * 80).  Synchronises.
 * ESP_E_BADCFG if the handle has no such kernel. */
int esp_debug_layer_timeline(esp_handle* h, uint64_t* stamps_ns, int32_t capacity, int32_t* n_out);

int esp_get_stats(esp_handle* h, esp_stats* out);

/* Self-test of the bounded waits the tensor-core kernels use (no counterpart in the paper): launches one
 * small kernel that waits on a barrier nothing ever signals; the wait must give up after its time limit
 * (50 ms), record the wait-timeout code and return normally.  *device_status_out [host] receives the code the
 * kernel recorded (1 = wait timed out, as expected).  The CUDA context stays usable.  `scratch` [device] >= 256
 * bytes. */
int esp_debug_wait_selftest(void* scratch, void* cuda_stream, int32_t* device_status_out);

/* The sampling noise of sample matching, for checking it bit by bit: noise_out [device] [n_tokens] fp32 receives
 * g(seed, position, v) for v = 0..n_tokens-1 (see esp_spec_cfg.temperature).  Asynchronous on cuda_stream. */
int esp_debug_gumbel(uint32_t seed_lo, uint32_t seed_hi, uint32_t position, int32_t n_tokens, float* noise_out,
                     void* cuda_stream);

/* Releases host-side bookkeeping only. */
void esp_free(esp_handle* h);

/* ---- stand-alone operators (the same kernels the step uses), for operator-level parity and timing ---- */

/* Tree-masked GQA attention (Figure 1 right / Figure 3: every row sees the cache and its own
 * root-to-self path).  All pointers [device].
 *   q        [batch][ESP_MAX_ROWS][n_q_heads][head_dim]
 *   kcache,vcache [batch][n_kv_heads][cap][head_dim]; positions 0..L-1 are the cache, the block
 *            row i's key/value sit at position L+i (the caller writes them there)
 *   anc      [batch][ESP_MAX_ROWS][2] uint64 ancestor-or-self bitmask over block rows
 *   depth    [batch][ESP_MAX_ROWS] int32, position of the row minus L
 *   out      [batch][ESP_MAX_ROWS][n_q_heads][head_dim]
 *   scratch  esp_tree_attention_scratch_bytes bytes
 * dtype as in esp_model_cfg; n_rows <= ESP_MAX_ROWS rows are real; L + ESP_MAX_ROWS <= cap.
 * The tensor-core path reads the cache in chunks of 128 positions that may reach up to position
 * L + ESP_MAX_ROWS - 1: positions beyond a row's visible keys get weight zero, but their VALUES still enter a
 * product with that zero, so kcache / vcache must hold finite numbers (zeros will do) up to there.
 * The call is asynchronous on cuda_stream.  A device-side problem (a bounded wait that ran out, an ancestor
 * mask that names a row the block does not have) is recorded in the first word of the scratch, which the call
 * clears when it starts; esp_tree_attention_status reads it back.
 * dcap (a multiple of 16, >= the largest depth) sets where each row's key list switches from the
 * tensor-core chunks to the position-by-position tail: keys at positions below
 * floor((L + depth - dcap) / 16) * 16 go through the chunked path, the rest through the tail. */
int esp_tree_attention_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim, int32_t cap,
                                     size_t* bytes_out);
int esp_tree_attention(int32_t dtype, int32_t batch, int32_t n_rows, int32_t L, int32_t cap, int32_t n_q_heads,
                       int32_t n_kv_heads, int32_t head_dim, int32_t dcap, const void* q, const void* kcache,
                       const void* vcache, const uint64_t* anc, const int32_t* depth, void* out, void* scratch,
                       size_t scratch_bytes, void* cuda_stream);
/* Device status of the last esp_tree_attention that used `scratch` [device] (NULL: of the last
 * esp_tree_attention_static on the current device): waits for cuda_stream, copies the status word to
 * *device_status_out [host] (may be NULL) and returns ESP_OK if it is 0, ESP_E_DEVICE otherwise. */
int esp_tree_attention_status(const void* scratch, void* cuda_stream, int32_t* device_status_out);

/* esp_tree_attention for callers that cannot hand over scratch memory (the paper has no counterpart; this is
 * a packaging variant of the operator above).  Meant for hosts that may not allocate device memory at the
 * point of the call: a serving loop whose device memory was budgeted up front and handed to other owners, a
 * plug-in running inside somebody else's process that must not touch the allocator, code between the
 * begin and end of work where an allocation would stall the whole device.  The split partials live in a
 * fixed array inside the library instead (ESP_STATIC_SCRATCH_BYTES, 32 MiB, held on every GPU that loads
 * the library until the process exits).  Same arguments, layouts and results as esp_tree_attention, minus
 * the scratch pair.  Returns ESP_E_WORKSPACE when the shape needs more than the array holds
 * (esp_tree_attention_scratch_bytes(batch, n_q_heads, head_dim, cap) > ESP_STATIC_SCRATCH_BYTES; e.g. 32
 * query heads of 128 with cap <= 3584 at batch 1 fit).  It allocates and frees nothing, on the host or the
 * device: the descriptors of the call live in its own stack frame.  The first call on each device looks up the
 * array's device address (a one-time query, no allocation); make that first call outside any stream capture.
 * All calls share the one array and it keeps the previous call's contents: the status word at its start is
 * cleared by every call (esp_tree_attention_status(NULL, ...) reads it), everything else is overwritten before
 * it is read.  Two calls whose kernels can overlap on the GPU (different streams, no dependency between them)
 * would write the same partials and race: keep them ordered. */
#define ESP_STATIC_SCRATCH_BYTES (32u << 20)
int esp_tree_attention_static(int32_t dtype, int32_t batch, int32_t n_rows, int32_t L, int32_t cap, int32_t n_q_heads,
                              int32_t n_kv_heads, int32_t head_dim, int32_t dcap, const void* q, const void* kcache,
                              const void* vcache, const uint64_t* anc, const int32_t* depth, void* out,
                              void* cuda_stream);

/* y[rows][n_out] (fp32) = x[rows][k_in] (bf16) * w[n_out][k_in]^T (bf16) on the tcgen05 path
 * (impl 0) or the CUDA-core path (impl 1).  All pointers [device]; x must hold ESP_MAX_ROWS
 * rows (rows beyond `rows` are ignored); scratch as esp_gemm_scratch_bytes says. */
int esp_gemm_scratch_bytes(size_t* bytes_out);
int esp_gemm_bf16(int32_t impl, int32_t rows, int32_t n_out, int32_t k_in, const void* x, const void* w, float* y,
                  void* scratch, size_t scratch_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ESP_B200_H */
