/*
 * CPU oracle, part 1: a plain fp32 decoder-only transformer evaluated on one
 * "block" of rows against a key/value cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct
 * reference that the CUDA path is compared against.  It shares no code,
 * header, table or constant with the CUDA library and must never be called
 * from the product path.
 *
 * What it computes.  The paper's method runs the frozen language model
 * f_theta once per step over a block made of the last accepted token, the
 * draft-tree nodes and the mask-token probes (Section 3.3, "block
 * complexity"), where every row may look at the cached context plus its own
 * root-to-self path (Figure 1 right, Figure 3, Appendix E).  The paper does
 * not define the model's numerics; the model here is the standard
 * LLaMA3/Qwen3 pre-norm decoder the paper names in Section 4 (RMSNorm, GQA
 * attention with rotary position embedding, SwiGLU feed-forward, optional
 * per-head RMSNorm on queries and keys).
 *
 * How it computes.  Everything is fp32.  Every output element of every
 * matrix product is one running sum over k = 0..K-1 in increasing k.  The
 * attention of a row is one pass over that row's own key list (cache
 * positions 0..L-1 in order, then the visible block rows in row order):
 * scores, their maximum, then sum of exponentials and the weighted value
 * sum, each accumulated in list order.  A row's result therefore depends
 * only on that row's inputs and its key list -- never on which other rows
 * share the block -- which is what makes tree verification reproduce plain
 * autoregressive decoding exactly (Section 2, "lossless").
 *
 * Weights are either fp32 or bf16 bit patterns (widened exactly).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t wdtype;  /* 0 = fp32, 1 = bf16 bit patterns */
    int32_t qk_norm; /* 1 = per-head RMSNorm on q and k before RoPE (Qwen3) */
    float rope_base, rms_eps;
} orc_cfg;

typedef struct {
    const void* embed;      /* [V][d] */
    const void* lm_head;    /* [V][d] (same pointer as embed when tied) */
    const void* final_norm; /* [d] */
    const void* const* wq;  /* per layer [Hq*h][d] */
    const void* const* wk;  /* per layer [Hkv*h][d] */
    const void* const* wv;  /* per layer [Hkv*h][d] */
    const void* const* wo;  /* per layer [d][Hq*h] */
    const void* const* w_gate; /* per layer [F][d] */
    const void* const* w_up;   /* per layer [F][d] */
    const void* const* w_down; /* per layer [d][F] */
    const void* const* norm_attn; /* per layer [d] */
    const void* const* norm_ffn;  /* per layer [d] */
    const void* const* q_norm;    /* per layer [h] or NULL */
    const void* const* k_norm;    /* per layer [h] or NULL */
} orc_weights;

static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static inline float wload(const void* w, int wdtype, size_t i) {
    return wdtype ? bf16_to_f32(((const uint16_t*)w)[i]) : ((const float*)w)[i];
}

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Row i of the embedding table, widened to fp32: e = E[token]. (Section 3.1) */
void orc_embed_row(const orc_cfg* c, const void* embed, int32_t token, float* out) {
    for (int j = 0; j < c->d_model; ++j) out[j] = wload(embed, c->wdtype, (size_t)token * c->d_model + j);
}

/* Y[M][N] = X[M][K] * W[N][K]^T.  Each Y[m][n] is the fp32 running sum of
 * X[m][k]*W[n][k] for k = 0, 1, ..., K-1.  X is passed transposed (xT[K][M])
 * so that the loop over rows m is the contiguous one; that changes nothing
 * about any single sum. */
#define ORC_NB 4
static void linear_T(const float* xT, int M, int K, const void* W, int wdtype, int N, float* Y) {
#pragma omp parallel
    {
        float* acc = (float*)malloc(sizeof(float) * (size_t)M * ORC_NB);
#pragma omp for schedule(static)
        for (int nb = 0; nb < (N + ORC_NB - 1) / ORC_NB; ++nb) {
            int n0 = nb * ORC_NB;
            int nn = N - n0 < ORC_NB ? N - n0 : ORC_NB;
            for (int i = 0; i < M * ORC_NB; ++i) acc[i] = 0.0f;
            for (int k = 0; k < K; ++k) {
                const float* xk = xT + (size_t)k * M;
                for (int j = 0; j < nn; ++j) {
                    float w = wload(W, wdtype, (size_t)(n0 + j) * K + k);
                    float* a = acc + (size_t)j * M;
                    for (int m = 0; m < M; ++m) a[m] = a[m] + xk[m] * w;
                }
            }
            for (int j = 0; j < nn; ++j)
                for (int m = 0; m < M; ++m) Y[(size_t)m * N + n0 + j] = acc[(size_t)j * M + m];
        }
        free(acc);
    }
}

/* Stand-alone entry to the matrix product above, for operator-level checks: y[M][N] = x[M][K] * W[N][K]^T. */
int orc_linear(int32_t M, int32_t K, int32_t N, const float* x, const void* W, int32_t wdtype, float* y) {
    float* xT = (float*)malloc(sizeof(float) * (size_t)M * K);
    if (!xT) return -1;
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) xT[(size_t)k * M + m] = x[(size_t)m * K + k];
    linear_T(xT, M, K, W, wdtype, N, y);
    free(xT);
    return 0;
}

static void transpose(const float* x, int M, int K, float* xT) {
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) xT[(size_t)k * M + m] = x[(size_t)m * K + k];
}

/* y = x * rsqrt(mean(x^2) + eps) * g over the last dimension n. */
static void rmsnorm(const float* x, int n, const void* g, int wdtype, float eps, float* y) {
    float ss = 0.0f;
    for (int i = 0; i < n; ++i) ss = ss + x[i] * x[i];
    float r = 1.0f / sqrtf(ss / (float)n + eps);
    for (int i = 0; i < n; ++i) y[i] = x[i] * r * (g ? wload(g, wdtype, i) : 1.0f);
}

/* Rotary embedding, "rotate-half" pairing (i, i + h/2), angle pos * base^(-2i/h). */
static void rope(float* x, int h, int32_t pos, float base) {
    int half = h / 2;
    for (int i = 0; i < half; ++i) {
        double inv = pow((double)base, -2.0 * (double)i / (double)h);
        double ang = (double)pos * inv;
        float cs = (float)cos(ang), sn = (float)sin(ang);
        float a = x[i], b = x[i + half];
        x[i] = a * cs - b * sn;
        x[i + half] = b * cs + a * sn;
    }
}

int orc_tree_attention(int32_t M, int32_t L, int32_t Hq, int32_t Hkv, int32_t h, const float* q,
                       const float* kc, const float* vc, const float* kb, const float* vb,
                       const uint8_t* vis, float* out);

/*
 * One forward pass over a block of M rows.
 *
 *  kcache, vcache : [n_layers][cap][Hkv][h] fp32; positions 0..L-1 valid. Read only.
 *  x              : [M][d] input vectors (token embeddings or the mask vector).
 *  pos            : [M] position id of each row (Figure 3 / Appendix E: a
 *                   node at depth t below the last accepted token sits at
 *                   L + t; mask rows take the positions that follow).
 *  vis            : [M][M] bytes; vis[r][i] != 0 iff row r may attend to
 *                   block row i (must include i == r).  Cache positions
 *                   0..L-1 are visible to every row.
 *  kblk, vblk     : [n_layers][M][Hkv][h] out; keys/values of the block rows,
 *                   for the caller to append to the cache.
 *  want           : [M] bytes; logits are produced only for rows with want != 0.
 *  logits         : [M][V] out (rows with want == 0 untouched); may be NULL.
 *  hidden_out     : [M][d] out, final-norm output; may be NULL.
 * Returns 0, or -1 on allocation failure / bad arguments.
 */
int orc_block_forward(const orc_cfg* c, const orc_weights* w, const float* kcache, const float* vcache,
                      int64_t cap, int32_t L, int32_t M, const float* x, const int32_t* pos,
                      const uint8_t* vis, float* kblk, float* vblk, const uint8_t* want, float* logits,
                      float* hidden_out) {
    const int d = c->d_model, Hq = c->n_q_heads, Hkv = c->n_kv_heads, h = c->head_dim, F = c->d_ffn;
    const int dq = Hq * h, dkv = Hkv * h;
    if (M <= 0 || L < 0 || L > cap || Hq % Hkv) return -1;
    size_t big = (size_t)(F > dq ? F : dq);
    if ((size_t)d > big) big = d;
    float* hres = (float*)malloc(sizeof(float) * (size_t)M * d);      /* residual stream */
    float* xn = (float*)malloc(sizeof(float) * (size_t)M * big);      /* normed / scratch */
    float* xT = (float*)malloc(sizeof(float) * (size_t)M * big);
    float* q = (float*)malloc(sizeof(float) * (size_t)M * dq);
    float* att = (float*)malloc(sizeof(float) * (size_t)M * dq);
    float* y = (float*)malloc(sizeof(float) * (size_t)M * d);
    float* g = (float*)malloc(sizeof(float) * (size_t)M * F);
    float* u = (float*)malloc(sizeof(float) * (size_t)M * F);
    if (!hres || !xn || !xT || !q || !att || !y || !g || !u) return -1;
    memcpy(hres, x, sizeof(float) * (size_t)M * d);

    for (int l = 0; l < c->n_layers; ++l) {
        float* kb = kblk + (size_t)l * M * dkv;
        float* vb = vblk + (size_t)l * M * dkv;
        const float* kc = kcache + (size_t)l * cap * dkv;
        const float* vc = vcache + (size_t)l * cap * dkv;
        /* attention sub-block */
        for (int m = 0; m < M; ++m)
            rmsnorm(hres + (size_t)m * d, d, w->norm_attn[l], c->wdtype, c->rms_eps, xn + (size_t)m * d);
        transpose(xn, M, d, xT);
        linear_T(xT, M, d, w->wq[l], c->wdtype, dq, q);
        linear_T(xT, M, d, w->wk[l], c->wdtype, dkv, kb);
        linear_T(xT, M, d, w->wv[l], c->wdtype, dkv, vb);
        for (int m = 0; m < M; ++m) {
            for (int hh = 0; hh < Hq; ++hh) {
                float* qh = q + (size_t)m * dq + (size_t)hh * h;
                if (c->qk_norm) rmsnorm(qh, h, w->q_norm[l], c->wdtype, c->rms_eps, qh);
                rope(qh, h, pos[m], c->rope_base);
            }
            for (int hh = 0; hh < Hkv; ++hh) {
                float* kh = kb + (size_t)m * dkv + (size_t)hh * h;
                if (c->qk_norm) rmsnorm(kh, h, w->k_norm[l], c->wdtype, c->rms_eps, kh);
                rope(kh, h, pos[m], c->rope_base);
            }
        }
        if (orc_tree_attention(M, L, Hq, Hkv, h, q, kc, vc, kb, vb, vis, att)) return -1;
        transpose(att, M, dq, xT);
        linear_T(xT, M, dq, w->wo[l], c->wdtype, d, y);
        for (size_t i = 0; i < (size_t)M * d; ++i) hres[i] = hres[i] + y[i];
        /* feed-forward sub-block: down( silu(gate(x)) * up(x) ) */
        for (int m = 0; m < M; ++m)
            rmsnorm(hres + (size_t)m * d, d, w->norm_ffn[l], c->wdtype, c->rms_eps, xn + (size_t)m * d);
        transpose(xn, M, d, xT);
        linear_T(xT, M, d, w->w_gate[l], c->wdtype, F, g);
        linear_T(xT, M, d, w->w_up[l], c->wdtype, F, u);
        for (size_t i = 0; i < (size_t)M * F; ++i) {
            float a = g[i];
            g[i] = (a / (1.0f + expf(-a))) * u[i];
        }
        transpose(g, M, F, xT);
        linear_T(xT, M, F, w->w_down[l], c->wdtype, d, y);
        for (size_t i = 0; i < (size_t)M * d; ++i) hres[i] = hres[i] + y[i];
    }
    /* final norm + LM head (logits = h * W, Section 3.2) on the wanted rows only */
    int nw = 0;
    for (int m = 0; m < M; ++m) {
        rmsnorm(hres + (size_t)m * d, d, w->final_norm, c->wdtype, c->rms_eps, xn + (size_t)m * d);
        if (want && want[m]) ++nw;
    }
    if (hidden_out) memcpy(hidden_out, xn, sizeof(float) * (size_t)M * d);
    if (logits && nw > 0) {
        float* xs = (float*)malloc(sizeof(float) * (size_t)nw * d);
        float* ys = (float*)malloc(sizeof(float) * (size_t)nw * c->vocab);
        float* xsT = (float*)malloc(sizeof(float) * (size_t)nw * d);
        if (!xs || !ys || !xsT) return -1;
        int j = 0;
        for (int m = 0; m < M; ++m)
            if (want[m]) memcpy(xs + (size_t)(j++) * d, xn + (size_t)m * d, sizeof(float) * d);
        transpose(xs, nw, d, xsT);
        linear_T(xsT, nw, d, w->lm_head, c->wdtype, c->vocab, ys);
        j = 0;
        for (int m = 0; m < M; ++m)
            if (want[m]) memcpy(logits + (size_t)m * c->vocab, ys + (size_t)(j++) * c->vocab, sizeof(float) * c->vocab);
        free(xs);
        free(ys);
        free(xsT);
    }
    free(hres); free(xn); free(xT); free(q); free(att); free(y); free(g); free(u);
    return 0;
}

/*
 * Tree-masked attention (Figure 1 right, Figure 3): row m, head hh attends to
 * cache positions 0..L-1 and to the block rows i with vis[m][i] != 0, softmax
 * scale 1/sqrt(h).  q [M][Hq][h], cache k/v [L][Hkv][h], block k/v
 * [M][Hkv][h], vis [M][M]; out [M][Hq][h].  One pass over the row's key list
 * in list order: scores and their maximum, then the sum of exponentials and
 * the weighted value sum.  Also the stand-alone operator workload.
 */
int orc_tree_attention(int32_t M, int32_t L, int32_t Hq, int32_t Hkv, int32_t h, const float* q,
                       const float* kc, const float* vc, const float* kb, const float* vb,
                       const uint8_t* vis, float* out) {
    if (Hq % Hkv) return -1;
    const int group = Hq / Hkv, dq = Hq * h, dkv = Hkv * h;
    const float scale = 1.0f / sqrtf((float)h);
#pragma omp parallel
    {
        float* s = (float*)malloc(sizeof(float) * (size_t)(L + M));
        const float** kp = (const float**)malloc(sizeof(float*) * (size_t)(L + M));
        const float** vp = (const float**)malloc(sizeof(float*) * (size_t)(L + M));
#pragma omp for collapse(2) schedule(static)
        for (int m = 0; m < M; ++m) {
            for (int hh = 0; hh < Hq; ++hh) {
                const int kvh = hh / group;
                const float* qh = q + (size_t)m * dq + (size_t)hh * h;
                int n = 0;
                for (int p = 0; p < L; ++p) {
                    kp[n] = kc + (size_t)p * dkv + (size_t)kvh * h;
                    vp[n] = vc + (size_t)p * dkv + (size_t)kvh * h;
                    ++n;
                }
                for (int i = 0; i < M; ++i)
                    if (vis[(size_t)m * M + i]) {
                        kp[n] = kb + (size_t)i * dkv + (size_t)kvh * h;
                        vp[n] = vb + (size_t)i * dkv + (size_t)kvh * h;
                        ++n;
                    }
                float mx = -INFINITY;
                for (int j = 0; j < n; ++j) {
                    float a = 0.0f;
                    for (int t = 0; t < h; ++t) a = a + qh[t] * kp[j][t];
                    s[j] = a * scale;
                    if (s[j] > mx) mx = s[j];
                }
                float den = 0.0f;
                float* o = out + (size_t)m * dq + (size_t)hh * h;
                for (int t = 0; t < h; ++t) o[t] = 0.0f;
                for (int j = 0; j < n; ++j) {
                    float p = expf(s[j] - mx);
                    den = den + p;
                    for (int t = 0; t < h; ++t) o[t] = o[t] + p * vp[j][t];
                }
                for (int t = 0; t < h; ++t) o[t] = o[t] / den;
            }
        }
        free(s);
        free((void*)kp);
        free((void*)vp);
    }
    return 0;
}
