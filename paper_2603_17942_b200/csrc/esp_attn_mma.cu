// Tree attention for bf16, head_dim 128.
//
// A row at position P attends to cache positions 0..T0-1 through the "bulk"
// CTAs (T0 as in tail_start(): the 16-aligned position below which keys are
// always cache resident): the KV cache of one KV head is streamed once per
// split through shared memory (16-byte cp.async, XOR swizzle) and shared by
// all query heads of the group and all block rows: a CTA holds 64 (row, head)
// pairs, a warp 16 of them, Q.K^T and P.V run on mma.sync m16n8k16 with fp32
// online softmax in registers.  The remaining positions T0..P -- the end of
// the cache plus the row's in-flight tree ancestors, found through its
// ancestor bitmask -- are summed by "tail" CTAs of the same launch, key by
// key in position order.  Every CTA stores (max, sum, weighted values)
// partials; a second small kernel (one warp per (row, head)) merges them in
// split order, tail last, and writes the output.
//
// Everything that decides a row's arithmetic -- the 64-key chunk grid, the
// split grid, the per-position mask -- is a function of absolute positions
// only, so the same token gets the same bits whether it is verified inside a
// tree block or decoded alone.
#include "esp_launch.h"

namespace esp {

namespace {

constexpr int HD = 128;
constexpr int CHUNK = 64;
constexpr int PAIRS = 64;  // (row, head) pairs per CTA
constexpr int KV_TILE_BYTES = CHUNK * HD * 2;
constexpr int TAIL_CTAS = 8;   // tail CTAs per group of 64 pairs: 8 pairs each, 2 per warp

__device__ __forceinline__ int tail_start_mma(int P, int dcap) {
    int t = P - dcap;
    return t <= 0 ? 0 : (t / 16) * 16;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte unit `u` (0..15) of key row `key` (0..63) inside a swizzled KV tile
__device__ __forceinline__ uint32_t kv_off(int key, int u) { return (uint32_t)(key * 256 + ((u ^ (key & 7)) << 4)); }

// ---- bulk: one split of the cache for the 64 (row, head) pairs of a group
__device__ __forceinline__ void attn_bulk_chunks(const AttnArgs& a, unsigned char* smem, int seq, int kvh, int row0, int split,
                                                 int group, int n_rows, int L, int T0max, const __nv_bfloat16* kbase,
                                                 const __nv_bfloat16* vbase) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // per-thread pairs: A = warp*16 + lane/4, B = A + 8
    int pr[2], ph[2], pT0[2];
    bool pv[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int pidx = warp * 16 + (lane >> 2) + i * 8;
        pr[i] = row0 + pidx / group;
        ph[i] = kvh * group + pidx % group;
        pv[i] = pr[i] < n_rows && pr[i] < RT;
        int depth = 0;
        if (pv[i]) depth = a.st ? a.st[seq].row_depth[pr[i]] : a.depth[seq * RT + pr[i]];
        pT0[i] = pv[i] ? tail_start_mma(L + depth, a.dcap) : 0;
    }
    const int beg = split * a.split_len;
    const int end = min(beg + a.split_len, T0max);
    const uint32_t s_base = smem_u32(smem);

    auto load_chunk = [&](int c, int stage) {
        const int base = beg + c * CHUNK;
        const uint32_t sk = s_base + stage * 2 * KV_TILE_BYTES, sv = sk + KV_TILE_BYTES;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int idx = threadIdx.x + i * 128;  // 0..1023
            const int key = idx >> 4, u = idx & 15;
            const int pos = base + key;
            const int nbytes = pos < end ? 16 : 0;
            const size_t goff = (size_t)(pos < end ? pos : beg) * HD + u * 8;
            cp_async16(sk + kv_off(key, u), kbase + goff, nbytes);
            cp_async16(sv + kv_off(key, u), vbase + goff, nbytes);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // The cache below T0 was written by earlier steps: request the first chunk before waiting for the kernel
    // that produces this block's queries.
    const int n_chunks = (end - beg + CHUNK - 1) / CHUNK;
    load_chunk(0, 0);
    pdl_wait();
    // Q fragments (A operand), straight from global memory
    uint32_t qf[HD / 16][4];
    {
        const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q);
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int col = ks * 16 + (lane & 3) * 2;
                uint32_t lo = 0, hi = 0;
                if (pv[i]) {
                    const __nv_bfloat16* qp = q + ((size_t)(seq * RT + pr[i]) * a.Hq + ph[i]) * HD + col;
                    lo = *reinterpret_cast<const uint32_t*>(qp);
                    hi = *reinterpret_cast<const uint32_t*>(qp + 8);
                }
                qf[ks][i] = lo;       // a0 (row A) / a1 (row B)
                qf[ks][2 + i] = hi;   // a2 / a3
            }
        }
    }

    float o[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    for (int c = 0; c < n_chunks; ++c) {
        const int stage = c & 1;
        if (c + 1 < n_chunks) {
            load_chunk(c + 1, stage ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const uint32_t sk = s_base + stage * 2 * KV_TILE_BYTES, sv = sk + KV_TILE_BYTES;
        // S = Q K^T  (16 pairs x 64 keys per warp)
        float s[CHUNK / 8][4];
#pragma unroll
        for (int nt = 0; nt < CHUNK / 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int nt = 0; nt < CHUNK / 8; ++nt) {
#pragma unroll
            for (int kp = 0; kp < HD / 32; ++kp) {
                uint32_t b0, b1, b2, b3;
                const int key = nt * 8 + (lane & 7);
                const int u = kp * 4 + (lane >> 3);
                ldsm_x4(sk + kv_off(key, u), b0, b1, b2, b3);
                mma_bf16(s[nt], qf[kp * 2], b0, b1);
                mma_bf16(s[nt], qf[kp * 2 + 1], b2, b3);
            }
        }
        // mask + online softmax (log2 domain)
        const int cbase = beg + c * CHUNK;
        float cmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < CHUNK / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int i = e >> 1;
                const int pos = cbase + nt * 8 + (lane & 3) * 2 + (e & 1);
                const float v = pos < pT0[i] ? s[nt][e] * a.scale_log2 : -INFINITY;
                s[nt][e] = v;
                cmax[i] = fmaxf(cmax[i], v);
            }
        }
        float scale_old[2], m_use[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            cmax[i] = fmaxf(cmax[i], __shfl_xor_sync(0xffffffffu, cmax[i], 1));
            cmax[i] = fmaxf(cmax[i], __shfl_xor_sync(0xffffffffu, cmax[i], 2));
            const float m_new = fmaxf(m_run[i], cmax[i]);
            m_use[i] = m_new == -INFINITY ? 0.f : m_new;
            scale_old[i] = exp2f(m_run[i] - m_use[i]);
            m_run[i] = m_new;
        }
        float csum[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < CHUNK / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int i = e >> 1;
                const float pexp = exp2f(s[nt][e] - m_use[i]);
                s[nt][e] = pexp;
                csum[i] += pexp;
            }
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            csum[i] += __shfl_xor_sync(0xffffffffu, csum[i], 1);
            csum[i] += __shfl_xor_sync(0xffffffffu, csum[i], 2);
            l_run[i] = l_run[i] * scale_old[i] + csum[i];
        }
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt) {
            o[nt][0] *= scale_old[0]; o[nt][1] *= scale_old[0];
            o[nt][2] *= scale_old[1]; o[nt][3] *= scale_old[1];
        }
        // O += P V
#pragma unroll
        for (int kk = 0; kk < CHUNK / 16; ++kk) {
            uint32_t pa[4];
            pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
            pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
            pa[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
            pa[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
            for (int np = 0; np < HD / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                const int key = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
                const int u = np * 2 + (lane >> 4);
                ldsm_x4_t(sv + kv_off(key, u), b0, b1, b2, b3);
                mma_bf16(o[np * 2], pa, b0, b1);
                mma_bf16(o[np * 2 + 1], pa, b2, b3);
            }
        }
        __syncthreads();
    }
    // partial (m, l, o) per (row, head, split)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        if (!pv[i]) continue;
        const size_t idx = ((size_t)(seq * RT + pr[i]) * a.Hq + ph[i]) * a.n_split_max + split;
        if ((lane & 3) == 0) a.part_ml[idx] = make_float2(m_run[i], l_run[i]);
        float* po = a.part_o + idx * HD + (lane & 3) * 2;
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt)
            *reinterpret_cast<float2*>(po + nt * 8) = make_float2(o[nt][i * 2], o[nt][i * 2 + 1]);
    }
}


// ---- tail: positions T0..P of one (row, head) pair, one warp, lane j owns key j of a 32-key chunk
__device__ __forceinline__ int nth_set_bit128(unsigned long long lo, unsigned long long hi, int n) {
    int c = __popcll(lo);
    unsigned long long m = lo;
    int base = 0;
    if (n >= c) { n -= c; m = hi; base = 64; }
    for (int i = 0; i < n; ++i) m &= m - 1;
    return m ? base + __ffsll((long long)m) - 1 : -1;
}

__device__ __forceinline__ void merge_ml(float& m, float& l, float (&o)[4], float cm, float cl, const float (&co)[4]) {
    const float mn = fmaxf(m, cm);
    const float a = exp2f(m - mn), b = exp2f(cm - mn);
    l = l * a + cl * b;
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = o[i] * a + co[i] * b;
    m = mn;
}

__global__ void __launch_bounds__(128, 3) k_attn_tree(AttnArgs a, int n_split_launch, int group, int rows_per_tile, int n_row_tiles) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_T0max;
    // Everything read before pdl_wait() -- the sequence state and the cache below T0 -- was written by earlier
    // steps; the queries and the block's own keys/values (written by the preceding kernel) are read after it.
    if (threadIdx.x == 0) pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x;                    // >= n_split_launch: the tail CTAs of the group
    const int kvh = blockIdx.y / n_row_tiles, rtile = blockIdx.y % n_row_tiles;
    const int seq = blockIdx.z;

    int n_rows, L;
    if (a.st) {
        const SeqState* st = a.st + seq;
        n_rows = st->active ? st->n_rows : 0;
        L = st->L;
    } else {
        n_rows = a.n_rows_fixed;
        L = a.L_fixed;
    }
    const int row0 = rtile * rows_per_tile;
    if (row0 >= n_rows) { pdl_wait(); return; }
    // the group needs keys up to the largest T0 of its rows (one round trip: a lane per row, then a warp max)
    if (warp == 0) {
        int t0 = 0;
        for (int r = row0 + lane; r < row0 + rows_per_tile && r < n_rows; r += 32) {
            const int depth = a.st ? a.st[seq].row_depth[r] : a.depth[seq * RT + r];
            t0 = max(t0, tail_start_mma(L + depth, a.dcap));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t0 = max(t0, __shfl_xor_sync(0xffffffffu, t0, o));
        if (lane == 0) s_T0max = t0;
    }
    __syncthreads();
    const int T0max = s_T0max;
    const int n_bulk = (T0max + a.split_len - 1) / a.split_len;     // bulk CTAs of this group that have keys
    const bool is_tail = split >= n_split_launch;
    if (!is_tail && split >= n_bulk) { pdl_wait(); return; }

    const __nv_bfloat16* kbase = reinterpret_cast<const __nv_bfloat16*>(a.kc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    const __nv_bfloat16* vbase = reinterpret_cast<const __nv_bfloat16*>(a.vc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;

    if (is_tail) {
        // ---------------- tail CTA t of the group: warp w takes pairs t*8 + w*2 + {0, 1}
        float* s_q = reinterpret_cast<float*>(smem) + warp * HD;
        const int tail_cta = split - n_split_launch;
        pdl_wait();
        for (int pi = 0; pi < PAIRS / TAIL_CTAS / 4; ++pi) {
            const int pidx = tail_cta * (PAIRS / TAIL_CTAS) + warp * (PAIRS / TAIL_CTAS / 4) + pi;
            const int r = row0 + pidx / group, head = kvh * group + pidx % group;
            if (r >= n_rows) break;
            int depth;
            unsigned long long lo, hi;
            if (a.st) {
                depth = a.st[seq].row_depth[r]; lo = a.st[seq].row_anc[r][0]; hi = a.st[seq].row_anc[r][1];
            } else {
                depth = a.depth[seq * RT + r]; lo = a.anc[(size_t)(seq * RT + r) * 2]; hi = a.anc[(size_t)(seq * RT + r) * 2 + 1];
            }
            const int P = L + depth, T0 = tail_start_mma(P, a.dcap);
            const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((size_t)(seq * RT + r) * a.Hq + head) * HD;
            __syncwarp();
            {
                const uint2 qq = *reinterpret_cast<const uint2*>(q + lane * 4);
                const __nv_bfloat162 q01 = *reinterpret_cast<const __nv_bfloat162*>(&qq.x), q23 = *reinterpret_cast<const __nv_bfloat162*>(&qq.y);
                s_q[lane * 4 + 0] = __low2float(q01); s_q[lane * 4 + 1] = __high2float(q01);
                s_q[lane * 4 + 2] = __low2float(q23); s_q[lane * 4 + 3] = __high2float(q23);
            }
            __syncwarp();
            float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
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
                    uint4 kreg[HD / 8];
#pragma unroll
                    for (int d8 = 0; d8 < HD / 8; ++d8) kreg[d8] = kr[d8];
                    float acc = 0.f;
#pragma unroll
                    for (int d8 = 0; d8 < HD / 8; ++d8) {
                        const uint4 kk = kreg[d8];
                        const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kk);
                        const float4 qa = *reinterpret_cast<const float4*>(s_q + d8 * 8), qb = *reinterpret_cast<const float4*>(s_q + d8 * 8 + 4);
                        acc = fmaf(qa.x, __low2float(k2[0]), acc); acc = fmaf(qa.y, __high2float(k2[0]), acc);
                        acc = fmaf(qa.z, __low2float(k2[1]), acc); acc = fmaf(qa.w, __high2float(k2[1]), acc);
                        acc = fmaf(qb.x, __low2float(k2[2]), acc); acc = fmaf(qb.y, __high2float(k2[2]), acc);
                        acc = fmaf(qb.z, __low2float(k2[3]), acc); acc = fmaf(qb.w, __high2float(k2[3]), acc);
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
                // weighted values, keys in position order; the loads of 8 keys are issued before their sums
                // (a key that is not in the chunk reads slot 0 with weight 0 and is skipped)
                for (int j0 = 0; j0 < 32; j0 += 8) {
                    float pj[8];
                    uint2 vv[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        pj[u] = __shfl_sync(0xffffffffu, pe, j0 + u);
                        const int sj = __shfl_sync(0xffffffffu, slot, j0 + u);
                        vv[u] = *reinterpret_cast<const uint2*>(vbase + (size_t)sj * HD + lane * 4);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (pj[u] != 0.f) {
                            const __nv_bfloat162 v01 = *reinterpret_cast<const __nv_bfloat162*>(&vv[u].x), v23 = *reinterpret_cast<const __nv_bfloat162*>(&vv[u].y);
                            co[0] = fmaf(pj[u], __low2float(v01), co[0]); co[1] = fmaf(pj[u], __high2float(v01), co[1]);
                            co[2] = fmaf(pj[u], __low2float(v23), co[2]); co[3] = fmaf(pj[u], __high2float(v23), co[3]);
                        }
                    }
                }
                merge_ml(m, l, o, cm, cl, co);
            }
            const size_t idx = ((size_t)(seq * RT + r) * a.Hq + head) * a.n_split_max + (a.n_split_max - 1);
            if (lane == 0) a.part_ml[idx] = make_float2(m, l);
            *reinterpret_cast<float4*>(a.part_o + idx * HD + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
        }
    } else {
        // ---------------- bulk CTA
        attn_bulk_chunks(a, smem, seq, kvh, row0, split, group, n_rows, L, T0max, kbase, vbase);
    }

}

// Merge of the partials of one (row, head) pair, one warp per pair: bulk splits in split order, the tail last.
__global__ void __launch_bounds__(128) k_attn_merge(AttnArgs a) {
    pdl_wait();
    if (threadIdx.x == 0) pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 4 + warp, head = blockIdx.y, seq = blockIdx.z;
    int n_rows, L;
    if (a.st) {
        const SeqState* st = a.st + seq;
        n_rows = st->active ? st->n_rows : 0;
        L = st->L;
    } else {
        n_rows = a.n_rows_fixed;
        L = a.L_fixed;
    }
    if (r >= n_rows) return;
    {
        const int depth = a.st ? a.st[seq].row_depth[r] : a.depth[seq * RT + r];
        const int T0 = tail_start_mma(L + depth, a.dcap);
        const int n_sp = (T0 + a.split_len - 1) / a.split_len;
        const size_t base = ((size_t)(seq * RT + r) * a.Hq + head) * a.n_split_max;
        float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
        for (int s0 = 0; s0 <= n_sp; s0 += 8) {
            float2 ml[8];
            float4 c4[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int sp = s0 + u;
                const size_t idx = base + (sp < n_sp ? sp : a.n_split_max - 1);
                if (sp <= n_sp) {
                    ml[u] = __ldcg(a.part_ml + idx);
                    c4[u] = __ldcg(reinterpret_cast<const float4*>(a.part_o + idx * HD + lane * 4));
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (s0 + u <= n_sp) {
                    const float co[4] = {c4[u].x, c4[u].y, c4[u].z, c4[u].w};
                    merge_ml(m, l, o, ml[u].x, ml[u].y, co);
                }
            }
        }
        const float inv = 1.0f / l;
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out) + ((size_t)(seq * RT + r) * a.Hq + head) * HD + lane * 4;
        const __nv_bfloat162 o01 = __floats2bfloat162_rn(o[0] * inv, o[1] * inv), o23 = __floats2bfloat162_rn(o[2] * inv, o[3] * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t*>(&o01);
        pk.y = *reinterpret_cast<const uint32_t*>(&o23);
        *reinterpret_cast<uint2*>(out) = pk;
    }
}

}  // namespace

// Two launches: k_attn_tree with grid.x = bulk splits + TAIL_CTAS tail CTAs per (KV head, row tile) group, each
// storing (max, sum, weighted values) partials, then k_attn_merge with one warp per (row, head).
int launch_attn_tree(const AttnArgs& a, int batch, int n_split_launch, cudaStream_t s, bool pdl) {
    if (a.h != HD || a.Hq % a.Hkv) return -1;
    const int group = a.Hq / a.Hkv;
    if (group > PAIRS || PAIRS % group) return -1;
    const int rows_per_tile = PAIRS / group;
    const int n_row_tiles = (RT + rows_per_tile - 1) / rows_per_tile;
    if (n_split_launch + 1 > a.n_split_max) return -1;
    static bool attr_set = false;
    const int smem = 4 * KV_TILE_BYTES;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_attn_tree, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return -1;
        attr_set = true;
    }
    dim3 grid(n_split_launch + TAIL_CTAS, a.Hkv * n_row_tiles, batch);
    launch_k(k_attn_tree, grid, dim3(128), (size_t)smem, s, pdl, a, n_split_launch, group, rows_per_tile, n_row_tiles);
    launch_k(k_attn_merge, dim3((RT + 3) / 4, a.Hq, batch), dim3(128), 0, s, pdl, a);
    return 0;
}

}  // namespace esp
