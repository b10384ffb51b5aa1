// Tensor-core "bulk" part of the tree attention for bf16, head_dim 128.
//
// A row at position P attends to cache positions 0..T0-1 here (T0 as in
// tail_start(): the 16-aligned position below which keys are always cache
// resident); the remaining positions, including the row's in-flight tree
// ancestors, are summed by the tail kernel.  The KV cache of one KV head is
// streamed once per split through shared memory (16-byte cp.async, XOR
// swizzle) and shared by all query heads of the group and all block rows:
// a CTA holds 64 (row, head) pairs, a warp 16 of them, Q.K^T and P.V run on
// mma.sync m16n8k16 with fp32 online softmax in registers.
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

__global__ void __launch_bounds__(128) k_attn_bulk_mma(AttnArgs a, int n_split_launch, int group, int rows_per_tile, int n_row_tiles) {
    extern __shared__ __align__(128) unsigned char smem[];
    pdl_wait();
    if (threadIdx.x == 0) pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x;
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
    if (row0 >= n_rows) return;
    // per-thread pairs: A = warp*16 + lane/4, B = A + 8
    int pr[2], ph[2], pT0[2];
    bool pv[2];
    int T0max = 0;
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
    // the CTA needs keys up to the largest T0 of its rows (block-uniform: computed from all rows of the tile)
    for (int r = row0; r < min(row0 + rows_per_tile, n_rows); ++r) {
        const int depth = a.st ? a.st[seq].row_depth[r] : a.depth[seq * RT + r];
        T0max = max(T0max, tail_start_mma(L + depth, a.dcap));
    }
    const int beg = split * a.split_len;
    const int end = min(beg + a.split_len, T0max);
    if (beg >= end) return;

    const __nv_bfloat16* kbase = reinterpret_cast<const __nv_bfloat16*>(a.kc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
    const __nv_bfloat16* vbase = reinterpret_cast<const __nv_bfloat16*>(a.vc) + ((size_t)seq * a.Hkv + kvh) * a.cap * HD;
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

    const int n_chunks = (end - beg + CHUNK - 1) / CHUNK;
    load_chunk(0, 0);
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

}  // namespace

int launch_attn_bulk_mma(const AttnArgs& a, int batch, int n_split_launch, cudaStream_t s, bool pdl) {
    if (a.h != HD || a.Hq % a.Hkv) return -1;
    const int group = a.Hq / a.Hkv;
    if (group > PAIRS || PAIRS % group) return -1;
    const int rows_per_tile = PAIRS / group;
    const int n_row_tiles = (RT + rows_per_tile - 1) / rows_per_tile;
    static bool attr_set = false;
    const int smem = 4 * KV_TILE_BYTES;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_attn_bulk_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return -1;
        attr_set = true;
    }
    dim3 grid(n_split_launch, a.Hkv * n_row_tiles, batch);
    launch_k(k_attn_bulk_mma, grid, dim3(128), (size_t)smem, s, pdl, a, n_split_launch, group, rows_per_tile, n_row_tiles);
    return 0;
}

}  // namespace esp
