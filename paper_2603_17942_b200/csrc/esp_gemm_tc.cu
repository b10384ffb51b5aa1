// Small-M bf16 GEMM for the decode-and-verify step on the Blackwell tensor
// cores: y[row][n] = sum_k x[row][k] * w[n][k] for at most 80 rows.
//
// The weight matrix is the MMA "A" operand (128 output features on the MMA-M
// dimension), the token rows are the "B" operand (MMA-N = 80), so the large
// operand fills the tensor core and the 80 rows cost no padding.  Both
// operands are K-major and arrive through TMA with the 128-byte swizzle;
// tcgen05.mma accumulates fp32 in tensor memory; four epilogue warps read it
// back with tcgen05.ld.
//
// The step is bound by streaming the weights once from HBM, so the work is
// cut stream-K style: the (tile, k-block) units of one GEMM are dealt out in
// equal contiguous ranges to one persistent CTA per SM.  A tile whose k-range
// is split over several CTAs is finished by whichever of them arrives last:
// every CTA stores its partial tile, bumps the tile's counter, and the last
// one sums the partials in CTA order (a fixed order, independent of arrival
// order and of the number of rows) and runs the fused epilogue.  No CTA ever
// waits for another.  Every mbarrier wait is bounded; on a timeout the
// kernel records DEV_E_WAIT_TIMEOUT, lets its copies drain, frees its tensor
// memory and returns.
#include <cuda.h>
#include <new>
#include <string.h>

#include "esp_epilogue.cuh"
#include "esp_launch.h"

namespace esp {

namespace {

constexpr int BK = 64;                       // k elements per stage (128 bytes of bf16)
constexpr int STAGES = 6;
constexpr int A_BYTES = TILE_N * BK * 2;     // 16384
constexpr int B_BYTES = RT * BK * 2;         // 10240
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TMEM_COLS = 256;               // two accumulator buffers of 128 columns
constexpr int NUM_THREADS = 192;
constexpr uint32_t WAIT_LIMIT = 1u << 20;

struct TcParams {
    CUtensorMap map_a[3];
    CUtensorMap map_b;
    int32_t rows_w[3];
    int32_t n_tiles, KB, grid, epi;
    float* partials;   // [grid][2][RT][TILE_N]
    int* counters;     // [n_tiles], zero between launches
    int* err;
    EpiArgs a;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait; false if it ran out (or another role already gave up).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    return false;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

// K-major operand tile in shared memory, rows of 128 bytes, 128-byte swizzle:
// 8-row groups are 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);       // start address
    d |= (uint64_t)1 << 16;                       // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset
    d |= (uint64_t)1 << 46;                       // descriptor version (Blackwell)
    d |= (uint64_t)2 << 61;                       // 128-byte swizzle
    return d;
}

// kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = 80
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(RT >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(IDESC), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// stream-K bookkeeping (all 64-bit so lm-head sized problems do not overflow)
__device__ __forceinline__ long long unit_begin(long long c, long long U, long long G) { return c * U / G; }
__device__ __forceinline__ int cta_of_unit(long long u, long long U, long long G) { return (int)(((u + 1) * G + U - 1) / U - 1); }

// which weight matrix / row the two 64-row halves of a tile come from
template <int EPI>
__device__ __forceinline__ void tile_source(const TcParams& p, int tile, int half, int& m, int& row) {
    if (EPI == EPI_SWIGLU) { m = half; row = tile * 64; return; }
    int feat = tile * TILE_N;
    m = 0;
    while (m < 2 && feat >= p.rows_w[m]) { feat -= p.rows_w[m]; ++m; }
    row = feat + half * 64;
}

template <int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1) k_gemm_tc(const __grid_constant__ TcParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* stages = smem;
    float* s_acc = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES);
    float* s_aux = s_acc + RT * ACC_LD;
    uint64_t* full = reinterpret_cast<uint64_t*>(s_aux + RT * 4);
    uint64_t* empty = full + STAGES;
    uint64_t* tfull = empty + STAGES;
    uint64_t* tempty = tfull + 2;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
    int* s_flag = const_cast<int*>(s_abort) + 1;    // [0] = wait failures of the epilogue warps, [1] = "I am last"

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long U = (long long)p.n_tiles * p.KB, G = p.grid;
    const long long u0 = unit_begin(blockIdx.x, U, G), u1 = unit_begin(blockIdx.x + 1, U, G);

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 128); }
        *s_abort = 0;
        s_flag[0] = 0;
        s_flag[1] = 0;
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

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (long long u = u0; u < u1 && ok;) {
                const int tile = (int)(u / p.KB), kb0 = (int)(u % p.KB);
                const int kb1 = (int)min((long long)p.KB, kb0 + (u1 - u));
                int m0, r0, m1, r1;
                tile_source<EPI>(p, tile, 0, m0, r0);
                tile_source<EPI>(p, tile, 1, m1, r1);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1, s_abort)) { ok = false; break; }
                    unsigned char* sa = stages + stage * STAGE_BYTES;
                    mbar_expect_tx(&full[stage], STAGE_BYTES);
                    tma_load_2d(sa, &p.map_a[m0], kb * BK, r0, &full[stage]);
                    tma_load_2d(sa + A_BYTES / 2, &p.map_a[m1], kb * BK, r1, &full[stage]);
                    tma_load_2d(sa + A_BYTES, &p.map_b, kb * BK, 0, &full[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                u += kb1 - kb0;
            }
            if (!ok) { set_error(p.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            int stage = 0, seg = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (long long u = u0; u < u1 && ok; ++seg) {
                const int kb0 = (int)(u % p.KB);
                const int kb1 = (int)min((long long)p.KB, kb0 + (u1 - u));
                const int buf = seg & 1;
                if (!mbar_wait(&tempty[buf], ((seg >> 1) & 1) ^ 1, s_abort)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + buf * 128;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&full[stage], phase, s_abort)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = smem_u32(stages + stage * STAGE_BYTES);
                    const uint64_t da = smem_desc(sa), db = smem_desc(sa + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma(tmem_d, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), (kb > kb0 || k > 0) ? 1u : 0u);
                    umma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit(&tfull[buf]);
                u += kb1 - kb0;
            }
            if (!ok) { set_error(p.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
        }
    } else {
        // ---------------- epilogue warps: TMEM -> registers -> partial or fused epilogue
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int f = q * 32 + lane;            // feature of the tile owned by this thread
        const int et = threadIdx.x - 64;        // 0..127 index among the epilogue threads
        const int n_rows = p.a.st ? (p.a.st->active ? p.a.st->n_rows : 0) : p.a.rows_fixed;
        int seg = 0;
        bool ok = true;
        for (long long u = u0; u < u1 && ok; ++seg) {
            const int tile = (int)(u / p.KB), kb0 = (int)(u % p.KB);
            const int kb1 = (int)min((long long)p.KB, kb0 + (u1 - u));
            const int buf = seg & 1;
            bool mine = true;
            if (lane == 0) mine = mbar_wait(&tfull[buf], (seg >> 1) & 1, s_abort);
            if (lane == 0 && !mine) atomicOr(&s_flag[0], 1);
            epi_bar(2);
            if (s_flag[0]) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + buf * 128 + ((uint32_t)(q * 32) << 16);
            const long long t_first = (long long)tile * p.KB;
            const int c_first = cta_of_unit(t_first, U, G), c_last = cta_of_unit(t_first + p.KB - 1, U, G);
            const bool whole = c_first == c_last;
            const int slot = (tile == (int)(u0 / p.KB)) ? 0 : 1;
            float* part = p.partials + ((size_t)(blockIdx.x * 2 + slot) * RT) * TILE_N;
#pragma unroll
            for (int c = 0; c < RT / 16; ++c) {
                float v[16];
                tmem_ld16(taddr + c * 16, v);
                if (whole) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) s_acc[(c * 16 + i) * ACC_LD + f] = v[i];
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c * 16 + i < n_rows) __stcg(&part[(c * 16 + i) * TILE_N + f], v[i]);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(&tempty[buf]);
            bool finish = whole;
            if (!whole) {
                __threadfence();
                epi_bar(2);
                if (et == 0) {
                    const int old = atomicAdd(&p.counters[tile], 1);
                    s_flag[1] = (old == c_last - c_first) ? 1 : 0;
                }
                epi_bar(2);
                finish = s_flag[1] != 0;
                if (finish) {
                    __threadfence();
                    for (int r = 0; r < n_rows; ++r) {
                        float acc = 0.f;
                        for (int c = c_first; c <= c_last; ++c) {
                            const int cslot = (tile == (int)(unit_begin(c, U, G) / p.KB)) ? 0 : 1;
                            acc += __ldcg(&p.partials[((size_t)(c * 2 + cslot) * RT + r) * TILE_N + f]);
                        }
                        s_acc[r * ACC_LD + f] = acc;
                    }
                    if (et == 0) p.counters[tile] = 0;
                }
            }
            if (finish) {
                epi_bar(2);
                run_epilogue<__nv_bfloat16, EPI>(s_acc, s_aux, tile, 0, p.a, f, 2);
            }
            epi_bar(2);
            u += kb1 - kb0;
        }
        if (!ok && lane == 0) { set_error(p.err, DEV_E_WAIT_TIMEOUT); *s_abort = 1; }
    }
    // ---------------- teardown (every thread arrives here)
    __syncthreads();
    if (*s_abort) {
        // give copies that may still be in flight time to land before the block's shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

constexpr size_t SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + sizeof(float) * (RT * ACC_LD + RT * 4) + 256;

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) return nullptr;
        fn = reinterpret_cast<EncodeFn>(p);
    }
    return fn;
}

// [rows][K] bf16 row-major, box = 64 k-elements x box_rows rows, 128-byte swizzle, out-of-range reads give zero
int make_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows) {
    EncodeFn enc = get_encode();
    if (!enc) return -1;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

}  // namespace

struct TcGemm {
    TcParams p;
};

size_t tc_gemm_partial_bytes(int n_sm) { return (size_t)n_sm * 2 * RT * TILE_N * sizeof(float); }
int tc_gemm_counter_ints() { return 4096; }
int tc_gemm_tiles(const TcGemm* g) { return g ? g->p.n_tiles : 0; }

int tc_gemm_create(TcGemm** out, int epi, const void* const w[3], const int32_t rows_w[3], int K, const void* x, int batch,
                   void* partials, size_t partial_bytes, int* counters, int n_sm, int* err) {
    if (!out || batch != 1 || K % 8 || n_sm < 1) return -1;
    if (reinterpret_cast<uintptr_t>(x) % 16) return -1;
    TcGemm* g = new (std::nothrow) TcGemm();
    if (!g) return -1;
    memset(&g->p, 0, sizeof(g->p));
    TcParams& p = g->p;
    int total_rows = 0;
    for (int i = 0; i < 3; ++i) {
        p.rows_w[i] = rows_w[i];
        if (w[i] && rows_w[i] > 0) {
            if (reinterpret_cast<uintptr_t>(w[i]) % 16 || make_map(&p.map_a[i], w[i], rows_w[i], K, 64)) { delete g; return -1; }
            total_rows += rows_w[i];
        } else if (i > 0) {
            p.map_a[i] = p.map_a[0];
        }
    }
    if (make_map(&p.map_b, x, RT, K, RT)) { delete g; return -1; }
    p.epi = epi;
    p.n_tiles = epi == EPI_SWIGLU ? (rows_w[0] + 63) / 64 : (total_rows + TILE_N - 1) / TILE_N;
    p.KB = (K + BK - 1) / BK;
    const long long U = (long long)p.n_tiles * p.KB;
    p.grid = (int)(U < n_sm ? U : n_sm);
    if (p.n_tiles > tc_gemm_counter_ints() || tc_gemm_partial_bytes(p.grid) > partial_bytes) { delete g; return -1; }
    p.partials = reinterpret_cast<float*>(partials);
    p.counters = counters;
    p.err = err;
    *out = g;
    return 0;
}

void tc_gemm_destroy(TcGemm* g) { delete g; }

int tc_gemm_launch(const TcGemm* g, const EpiArgs& a, cudaStream_t s) {
    if (!g) return ESP_E_ARG;
    TcParams p = g->p;
    p.a = a;
#define ESP_TC_CASE(E)                                                                                        \
    case E: {                                                                                                 \
        static bool attr_set = false;                                                                         \
        if (!attr_set) {                                                                                      \
            if (cudaFuncSetAttribute(k_gemm_tc<E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess) return ESP_E_CUDA; \
            attr_set = true;                                                                                  \
        }                                                                                                     \
        k_gemm_tc<E><<<p.grid, NUM_THREADS, SMEM_BYTES, s>>>(p);                                              \
    } break;
    switch (p.epi) {
        ESP_TC_CASE(EPI_STORE_F32)
        ESP_TC_CASE(EPI_QKV)
        ESP_TC_CASE(EPI_RESID)
        ESP_TC_CASE(EPI_SWIGLU)
        ESP_TC_CASE(EPI_LOGITS)
        default: return ESP_E_ARG;
    }
#undef ESP_TC_CASE
    return cudaGetLastError() == cudaSuccess ? ESP_OK : ESP_E_CUDA;
}

}  // namespace esp
