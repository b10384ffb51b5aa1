// Pieces of the small-M tcgen05 GEMM shared by the kernel that runs one GEMM per launch and the kernel
// that runs all layers in one launch: stage geometry, the instruction descriptor and the walk over a CTA's
// stream-K range.
#pragma once

#include "esp_launch.h"
#include "esp_tc.cuh"

namespace esp {

constexpr int BK = 64;                       // k elements per stage (128 bytes of bf16)
constexpr int A_BYTES = TILE_N * BK * 2;     // one (tile, k-block) unit of repacked weights: 16384

// kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = 80 per sequence
__host__ __device__ constexpr uint32_t idesc_of(int nr) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nr >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);
}

// One (tile, k-range) piece of a CTA's stream-K range.
struct Seg {
    int tile, kb0, kb1, slot;
    bool whole;
};

// A CTA's unit range [u0, u1) cut at tile boundaries.  Segments are handed out with the partial ones first
// (tail piece, then head piece), whole tiles after them: partial tiles are then complete early in every
// CTA's timeline and the CTA that finishes one does so while the weight stream of its whole tiles is running.
struct Range {
    int first_tile, last_tile, head_kb0, tail_kb1, KB, n_seg, slots;
    bool tail_partial;
};
__device__ __forceinline__ Range make_range(long long u0, long long u1, int KB, int slots) {
    Range r;
    r.KB = KB;
    r.slots = slots;
    r.first_tile = (int)(u0 / KB);
    r.head_kb0 = (int)(u0 % KB);
    r.last_tile = (int)((u1 - 1) / KB);
    r.tail_kb1 = (int)((u1 - 1) % KB) + 1;
    r.n_seg = r.last_tile - r.first_tile + 1;
    r.tail_partial = r.n_seg > 1 && r.tail_kb1 < KB;
    return r;
}
__device__ __forceinline__ Seg get_seg(const Range& r, int i) {
    Seg s;
    if (r.n_seg == 1) {
        s.tile = r.first_tile; s.kb0 = r.head_kb0; s.kb1 = r.tail_kb1; s.slot = 0;
    } else {
        // order: [tail if partial] head, middle tiles, [tail if whole]
        int idx = r.tail_partial ? i - 1 : i;
        if (idx < 0 || idx == r.n_seg - 1) { s.tile = r.last_tile; s.kb0 = 0; s.kb1 = r.tail_kb1; s.slot = 1; }
        else if (idx == 0) { s.tile = r.first_tile; s.kb0 = r.head_kb0; s.kb1 = r.KB; s.slot = 0; }
        else { s.tile = r.first_tile + idx; s.kb0 = 0; s.kb1 = r.KB; s.slot = 1; }
    }
    s.slot = s.tile - r.first_tile < r.slots - 1 ? s.tile - r.first_tile : r.slots - 1;
    s.whole = s.kb0 == 0 && s.kb1 == r.KB;
    return s;
}

// What the all-layers kernel needs to know about a GEMM plan (every layer has the same geometry).
struct TcGemmGeom {
    int n_tiles, KB, grid, slots, nrs, planes, plane_seqs;
    const TileSrc* table;            // contributor table of the consumers
    const unsigned char* packed;     // this plan's repacked weights
    float* partials;
    CUtensorMap map_b;               // activations, box of one sequence
};
void tc_gemm_geometry(const TcGemm* g, TcGemmGeom* out);

}  // namespace esp
