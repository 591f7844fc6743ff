// Pieces shared by the tensor-core kernels: chunk geometry, host-side tensor-map
// encoding, the per-segment state records in the workspace, and the device helpers
// for the feature map on a swizzled tile row.
#pragma once

#include <cudaTypedefs.h>

#include "la_common.cuh"
#include "la_sm100.cuh"

namespace la {
namespace tc {

constexpr int kChunk = 128;                  // positions per chunk = MMA M
constexpr int kDim = 64;                     // D = M = 64: one 128-byte swizzle row
constexpr int kTileBytes = kChunk * kDim * 2;  // one [128][64] bf16 tile
constexpr int kStateFloats = kDim * (kDim + 1);  // [S (64x64) | Z (64)] per record

// How a (batch, head) sequence is cut into segments that run concurrently.
struct Segmentation {
    int nseg;             // segments per sequence
    int chunks_per_seg;   // chunks in every segment but possibly the last
};

// 2-D view of a [rows][64] bf16 tensor with a [box_rows][64] box and the 128-byte swizzle.
int encode_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows);

// ---------------------------------------------------------------------------
// Feature map on one 128-byte row of a swizzled tile, in place: thread-per-row.
// `row_base` is the shared-memory address of the row; r7 = row & 7 (swizzle key).
// ---------------------------------------------------------------------------
__device__ __forceinline__ float phi_fast(float x) {
    // elu(x) + 1 with the hardware exponential: exp(x) = 2^(x * log2 e)
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 1.4426950408889634f));
    return x > 0.f ? x + 1.f : e;
}

__device__ __forceinline__ void phi_row_inplace(uint32_t row_base, uint32_t r7) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        // elementwise, so the logical order is irrelevant; visiting chunk c ^ r7 keeps the
        // eight rows of a quarter-warp on eight different bank groups
        const uint32_t addr = row_base + ((c ^ r7) << 4);
        uint32_t v0, v1, v2, v3;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(addr));
        v0 = sm100::pack_bf16x2(phi_fast(sm100::bf16_lo(v0)), phi_fast(sm100::bf16_hi(v0)));
        v1 = sm100::pack_bf16x2(phi_fast(sm100::bf16_lo(v1)), phi_fast(sm100::bf16_hi(v1)));
        v2 = sm100::pack_bf16x2(phi_fast(sm100::bf16_lo(v2)), phi_fast(sm100::bf16_hi(v2)));
        v3 = sm100::pack_bf16x2(phi_fast(sm100::bf16_lo(v3)), phi_fast(sm100::bf16_hi(v3)));
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v0), "r"(v1), "r"(v2), "r"(v3) : "memory");
    }
}

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t (&v)[4]) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

}  // namespace tc
}  // namespace la
