// Warp-level tensor-core building blocks for the tiled kernels: 16-byte async copies into
// swizzled shared-memory tiles, ldmatrix fragment loads and the bf16 m16n8k16 MMA.
//
// Shared tiles hold rows of 64 bf16 (128 bytes, eight 16-byte chunks); chunk c of row r
// lives at chunk position c ^ (r & 7), so the eight rows an ldmatrix reads at one chunk
// index fall into eight different bank groups.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace bpt {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of 16-byte chunk `chunk` of row `row` inside a [rows][64] bf16 tile
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// A fragments (16 rows x 64 k) of rows row0.. of a swizzled tile: a[ks][0..3] for k-step ks
__device__ __forceinline__ void load_a_frags(uint32_t tile_base, int row0, int lane, uint32_t (&a)[4][4]) {
    // matrix j of the x4: rows (j & 1) * 8, k-chunk (j >> 1)
    const int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const int cj = lane >> 4;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) ldsm_x4(tile_base + tile_off(r, ks * 2 + cj), a[ks][0], a[ks][1], a[ks][2], a[ks][3]);
}

// B fragments for S = A * X^T where X is a swizzled [rows][64] tile (rows = n index):
// two n8 tiles (rows row0..row0+15), k-step ks.  b[0..1]: rows row0..+7, b[2..3]: rows +8..+15.
__device__ __forceinline__ void load_b_rows(uint32_t tile_base, int row0, int ks, int lane, uint32_t (&b)[4]) {
    const int r = row0 + (lane & 7) + (lane >> 4) * 8;
    const int cj = (lane >> 3) & 1;
    ldsm_x4(tile_base + tile_off(r, ks * 2 + cj), b[0], b[1], b[2], b[3]);
}

// B fragments for O = P * X where X is a swizzled [rows][64] tile (rows = k index): k-step
// over rows row0..row0+15, two n8 tiles of columns 16*np .. 16*np+15.
// b[0..1]: columns 16np..+7, b[2..3]: columns 16np+8..+15.
__device__ __forceinline__ void load_b_cols(uint32_t tile_base, int row0, int np, int lane, uint32_t (&b)[4]) {
    const int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const int cj = lane >> 4;
    ldsm_x4_t(tile_base + tile_off(r, np * 2 + cj), b[0], b[1], b[2], b[3]);
}

// A fragment of X^T for a k-step of 16 rows of X: X is stored [k index][m index] (bf16, row
// stride `stride` bytes); returns A(m0.., k0..) of the m16 x k16 product operand.
__device__ __forceinline__ void load_a_trans(uint32_t base, int stride, int k0, int m0, int lane, uint32_t (&a)[4]) {
    const int krow = k0 + (lane & 7) + ((lane >> 4) & 1) * 8;
    const int mchunk = (m0 >> 3) + ((lane >> 3) & 1);
    ldsm_x4_t(base + krow * stride + mchunk * 16, a[0], a[1], a[2], a[3]);
}

// A fragment (16 rows x 16 k) of a plain row-major bf16 tile with row stride `stride` bytes.
__device__ __forceinline__ void load_a_plain(uint32_t base, int stride, int row0, int k0, int lane, uint32_t (&a)[4]) {
    const int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const int ch = (k0 >> 3) + (lane >> 4);
    ldsm_x4(base + r * stride + ch * 16, a[0], a[1], a[2], a[3]);
}

}  // namespace bpt
