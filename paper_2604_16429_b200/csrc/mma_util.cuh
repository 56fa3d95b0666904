// Warp-level tensor-core helpers (mma.sync m16n8k16 bf16, ldmatrix, cp.async) used by the
// backward kernels.  Tiles are 64 rows x 64 bf16 (128 bytes per row) in shared memory with the
// 16-byte pieces of a row XOR-swizzled by (row & 7), so every ldmatrix phase is conflict free.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace mosaic {

constexpr int kTileBytes = kChunk * kD * 2;  // 8 KB

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

// Stage chunk c of block j of one [N,d] bf16 tensor (unit base `x`) into a swizzled tile.
template <int THREADS>
__device__ __forceinline__ void load_tile(uint32_t tile, const __nv_bfloat16* __restrict__ x, const Geo& g, int j,
                                          int c, int tid) {
#pragma unroll
  for (int it = 0; it < (kChunk * 8) / THREADS; ++it) {
    int p = tid + it * THREADS;
    int row = p >> 3, ch = p & 7;
    const __nv_bfloat16* src = x + chunk_token(g, j, c, row) * kD + ch * 8;
    cp_async16(tile + row * 128 + ((ch ^ (row & 7)) << 4), src);
  }
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// A fragment: rows row0..row0+15, columns 16*kk..16*kk+15 of a [row][col] tile.
__device__ __forceinline__ void load_A(uint32_t tile, int row0, int kk, int lane, uint32_t (&a)[4]) {
  int row = row0 + (lane & 15), ch = kk * 2 + (lane >> 4);
  ldsm_x4(tile + row * 128 + ((ch ^ (row & 7)) << 4), a);
}
// B fragments of two n-tiles for B[k][n] = T[n][k] (tile rows are n): n in n0..n0+15, k-step kk.
// r[0], r[1] belong to n-tile n0/8; r[2], r[3] to the next one.
__device__ __forceinline__ void load_B(uint32_t tile, int n0, int kk, int lane, uint32_t (&r)[4]) {
  int row = n0 + (lane & 7) + ((lane >> 4) << 3), ch = kk * 2 + ((lane >> 3) & 1);
  ldsm_x4(tile + row * 128 + ((ch ^ (row & 7)) << 4), r);
}
// B fragments of two n-tiles for B[k][n] = T[k][n] (tile rows are k): k in k0..k0+15, n in n0..n0+15.
__device__ __forceinline__ void load_Bt(uint32_t tile, int k0, int n0, int lane, uint32_t (&r)[4]) {
  int row = k0 + (lane & 7) + (((lane >> 3) & 1) << 3), ch = (n0 >> 3) + (lane >> 4);
  ldsm_x4_t(tile + row * 128 + ((ch ^ (row & 7)) << 4), r);
}

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// C[16 x 64] += A[16 x 64] * B, A given as four k-step fragments, B[k][n] = T[n][k].
__device__ __forceinline__ void gemm_nt(float (&c)[8][4], const uint32_t (&a)[4][4], uint32_t tile, int lane) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk)
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t r[4];
      load_B(tile, np * 16, kk, lane, r);
      mma16816(c[2 * np], a[kk], r[0], r[1]);
      mma16816(c[2 * np + 1], a[kk], r[2], r[3]);
    }
}
// C[16 x 64] += A[16 x 64] * T, T a [k][n] tile (k = the 64 tile rows).
__device__ __forceinline__ void gemm_nn(float (&c)[8][4], const uint32_t (&a)[4][4], uint32_t tile, int lane) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk)
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t r[4];
      load_Bt(tile, kk * 16, np * 16, lane, r);
      mma16816(c[2 * np], a[kk], r[0], r[1]);
      mma16816(c[2 * np + 1], a[kk], r[2], r[3]);
    }
}
// Accumulator layout [16 x 64] fp32 -> A-operand fragments (bf16) of the same matrix.
__device__ __forceinline__ void acc_to_A(const float (&c)[8][4], uint32_t (&a)[4][4]) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    a[kk][0] = pack_bf16(c[2 * kk][0], c[2 * kk][1]);
    a[kk][1] = pack_bf16(c[2 * kk][2], c[2 * kk][3]);
    a[kk][2] = pack_bf16(c[2 * kk + 1][0], c[2 * kk + 1][1]);
    a[kk][3] = pack_bf16(c[2 * kk + 1][2], c[2 * kk + 1][3]);
  }
}

}  // namespace mosaic
