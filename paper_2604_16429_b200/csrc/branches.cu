// Compression branch and gated sum of the three-branch form of the operator.
//
// Paper: Eq. of the aggregated output (section "Native Sparse Attention") and the "Compression" paragraph of the
// section "Block-Sparse Attention": block-level softmax attention abar_ij over ALL m blocks on the mean-pooled
// queries and keys, obar_i = sum_j abar_ij vbar_j, the same vector for every token of query block i; then
//   o_l = g_CG(l) obar_i + g_FG(l) oFG_l + g_L(l) oL_l .
// The selection and local branch outputs oFG, oL come from two launches of the attention kernel (selected blocks
// only / neighbourhood only, each with its own softmax).
#include <cuda_bf16.h>

#include "common.cuh"

namespace mosaic {

namespace {

constexpr int kCR = 4;          // query blocks per warp
constexpr int kCW = 8;          // warps per CTA
constexpr int kCJ = 64;         // key blocks per staged chunk
constexpr int kCStr = kD + 4;   // padded row (floats)

struct CompressSmem {
  float qs[kCW * kCR][kCStr];   // pooled query sums of the CTA's rows
  float ks[kCJ][kCStr];         // pooled key sums of the chunk
  float vs[kCJ][kD];            // pooled value sums of the chunk
  float w[kCW * kCR][kCJ];      // softmax numerators of the chunk
};

// ------------------------------------------------------------------------------------------
// compress_kernel: streaming softmax attention on the pooled vectors, fp32 on the CUDA cores (2 m^2 d FLOP per
// unit and product: far too small for a tensor-core pipeline).  A CTA owns 32 query blocks of one unit (4 per
// warp) and stages the pooled keys and values in chunks of 64 blocks; a lane scores keys lane and lane + 32 of
// the chunk for its warp's rows and accumulates channels 2 lane, 2 lane + 1 of their outputs.
// Pooled sums are block SUMS: the means' 1/b enters as scale / b^2 on the logits and 1/b on the output.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kCW * 32) compress_kernel(Geo g, const float* __restrict__ pq,
                                                            const float* __restrict__ pk, const float* __restrict__ pv,
                                                            float* __restrict__ ocg, float* __restrict__ lse2) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  CompressSmem& sm = *reinterpret_cast<CompressSmem*>(smem_raw);
  constexpr int TI = kCW * kCR, NT = kCW * 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tiles = (g.m + TI - 1) / TI;
  const int u = blockIdx.x / tiles, i0 = (blockIdx.x - u * tiles) * TI;
  const float* pq_u = pq + (long long)u * g.m * kD;
  const float* pk_u = pk + (long long)kv_unit(g, u) * g.m * kD;   // grouped-query attention: the group's key/value head
  const float* pv_u = pv + (long long)kv_unit(g, u) * g.m * kD;
  const float inv_b = 1.0f / (float)g.b;
  const float sl2 = g.scale_log2 * inv_b * inv_b;  // logits in base-2 units

  for (int e = tid; e < TI * (kD / 4); e += NT) {
    const int r = e / (kD / 4), c4 = e - r * (kD / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + r < g.m) v = __ldg(reinterpret_cast<const float4*>(pq_u + (long long)(i0 + r) * kD + 4 * c4));
    *reinterpret_cast<float4*>(&sm.qs[r][4 * c4]) = v;
  }
  float mx[kCR], z[kCR], acc[kCR][2];
#pragma unroll
  for (int a = 0; a < kCR; ++a) { mx[a] = -INFINITY; z[a] = 0.f; acc[a][0] = 0.f; acc[a][1] = 0.f; }

  for (int j0 = 0; j0 < g.m; j0 += kCJ) {
    __syncthreads();  // the previous chunk is consumed (and qs is written on the first pass)
    for (int e = tid; e < kCJ * (kD / 4); e += NT) {
      const int jj = e / (kD / 4), c4 = e - jj * (kD / 4);
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
      if (j0 + jj < g.m) {
        kv = __ldg(reinterpret_cast<const float4*>(pk_u + (long long)(j0 + jj) * kD + 4 * c4));
        vv = __ldg(reinterpret_cast<const float4*>(pv_u + (long long)(j0 + jj) * kD + 4 * c4));
      }
      *reinterpret_cast<float4*>(&sm.ks[jj][4 * c4]) = kv;
      *reinterpret_cast<float4*>(&sm.vs[jj][4 * c4]) = vv;
    }
    __syncthreads();
    // scores of keys lane and lane + 32 for the warp's rows
    float s[kCR][2];
#pragma unroll
    for (int a = 0; a < kCR; ++a) { s[a][0] = 0.f; s[a][1] = 0.f; }
#pragma unroll 4
    for (int c4 = 0; c4 < kD / 4; ++c4) {
      const float4 k0 = *reinterpret_cast<const float4*>(&sm.ks[lane][4 * c4]);
      const float4 k1 = *reinterpret_cast<const float4*>(&sm.ks[lane + 32][4 * c4]);
#pragma unroll
      for (int a = 0; a < kCR; ++a) {
        const float4 qv = *reinterpret_cast<const float4*>(&sm.qs[warp * kCR + a][4 * c4]);
        s[a][0] = fmaf(qv.x, k0.x, fmaf(qv.y, k0.y, fmaf(qv.z, k0.z, fmaf(qv.w, k0.w, s[a][0]))));
        s[a][1] = fmaf(qv.x, k1.x, fmaf(qv.y, k1.y, fmaf(qv.z, k1.z, fmaf(qv.w, k1.w, s[a][1]))));
      }
    }
    const bool ok0 = j0 + lane < g.m, ok1 = j0 + lane + 32 < g.m;
#pragma unroll
    for (int a = 0; a < kCR; ++a) {
      const float x0 = ok0 ? s[a][0] * sl2 : -INFINITY, x1 = ok1 ? s[a][1] * sl2 : -INFINITY;
      float cm = fmaxf(x0, x1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
      const float nm = fmaxf(mx[a], cm);  // finite: every chunk holds at least one block
      const float alpha = exp2f(mx[a] - nm);
      mx[a] = nm;
      const float w0 = exp2f(x0 - nm), w1 = exp2f(x1 - nm);
      z[a] = z[a] * alpha + w0 + w1;   // this lane's share of the normaliser
      acc[a][0] *= alpha;
      acc[a][1] *= alpha;
      sm.w[warp * kCR + a][lane] = w0;
      sm.w[warp * kCR + a][lane + 32] = w1;
    }
    __syncwarp();
    // accumulate channels 2 lane, 2 lane + 1 over the chunk's keys
    const int nj = min(kCJ, g.m - j0);
    for (int jj = 0; jj < nj; ++jj) {
      const float2 vv = *reinterpret_cast<const float2*>(&sm.vs[jj][2 * lane]);
#pragma unroll
      for (int a = 0; a < kCR; ++a) {
        const float w = sm.w[warp * kCR + a][jj];
        acc[a][0] = fmaf(w, vv.x, acc[a][0]);
        acc[a][1] = fmaf(w, vv.y, acc[a][1]);
      }
    }
  }
#pragma unroll
  for (int a = 0; a < kCR; ++a) {
    float zz = z[a];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) zz += __shfl_xor_sync(0xffffffffu, zz, o);
    const int i = i0 + warp * kCR + a;
    if (i < g.m) {
      const float f = inv_b / zz;
      *reinterpret_cast<float2*>(ocg + ((long long)u * g.m + i) * kD + 2 * lane) = make_float2(acc[a][0] * f, acc[a][1] * f);
      // base-2 log-sum-exp of the row's block-level logits, for the backward (which recomputes abar from it)
      if (lse2 && lane == 0) lse2[(long long)u * g.m + i] = mx[a] + log2f(zz);
    }
  }
}

// ------------------------------------------------------------------------------------------
// combine_kernel: o = g_CG * obar(block of the token) + g_FG * oFG + g_L * oL, eight lanes per token (16 bytes of
// each bf16 tensor per lane), fp32 arithmetic, bf16 result.  HBM-bound: reads 2 * 128 B + 12 B per token (the
// block's obar comes from L2), writes 128 B.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) combine_kernel(Geo g, const float* __restrict__ ocg, const uint4* __restrict__ o_fg,
                                                      const uint4* __restrict__ o_l, const float* __restrict__ gates,
                                                      uint4* __restrict__ o) {
  const long long x = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;  // token over all units
  const int part = threadIdx.x & 7;
  if (x >= (long long)g.U * g.N) return;
  const int u = (int)(x / g.N);
  const long long t = x - (long long)u * g.N;
  const int lat = (int)(t / g.nlon), lon = (int)(t - (long long)lat * g.nlon);
  const int blk = (lat / g.bh) * g.nbw + lon / g.bw;
  const float gc = __ldg(gates + x * 3), gf = __ldg(gates + x * 3 + 1), gl = __ldg(gates + x * 3 + 2);
  const float4* cg = reinterpret_cast<const float4*>(ocg + ((long long)u * g.m + blk) * kD + 8 * part);
  const float4 c0 = __ldg(cg), c1 = __ldg(cg + 1);
  const float cgv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
  const uint4 a = __ldg(o_fg + x * 8 + part), b = __ldg(o_l + x * 8 + part);
  const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
  uint32_t r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a0, a1, b0, b1;
    unpack16x2(av[i], g.f16 != 0, a0, a1);
    unpack16x2(bv[i], g.f16 != 0, b0, b1);
    r[i] = pack16x2(gc * cgv[2 * i] + gf * a0 + gl * b0, gc * cgv[2 * i + 1] + gf * a1 + gl * b1, g.f16 != 0);
  }
  o[x * 8 + part] = make_uint4(r[0], r[1], r[2], r[3]);
}

}  // namespace

int launch_compress(const HostCtx& c, const float* pooled_q, const float* pooled_k, const float* pooled_v, float* ocg,
                    float* lse2) {
  const Geo& g = c.g;
  const size_t smem = sizeof(CompressSmem);
  static unsigned long long configured = 0;  // devices on which the kernel's shared-memory opt-in is set
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 0 || dev >= 64) return MOSAIC_E_UNSUPPORTED;
  if (!((configured >> dev) & 1ull)) {
    if (cudaFuncSetAttribute(compress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return MOSAIC_E_CUDA;
    configured |= 1ull << dev;
  }
  const int tiles = (g.m + kCW * kCR - 1) / (kCW * kCR);
  compress_kernel<<<(unsigned)(g.U * tiles), kCW * 32, smem, c.stream>>>(g, pooled_q, pooled_k, pooled_v, ocg, lse2);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_combine(const HostCtx& c, const float* ocg, const void* o_fg, const void* o_l, const float* gates, void* o) {
  const Geo& g = c.g;
  const long long blocks = ((long long)g.U * g.N * 8 + 255) / 256;
  if (blocks > 0x7fffffffll) return MOSAIC_E_UNSUPPORTED;
  combine_kernel<<<(unsigned)blocks, 256, 0, c.stream>>>(g, ocg, (const uint4*)o_fg, (const uint4*)o_l, gates, (uint4*)o);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

}  // namespace mosaic
