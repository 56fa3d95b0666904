// Backward of the three-branch form: the pieces around the two attention backward passes.
//
// Paper: Eq. of the aggregated output (section "Native Sparse Attention"), o_l = g_CG obar_i + g_FG oFG_l + g_L oL_l,
// and the "Compression" paragraph of the section "Block-Sparse Attention" (obar_i = sum_j abar_ij vbar_j with
// abar = softmax over all m blocks of the mean-pooled queries and keys).  With dO the gradient of o:
//   gates:        dg_X(l) = <dO_l, oX_l>                                   (X = CG, FG, L)
//   attention:    the selection and the local branch are softmax attentions of their own, so each takes the
//                 attention backward with dO scaled by its gate (gate_kernel writes g_FG dO and g_L dO)
//   compression:  dobar_i = sum_{l in block i} g_CG(l) dO_l ;  with delta_i = <dobar_i, obar_i>,
//                 dp_ij = <dobar_i, vbar_j>, ds_ij = abar_ij (dp_ij - delta_i):
//                 dvbar_j = sum_i abar_ij dobar_i,  dqbar_i = scale sum_j ds_ij kbar_j,  dkbar_j = scale sum_i ds_ij qbar_i ;
//                 a mean spreads its gradient evenly: every token of a block receives 1/b of the block's.
//                 This is the only path by which gradient reaches the block-level (routing) scores.
// Everything here is fp32 on the CUDA cores: 4 m^2 d FLOP per unit and sum, far too small for a tensor-core pipeline.
#include <cuda_bf16.h>

#include "common.cuh"

namespace mosaic {

namespace {

__device__ __forceinline__ int token_block(const Geo& g, long long t) {
  const int lat = (int)(t / g.nlon), lon = (int)(t - (long long)lat * g.nlon);
  return (lat / g.bh) * g.nbw + lon / g.bw;
}
__device__ __forceinline__ void unpack8(const Geo& g, const uint4& v, float (&f)[8]) {
  const uint32_t x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) unpack16x2(x[i], g.f16 != 0, f[2 * i], f[2 * i + 1]);
}
__device__ __forceinline__ uint4 pack8(const Geo& g, const float (&f)[8]) {
  uint32_t r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) r[i] = pack16x2(f[2 * i], f[2 * i + 1], g.f16 != 0);
  return make_uint4(r[0], r[1], r[2], r[3]);
}

// ------------------------------------------------------------------------------------------
// gate_kernel: per token the three gate gradients and the gated copies of dO for the two attention branches.
// Eight lanes per token, 16 bytes of each bf16 tensor per lane.  HBM-bound: reads 3 * 128 B + 12 B, writes
// 2 * 128 B + 12 B per token (the block's obar comes from L2).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gate_kernel(Geo g, const uint4* __restrict__ d_o, const uint4* __restrict__ o_fg,
                                                   const uint4* __restrict__ o_l, const float* __restrict__ ocg,
                                                   const float* __restrict__ gates, float* __restrict__ dgates,
                                                   uint4* __restrict__ do_fg, uint4* __restrict__ do_l) {
  const long long x = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;  // token over all units
  const int part = threadIdx.x & 7;
  const bool live = x < (long long)g.U * g.N;  // idle lanes of the last warp still take part in the shuffles
  float dc = 0.f, df = 0.f, dl = 0.f;
  if (live) {
    const int u = (int)(x / g.N);
    const int blk = token_block(g, x - (long long)u * g.N);
    const float gf = __ldg(gates + x * 3 + 1), gl = __ldg(gates + x * 3 + 2);
    const float4* cg = reinterpret_cast<const float4*>(ocg + ((long long)u * g.m + blk) * kD + 8 * part);
    const float4 c0 = __ldg(cg), c1 = __ldg(cg + 1);
    const float cgv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    float go[8], a[8], b[8], sf[8], sl[8];
    unpack8(g, __ldg(d_o + x * 8 + part), go);
    unpack8(g, __ldg(o_fg + x * 8 + part), a);
    unpack8(g, __ldg(o_l + x * 8 + part), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      dc = fmaf(go[i], cgv[i], dc);
      df = fmaf(go[i], a[i], df);
      dl = fmaf(go[i], b[i], dl);
      sf[i] = gf * go[i];
      sl[i] = gl * go[i];
    }
    do_fg[x * 8 + part] = pack8(g, sf);
    do_l[x * 8 + part] = pack8(g, sl);
  }
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) {
    dc += __shfl_xor_sync(0xffffffffu, dc, o);
    df += __shfl_xor_sync(0xffffffffu, df, o);
    dl += __shfl_xor_sync(0xffffffffu, dl, o);
  }
  if (live && part == 0) {
    dgates[x * 3] = dc;
    dgates[x * 3 + 1] = df;
    dgates[x * 3 + 2] = dl;
  }
}

// ------------------------------------------------------------------------------------------
// gated_pool_kernel: dobar_i = sum over the block's tokens (row-major) of g_CG dO, fp32.  Eight lanes per
// (unit, block), eight channels per lane.  HBM-bound: reads dO once.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gated_pool_kernel(Geo g, const uint4* __restrict__ d_o,
                                                         const float* __restrict__ gates, float* __restrict__ dob) {
  const int sub = threadIdx.x & 7;
  const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  if (w >= (long long)g.U * g.m) return;
  const int u = (int)(w / g.m), j = (int)(w - (long long)u * g.m);
  const int by = j / g.nbw, bx = j - by * g.nbw;
  float acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.f;
  for (int r = 0; r < g.bh; ++r) {
    const long long t0 = (long long)u * g.N + (long long)(by * g.bh + r) * g.nlon + bx * g.bw;
    for (int c = 0; c < g.bw; ++c) {
      float go[8];
      unpack8(g, __ldg(d_o + (t0 + c) * 8 + sub), go);
      const float gc = __ldg(gates + (t0 + c) * 3);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = fmaf(gc, go[e], acc[e]);
    }
  }
  float4* dst = reinterpret_cast<float4*>(dob + w * kD + 8 * sub);
  dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
  dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
}

constexpr int kBR = 4;          // stationary blocks per warp
constexpr int kBW = 8;          // warps per CTA
constexpr int kBJ = 64;         // streamed blocks per staged chunk
constexpr int kBStr = kD + 4;   // padded row (floats)

struct CompressBwdSmem {
  float a1[kBW * kBR][kBStr];   // stationary side: pooled query sums (query side) / pooled key sums (key side)
  float a2[kBW * kBR][kBStr];   //                  dobar                       / pooled value sums
  float b1[kBJ][kBStr];         // streamed side:   pooled key sums             / pooled query sums
  float b2[kBJ][kBStr];         //                  pooled value sums           / dobar
  float wa[kBW * kBR][kBJ];     // abar of the chunk
  float wd[kBW * kBR][kBJ];     // ds of the chunk
  float st_lse[kBJ], st_delta[kBJ];  // key side: log-sum-exp (base 2) and delta of the streamed query blocks
};

// ------------------------------------------------------------------------------------------
// compress_bwd_kernel<KEY_SIDE>: the block-level softmax backward, recomputing abar from the saved base-2
// log-sum-exp.  A CTA owns 32 blocks of one unit (4 per warp) and streams the other side in chunks of 64; a lane
// scores streamed blocks lane and lane + 32 for its warp's rows, then owns channels 2 lane, 2 lane + 1 of the sums.
//   query side (KEY_SIDE = false): rows i; writes delta_i and dqm_i = scale / b^2 * sum_j ds_ij ksum_j
//   key side   (KEY_SIDE = true):  rows j of a key/value unit, summed over the query heads of its group;
//                                  writes dkm_j = scale / b^2 * sum_i ds_ij qsum_i and dvm_j = 1/b * sum_i abar_ij dobar_i
// (sums are block SUMS; dqm, dkm, dvm are what every token of the block receives).  Summation order is fixed.
// ------------------------------------------------------------------------------------------
template <bool KEY_SIDE>
__global__ void __launch_bounds__(kBW * 32) compress_bwd_kernel(Geo g, const float* __restrict__ pq,
                                                                const float* __restrict__ pk,
                                                                const float* __restrict__ pv,
                                                                const float* __restrict__ dob,
                                                                const float* __restrict__ ocg,
                                                                const float* __restrict__ lse2, float* __restrict__ delta,
                                                                float* __restrict__ out1, float* __restrict__ out2) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  CompressBwdSmem& sm = *reinterpret_cast<CompressBwdSmem*>(smem_raw);
  constexpr int TI = kBW * kBR, NT = kBW * 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tiles = (g.m + TI - 1) / TI;
  const int u = blockIdx.x / tiles, r0 = (blockIdx.x - u * tiles) * TI;  // u: query unit / key-value unit
  const float inv_b = 1.0f / (float)g.b;
  const float sl2 = g.scale_log2 * inv_b * inv_b;
  const int ratio = g.H / g.Hkv;
  const int ukv = KEY_SIDE ? u : kv_unit(g, u);
  const float* s1 = (KEY_SIDE ? pk : pq) + (long long)u * g.m * kD;
  const float* s2 = (KEY_SIDE ? pv : dob) + (long long)u * g.m * kD;
  for (int e = tid; e < TI * (kD / 4); e += NT) {
    const int r = e / (kD / 4), c4 = e - r * (kD / 4);
    float4 v1 = make_float4(0.f, 0.f, 0.f, 0.f), v2 = v1;
    if (r0 + r < g.m) {
      v1 = __ldg(reinterpret_cast<const float4*>(s1 + (long long)(r0 + r) * kD + 4 * c4));
      v2 = __ldg(reinterpret_cast<const float4*>(s2 + (long long)(r0 + r) * kD + 4 * c4));
    }
    *reinterpret_cast<float4*>(&sm.a1[r][4 * c4]) = v1;
    *reinterpret_cast<float4*>(&sm.a2[r][4 * c4]) = v2;
  }
  // query side: the rows' own log-sum-exp and delta_i = <dobar_i, obar_i> (lanes split the channels)
  float row_lse[kBR], row_delta[kBR];
#pragma unroll
  for (int a = 0; a < kBR; ++a) { row_lse[a] = 0.f; row_delta[a] = 0.f; }
  if (!KEY_SIDE) {
#pragma unroll
    for (int a = 0; a < kBR; ++a) {
      const int i = r0 + warp * kBR + a;
      float dd = 0.f;
      if (i < g.m) {
        const float2 x = __ldg(reinterpret_cast<const float2*>(dob + ((long long)u * g.m + i) * kD + 2 * lane));
        const float2 y = __ldg(reinterpret_cast<const float2*>(ocg + ((long long)u * g.m + i) * kD + 2 * lane));
        dd = fmaf(x.x, y.x, x.y * y.y);
        row_lse[a] = __ldg(lse2 + (long long)u * g.m + i);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dd += __shfl_xor_sync(0xffffffffu, dd, o);
      row_delta[a] = dd;
      if (i < g.m && lane == 0) delta[(long long)u * g.m + i] = dd;
    }
  }
  float acc1[kBR][2], acc2[kBR][2];
#pragma unroll
  for (int a = 0; a < kBR; ++a) { acc1[a][0] = acc1[a][1] = acc2[a][0] = acc2[a][1] = 0.f; }

  const int passes = KEY_SIDE ? ratio : 1;
  for (int pass = 0; pass < passes; ++pass) {
    // the streamed side: the keys and values of the row unit's group (query side) / one query head of the group (key side)
    const int us = KEY_SIDE ? (u / g.Hkv) * g.H + (u - (u / g.Hkv) * g.Hkv) * ratio + pass : ukv;
    const float* t1 = (KEY_SIDE ? pq : pk) + (long long)us * g.m * kD;
    const float* t2 = (KEY_SIDE ? dob : pv) + (long long)us * g.m * kD;
    for (int j0 = 0; j0 < g.m; j0 += kBJ) {
      __syncthreads();  // the previous chunk is consumed (and the stationary rows are written on the first pass)
      for (int e = tid; e < kBJ * (kD / 4); e += NT) {
        const int jj = e / (kD / 4), c4 = e - jj * (kD / 4);
        float4 v1 = make_float4(0.f, 0.f, 0.f, 0.f), v2 = v1;
        if (j0 + jj < g.m) {
          v1 = __ldg(reinterpret_cast<const float4*>(t1 + (long long)(j0 + jj) * kD + 4 * c4));
          v2 = __ldg(reinterpret_cast<const float4*>(t2 + (long long)(j0 + jj) * kD + 4 * c4));
        }
        *reinterpret_cast<float4*>(&sm.b1[jj][4 * c4]) = v1;
        *reinterpret_cast<float4*>(&sm.b2[jj][4 * c4]) = v2;
      }
      if (KEY_SIDE && tid < kBJ) {
        const bool in = j0 + tid < g.m;
        sm.st_lse[tid] = in ? __ldg(lse2 + (long long)us * g.m + j0 + tid) : 0.f;
        sm.st_delta[tid] = in ? __ldg(delta + (long long)us * g.m + j0 + tid) : 0.f;
      }
      __syncthreads();
      float s[kBR][2], dp[kBR][2];
#pragma unroll
      for (int a = 0; a < kBR; ++a) { s[a][0] = s[a][1] = dp[a][0] = dp[a][1] = 0.f; }
#pragma unroll 2
      for (int c4 = 0; c4 < kD / 4; ++c4) {
        const float4 k0 = *reinterpret_cast<const float4*>(&sm.b1[lane][4 * c4]);
        const float4 k1 = *reinterpret_cast<const float4*>(&sm.b1[lane + 32][4 * c4]);
        const float4 v0 = *reinterpret_cast<const float4*>(&sm.b2[lane][4 * c4]);
        const float4 v1 = *reinterpret_cast<const float4*>(&sm.b2[lane + 32][4 * c4]);
#pragma unroll
        for (int a = 0; a < kBR; ++a) {
          const float4 x = *reinterpret_cast<const float4*>(&sm.a1[warp * kBR + a][4 * c4]);
          const float4 y = *reinterpret_cast<const float4*>(&sm.a2[warp * kBR + a][4 * c4]);
          s[a][0] = fmaf(x.x, k0.x, fmaf(x.y, k0.y, fmaf(x.z, k0.z, fmaf(x.w, k0.w, s[a][0]))));
          s[a][1] = fmaf(x.x, k1.x, fmaf(x.y, k1.y, fmaf(x.z, k1.z, fmaf(x.w, k1.w, s[a][1]))));
          dp[a][0] = fmaf(y.x, v0.x, fmaf(y.y, v0.y, fmaf(y.z, v0.z, fmaf(y.w, v0.w, dp[a][0]))));
          dp[a][1] = fmaf(y.x, v1.x, fmaf(y.y, v1.y, fmaf(y.z, v1.z, fmaf(y.w, v1.w, dp[a][1]))));
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int jj = lane + 32 * h;
        const bool in = j0 + jj < g.m;
        const float l_s = KEY_SIDE ? sm.st_lse[jj] : 0.f, d_s = KEY_SIDE ? sm.st_delta[jj] : 0.f;
#pragma unroll
        for (int a = 0; a < kBR; ++a) {
          const bool row_in = r0 + warp * kBR + a < g.m;
          const float lse_q = KEY_SIDE ? l_s : row_lse[a], del_q = KEY_SIDE ? d_s : row_delta[a];
          const float ab = (in && row_in) ? exp2f(s[a][h] * sl2 - lse_q) : 0.f;
          sm.wa[warp * kBR + a][jj] = ab;
          sm.wd[warp * kBR + a][jj] = ab * (dp[a][h] * inv_b - del_q);
        }
      }
      __syncwarp();
      const int nj = min(kBJ, g.m - j0);
      for (int jj = 0; jj < nj; ++jj) {
        const float2 x1 = *reinterpret_cast<const float2*>(&sm.b1[jj][2 * lane]);
        const float2 x2 = *reinterpret_cast<const float2*>(&sm.b2[jj][2 * lane]);
#pragma unroll
        for (int a = 0; a < kBR; ++a) {
          const float wd = sm.wd[warp * kBR + a][jj];
          acc1[a][0] = fmaf(wd, x1.x, acc1[a][0]);
          acc1[a][1] = fmaf(wd, x1.y, acc1[a][1]);
          if (KEY_SIDE) {
            const float wa = sm.wa[warp * kBR + a][jj];
            acc2[a][0] = fmaf(wa, x2.x, acc2[a][0]);
            acc2[a][1] = fmaf(wa, x2.y, acc2[a][1]);
          }
        }
      }
    }
  }
  const float f1 = g.scale * inv_b * inv_b;
#pragma unroll
  for (int a = 0; a < kBR; ++a) {
    const int r = r0 + warp * kBR + a;
    if (r < g.m) {
      const long long at = ((long long)u * g.m + r) * kD + 2 * lane;
      *reinterpret_cast<float2*>(out1 + at) = make_float2(acc1[a][0] * f1, acc1[a][1] * f1);
      if (KEY_SIDE) *reinterpret_cast<float2*>(out2 + at) = make_float2(acc2[a][0] * inv_b, acc2[a][1] * inv_b);
    }
  }
}

// ------------------------------------------------------------------------------------------
// sum_kernel: x = bf16(x_L + x_FG + xm[block of the token]) for one gradient tensor: the two attention branches'
// gradients (bf16) plus what the compression branch gives every token of the block (fp32).  Eight lanes per
// token.  HBM-bound: reads 2 * 128 B, writes 128 B per token.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) sum_kernel(Geo g, long long tokens, const uint4* __restrict__ x_l,
                                                  const uint4* __restrict__ x_fg, const float* __restrict__ xm,
                                                  uint4* __restrict__ out) {
  const long long x = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  const int part = threadIdx.x & 7;
  if (x >= tokens) return;
  const long long u = x / g.N;
  const int blk = token_block(g, x - u * g.N);
  const float4* cm = reinterpret_cast<const float4*>(xm + (u * g.m + blk) * kD + 8 * part);
  const float4 c0 = __ldg(cm), c1 = __ldg(cm + 1);
  const float cv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
  float a[8], b[8], r[8];
  unpack8(g, __ldg(x_l + x * 8 + part), a);
  if (x_fg) unpack8(g, __ldg(x_fg + x * 8 + part), b);
#pragma unroll
  for (int i = 0; i < 8; ++i) r[i] = a[i] + (x_fg ? b[i] : 0.f) + cv[i];
  out[x * 8 + part] = pack8(g, r);
}

}  // namespace

int launch_gate(const HostCtx& c, const void* d_o, const void* o_fg, const void* o_l, const float* ocg,
                const float* gates, float* dgates, void* do_fg, void* do_l, float* dob) {
  const Geo& g = c.g;
  const long long blocks = ((long long)g.U * g.N * 8 + 255) / 256;
  if (blocks > 0x7fffffffll) return MOSAIC_E_UNSUPPORTED;
  gate_kernel<<<(unsigned)blocks, 256, 0, c.stream>>>(g, (const uint4*)d_o, (const uint4*)o_fg, (const uint4*)o_l, ocg,
                                                      gates, dgates, (uint4*)do_fg, (uint4*)do_l);
  if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  const long long pblocks = ((long long)g.U * g.m * 8 + 255) / 256;
  gated_pool_kernel<<<(unsigned)pblocks, 256, 0, c.stream>>>(g, (const uint4*)d_o, gates, dob);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_compress_bwd(const HostCtx& c, const float* pq, const float* pk, const float* pv, const float* dob,
                        const float* ocg, const float* lse2, float* delta, float* dqm, float* dkm, float* dvm) {
  const Geo& g = c.g;
  const size_t smem = sizeof(CompressBwdSmem);
  static unsigned long long configured = 0;  // devices on which the kernels' shared-memory opt-in is set
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 0 || dev >= 64) return MOSAIC_E_UNSUPPORTED;
  if (!((configured >> dev) & 1ull)) {
    if (cudaFuncSetAttribute(compress_bwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(compress_bwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return MOSAIC_E_CUDA;
    configured |= 1ull << dev;
  }
  const int tiles = (g.m + kBW * kBR - 1) / (kBW * kBR);
  compress_bwd_kernel<false><<<(unsigned)(g.U * tiles), kBW * 32, smem, c.stream>>>(g, pq, pk, pv, dob, ocg, lse2, delta,
                                                                                   dqm, nullptr);
  if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  compress_bwd_kernel<true><<<(unsigned)(g.Ukv * tiles), kBW * 32, smem, c.stream>>>(g, pq, pk, pv, dob, ocg, lse2, delta,
                                                                                    dkm, dvm);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_grad_sum(const HostCtx& c, int units, const void* x_l, const void* x_fg, const float* xm, void* out) {
  const Geo& g = c.g;
  const long long tokens = (long long)units * g.N;
  const long long blocks = (tokens * 8 + 255) / 256;
  if (blocks > 0x7fffffffll) return MOSAIC_E_UNSUPPORTED;
  sum_kernel<<<(unsigned)blocks, 256, 0, c.stream>>>(g, tokens, (const uint4*)x_l, (const uint4*)x_fg, xm, (uint4*)out);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

}  // namespace mosaic
