// Two-dimensional rotary position embedding of Q and K.
//
// Paper, "Overall architecture" paragraph: RoPE on queries and keys encodes longitude and latitude; the head
// dimension is split equally between the two coordinates and each half receives a standard RoPE of its angle in
// radians (architecture table of the appendix: theta = 10000).  Channels [0, d/2) belong to the longitude,
// [d/2, d) to the latitude; inside a half of width D = d/2 the pair (2i, 2i+1) turns by pos * theta^(-2i/D).
//
// HBM-bound: every element of Q and K is read and written once.  Eight lanes per token, a lane owns eight channels
// (four pairs, 16 bytes) and walks all units of both tensors with the same four (cos, sin), which it computes once
// in fp64; the rotation is fp64 too (a few fp64 FMAs per 16 bytes moved), rounded to fp32 and then to the storage type.
#include <cuda_bf16.h>

#include "common.cuh"

namespace mosaic {

namespace {

__device__ __forceinline__ uint4 rotate8(const uint4& v, const double (&c)[4], const double (&s)[4], bool f16) {
  const uint32_t x[4] = {v.x, v.y, v.z, v.w};
  uint32_t r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float lo, hi;
    unpack16x2(x[i], f16, lo, hi);
    const double x0 = (double)lo, x1 = (double)hi;
    const float y0 = __double2float_rn(x0 * c[i] - x1 * s[i]), y1 = __double2float_rn(x0 * s[i] + x1 * c[i]);
    r[i] = pack16x2(y0, y1, f16);
  }
  return make_uint4(r[0], r[1], r[2], r[3]);
}

__global__ void __launch_bounds__(256) rope_kernel(Geo g, const uint4* __restrict__ q, const uint4* __restrict__ k,
                                                   const float* __restrict__ pos, double theta,
                                                   uint4* __restrict__ q_out, uint4* __restrict__ k_out) {
  const long long x = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;  // token of the grid
  const int part = threadIdx.x & 7;
  if (x >= g.N) return;
  const double p = (double)__ldg(pos + 2 * x + (part >> 2));  // longitude for channels 0..31, latitude for 32..63
  double c[4], s[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int i = 4 * (part & 3) + j;                         // pair inside the half, D = kD / 2
    sincos(p * pow(theta, -2.0 * i / (kD / 2)), &s[j], &c[j]);
  }
#pragma unroll 4
  for (int u = 0; u < g.U; ++u) {
    const long long at = ((long long)u * g.N + x) * 8 + part;
    q_out[at] = rotate8(__ldg(q + at), c, s, g.f16 != 0);
  }
#pragma unroll 4
  for (int u = 0; u < g.Ukv; ++u) {
    const long long at = ((long long)u * g.N + x) * 8 + part;
    k_out[at] = rotate8(__ldg(k + at), c, s, g.f16 != 0);
  }
}

}  // namespace

int launch_rope(const HostCtx& c, const void* q, const void* k, const float* pos, double theta, void* q_out, void* k_out) {
  const Geo& g = c.g;
  const long long blocks = (g.N * 8 + 255) / 256;
  if (blocks > 0x7fffffffll) return MOSAIC_E_UNSUPPORTED;
  rope_kernel<<<(unsigned)blocks, 256, 0, c.stream>>>(g, (const uint4*)q, (const uint4*)k, pos, theta, (uint4*)q_out,
                                                      (uint4*)k_out);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

}  // namespace mosaic
