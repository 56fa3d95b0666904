// Selection: block pooling, block-level scores, per-query-block top-k.
//
// Paper, section "Block-Sparse Attention": paragraph "Compression" defines the pooled block
// representations (phi = mean pooling) and the block-level score; paragraph "Selection" takes the
// top-n key blocks per query block.  The mean's 1/b, the 1/sqrt(d_k) and the row softmax are
// strictly increasing, so ranking the raw dot product of block SUMS gives the same blocks.
//
// Arithmetic is fixed so that the chosen ids are unique and reproducible bit for bit:
//   pooled sum  = fp64 accumulation over the block's tokens in row-major order, one rounding to fp32
//   score       = fp64 accumulation over channels 0..d-1 of the exact products of two fp32 values
//   order       = (score descending, block id ascending); +0 == -0; a NaN ranks last
#include "common.cuh"

namespace mosaic {

// ------------------------------------------------------------------------------------------
// pool_kernel: one warp per (tensor, unit, block); lane owns channels 2*lane, 2*lane+1.
// HBM-bound: reads 2*U*N*d*2 bytes once, every warp request is one full 128-byte line.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pool_kernel(Geo g, const uint32_t* __restrict__ q,
                                                   const uint32_t* __restrict__ k, float* __restrict__ pq,
                                                   float* __restrict__ pk) {
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long per_tensor = (long long)g.U * g.m;
  if (warp >= 2 * per_tensor) return;
  const int which = warp >= per_tensor;
  const long long w = warp - which * per_tensor;
  const int u = (int)(w / g.m), j = (int)(w - (long long)u * g.m);
  const uint32_t* src = (which ? k : q) + (long long)u * g.N * (kD / 2) + lane;
  const int by = j / g.nbw, bx = j - by * g.nbw;
  double a0 = 0.0, a1 = 0.0;
  for (int r = 0; r < g.bh; ++r) {
    const uint32_t* row = src + ((long long)(by * g.bh + r) * g.nlon + bx * g.bw) * (kD / 2);
    // bw is 8 or 16: issue the row's loads together, then add in token order
    uint32_t v[16];
#pragma unroll
    for (int c = 0; c < 16; ++c)
      if (c < g.bw) v[c] = __ldg(row + c * (kD / 2));
#pragma unroll
    for (int c = 0; c < 16; ++c)
      if (c < g.bw) {
        a0 += (double)__uint_as_float(v[c] << 16);
        a1 += (double)__uint_as_float(v[c] & 0xffff0000u);
      }
  }
  float* dst = (which ? pk : pq) + ((long long)u * g.m + j) * kD + 2 * lane;
  *reinterpret_cast<float2*>(dst) = make_float2((float)a0, (float)a1);
}

// ------------------------------------------------------------------------------------------
// topk_kernel: a CTA owns TQ query blocks of one unit and streams the pooled keys in chunks
// of JC blocks through shared memory.  Thread t scores key block (chunk*JC + t) against the
// TQ pooled queries (fp64 FMA chain over channels); then one warp per query row merges the
// chunk into a sorted k-entry list held one entry per lane.
// ------------------------------------------------------------------------------------------
constexpr int TQ = 16;
constexpr int JC = 256;
constexpr int KPAD = kD + 1;

// Total-order key: larger key = better score.  0 = not a candidate, 1 = NaN.
__device__ __forceinline__ unsigned long long score_key(double s) {
  if (s != s) return 1ull;
  s += 0.0;  // -0 -> +0
  unsigned long long b = (unsigned long long)__double_as_longlong(s);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

// does (ka, ia) rank before (kb, ib)?
__device__ __forceinline__ bool ranks_before(unsigned long long ka, int ia, unsigned long long kb, int ib) {
  return ka > kb || (ka == kb && ia < ib);
}

__global__ void __launch_bounds__(JC) topk_kernel(Geo g, const float* __restrict__ pq,
                                                  const float* __restrict__ pk, int32_t* __restrict__ block_idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* qs = reinterpret_cast<double*>(smem_raw);                         // [TQ][kD]
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(qs + TQ * kD);  // [TQ][JC]
  float* ks = reinterpret_cast<float*>(keys + TQ * JC);                     // [JC][KPAD]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tiles = (g.m + TQ - 1) / TQ;
  const int u = blockIdx.x / tiles, i0 = (blockIdx.x - u * tiles) * TQ;
  const float* pq_u = pq + (long long)u * g.m * kD;
  const float* pk_u = pk + (long long)u * g.m * kD;

  for (int e = tid; e < TQ * kD; e += JC) {
    int r = e / kD, i = i0 + r;
    qs[e] = i < g.m ? (double)pq_u[(long long)i * kD + (e - r * kD)] : 0.0;
  }

  // sorted list of the best candidates so far: entry `lane` of each row this warp owns
  constexpr int RPW = TQ / (JC / 32);  // rows per warp
  unsigned long long lkey[RPW];
  int lid[RPW];
#pragma unroll
  for (int r = 0; r < RPW; ++r) { lkey[r] = 0ull; lid[r] = -1; }

  for (int j0 = 0; j0 < g.m; j0 += JC) {
    __syncthreads();  // previous chunk fully merged (and qs written on the first pass)
    const int nj = min(JC, g.m - j0);
    for (int e = tid; e < nj * kD; e += JC) {
      int jj = e / kD;
      ks[jj * KPAD + (e - jj * kD)] = pk_u[(long long)j0 * kD + e];
    }
    __syncthreads();
    {
      const int j = j0 + tid;
      double acc[TQ];
#pragma unroll
      for (int r = 0; r < TQ; ++r) acc[r] = 0.0;
      if (tid < nj) {
        for (int c = 0; c < kD; ++c) {
          const double kc = (double)ks[tid * KPAD + c];
#pragma unroll
          for (int r = 0; r < TQ; ++r) acc[r] = fma(qs[r * kD + c], kc, acc[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < TQ; ++r) {
        const int i = i0 + r;
        const bool cand = tid < nj && i < g.m && !is_local(g, i, j);
        keys[r * JC + tid] = cand ? score_key(acc[r]) : 0ull;
      }
    }
    __syncthreads();
    // merge: repeatedly take the best remaining chunk entry while it still enters the list
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) {
      const int r = warp * RPW + rr;
      unsigned long long* row = keys + r * JC;
      for (int round = 0; round < g.topk; ++round) {
        unsigned long long bk = 0ull;
        int bj = 0x7fffffff;
#pragma unroll
        for (int s = 0; s < JC / 32; ++s) {
          unsigned long long kk = row[lane + 32 * s];
          int jj = j0 + lane + 32 * s;
          if (kk != 0ull && ranks_before(kk, jj, bk, bj)) { bk = kk; bj = jj; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          unsigned long long ok = __shfl_xor_sync(0xffffffffu, bk, o);
          int oj = __shfl_xor_sync(0xffffffffu, bj, o);
          if (ok != 0ull && ranks_before(ok, oj, bk, bj)) { bk = ok; bj = oj; }
        }
        if (bk == 0ull) break;  // chunk exhausted
        // list is sorted best-first; its last wanted entry sits in lane topk-1
        unsigned long long tk = __shfl_sync(0xffffffffu, lkey[rr], g.topk - 1);
        int ti = __shfl_sync(0xffffffffu, lid[rr], g.topk - 1);
        if (tk != 0ull && !ranks_before(bk, bj, tk, ti)) break;  // nothing left that enters
        // insert at position p = number of entries ranking before the new one
        bool before = lkey[rr] != 0ull && ranks_before(lkey[rr], lid[rr], bk, bj);
        int p = __popc(__ballot_sync(0xffffffffu, before));
        unsigned long long uk = __shfl_up_sync(0xffffffffu, lkey[rr], 1);
        int ui = __shfl_up_sync(0xffffffffu, lid[rr], 1);
        if (lane == p) { lkey[rr] = bk; lid[rr] = bj; }
        else if (lane > p) { lkey[rr] = uk; lid[rr] = ui; }
        if (lane == ((bj - j0) & 31)) row[bj - j0] = 0ull;  // taken
        __syncwarp();
      }
    }
  }
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr) {
    const int i = i0 + warp * RPW + rr;
    if (i < g.m && lane < g.topk)
      block_idx[((long long)u * g.m + i) * g.topk + lane] = lkey[rr] != 0ull ? lid[rr] : -1;
  }
}

int launch_select(const HostCtx& c, const void* q, const void* k, int32_t* block_idx, float* pooled_q,
                  float* pooled_k) {
  const Geo& g = c.g;
  {
    long long warps = 2ll * g.U * g.m;
    int wpb = 8;
    long long blocks = (warps + wpb - 1) / wpb;
    pool_kernel<<<(unsigned)blocks, wpb * 32, 0, c.stream>>>(g, (const uint32_t*)q, (const uint32_t*)k,
                                                             pooled_q, pooled_k);
    if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  }
  if (g.topk > 0) {
    size_t smem = sizeof(double) * TQ * kD + sizeof(unsigned long long) * TQ * JC + sizeof(float) * JC * KPAD;
    static bool attr_set = false;
    if (!attr_set) {
      if (cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return MOSAIC_E_CUDA;
      attr_set = true;
    }
    int tiles = (g.m + TQ - 1) / TQ;
    topk_kernel<<<(unsigned)(g.U * tiles), JC, smem, c.stream>>>(g, pooled_q, pooled_k, block_idx);
    if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  }
  return MOSAIC_OK;
}

}  // namespace mosaic
