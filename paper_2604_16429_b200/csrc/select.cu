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
// pool_kernel: eight lanes per (tensor, unit, block), four blocks per warp; a lane owns eight
// consecutive channels (one 16-byte load per token) and adds them in token order, row-major inside
// the block, so every channel is one sequential fp64 chain.  HBM-bound: reads 2*U*N*d*2 bytes once;
// the loads of a whole block row are in flight together.
// ------------------------------------------------------------------------------------------
template <int BW>
__global__ void __launch_bounds__(256) pool_kernel(Geo g, const uint4* __restrict__ q, const uint4* __restrict__ k,
                                                   float* __restrict__ pq, float* __restrict__ pk) {
  const int sub = threadIdx.x & 7;  // which 8 channels
  const long long grp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  const long long per_tensor = (long long)g.U * g.m;
  if (grp >= 2 * per_tensor) return;
  const int which = grp >= per_tensor;
  const long long w = grp - which * per_tensor;
  const int u = (int)(w / g.m), j = (int)(w - (long long)u * g.m);
  const uint4* src = (which ? k : q) + (long long)u * g.N * (kD / 8) + sub;
  const int by = j / g.nbw, bx = j - by * g.nbw;
  double acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.0;
  for (int r = 0; r < g.bh; ++r) {
    const uint4* row = src + ((long long)(by * g.bh + r) * g.nlon + bx * BW) * (kD / 8);
    uint4 v[BW];
#pragma unroll
    for (int c = 0; c < BW; ++c) v[c] = __ldg(row + c * (kD / 8));
#pragma unroll
    for (int c = 0; c < BW; ++c) {
      const uint32_t x[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        acc[2 * e] += (double)__uint_as_float(x[e] << 16);
        acc[2 * e + 1] += (double)__uint_as_float(x[e] & 0xffff0000u);
      }
    }
  }
  float4* dst = reinterpret_cast<float4*>((which ? pk : pq) + ((long long)u * g.m + j) * kD + 8 * sub);
  dst[0] = make_float4((float)acc[0], (float)acc[1], (float)acc[2], (float)acc[3]);
  dst[1] = make_float4((float)acc[4], (float)acc[5], (float)acc[6], (float)acc[7]);
}

// ------------------------------------------------------------------------------------------
// topk_kernel<TI>: a CTA owns TI query blocks of one unit and streams the pooled keys in chunks of
// JT blocks through shared memory (as fp64, channel-major).  The TI x JT scores of a chunk are a
// register-tiled fp64 product: thread (ty, tx) holds the scores of rows ty + 16a and keys tx + 16b
// and runs one FMA chain over channels 0..d-1 per score, so each score is the sequential sum the
// selection is defined by.  Scores become sortable keys; a key that cannot enter its row's list
// (worse than the row's current k-th best) is dropped at once.
// Merge: one warp per query row keeps the sorted k-entry list, one entry per lane; the rows of a warp
// advance in lockstep so that their reductions overlap.
// ------------------------------------------------------------------------------------------

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

template <int TI, int JT>
struct TopkSmem {
  static constexpr int KSTR = JT + 1;  // padded row of the key tile: conflict-free transposing stores
  double qs[kD][TI];                   // pooled queries of this CTA, channel-major
  double ks[kD][KSTR];                 // pooled keys of the current chunk, channel-major
  unsigned long long keys[TI][JT];     // candidate keys of the current chunk (0 = none)
  unsigned long long thr[TI];          // key of the row's current k-th best (0 while the list is short)
  int flag[TI];                        // the row has a candidate in this chunk
  short iy[TI], ix[TI], jy[JT], jx[JT];  // block coordinates of the rows and of the chunk's keys
};

template <int TI, int JT>
__global__ void __launch_bounds__(256) topk_kernel(Geo g, const float* __restrict__ pq,
                                                   const float* __restrict__ pk, int32_t* __restrict__ block_idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TopkSmem<TI, JT>& sm = *reinterpret_cast<TopkSmem<TI, JT>*>(smem_raw);
  constexpr int RJ = JT / 16;                 // keys per thread
  constexpr int RI = TI / 16;                 // query rows per thread
  constexpr int RPW = TI / 8;                 // query rows per warp in the merge

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tx = tid & 15, ty = tid >> 4;
  const int tiles = (g.m + TI - 1) / TI;
  const int u = blockIdx.x / tiles, i0 = (blockIdx.x - u * tiles) * TI;
  const float* pq_u = pq + (long long)u * g.m * kD;
  const float* pk_u = pk + (long long)u * g.m * kD;

  for (int e = tid; e < TI * kD; e += 256) {
    const int r = e / kD, c = e - r * kD, i = i0 + r;
    sm.qs[c][r] = i < g.m ? (double)pq_u[(long long)i * kD + c] : 0.0;
  }
  for (int r = tid; r < TI; r += 256) {
    const int i = min(i0 + r, g.m - 1);
    sm.thr[r] = 0ull;
    sm.iy[r] = (short)(i / g.nbw);
    sm.ix[r] = (short)(i - (i / g.nbw) * g.nbw);
  }

  // sorted list of the best candidates so far: entry `lane` of each row this warp owns
  unsigned long long lkey[RPW];
  int lid[RPW];
#pragma unroll
  for (int r = 0; r < RPW; ++r) { lkey[r] = 0ull; lid[r] = -1; }

  for (int j0 = 0; j0 < g.m; j0 += JT) {
    __syncthreads();  // previous chunk fully merged (and qs, thr written on the first pass)
    const int nj = min(JT, g.m - j0);
#pragma unroll
    for (int e = tid; e < JT * kD / 4; e += 256) {
      const int jj = e / (kD / 4), c4 = (e - jj * (kD / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (jj < nj) v = __ldg(reinterpret_cast<const float4*>(pk_u + (long long)(j0 + jj) * kD + c4));
      sm.ks[c4][jj] = (double)v.x;
      sm.ks[c4 + 1][jj] = (double)v.y;
      sm.ks[c4 + 2][jj] = (double)v.z;
      sm.ks[c4 + 3][jj] = (double)v.w;
    }
    if (tid < JT) {
      const int j = min(j0 + tid, g.m - 1);
      sm.jy[tid] = (short)(j / g.nbw);
      sm.jx[tid] = (short)(j - (j / g.nbw) * g.nbw);
    }
    for (int r = tid; r < TI; r += 256) sm.flag[r] = 0;
    __syncthreads();
    {
      double acc[RI][RJ];
#pragma unroll
      for (int a = 0; a < RI; ++a)
#pragma unroll
        for (int b = 0; b < RJ; ++b) acc[a][b] = 0.0;
#pragma unroll 8
      for (int c = 0; c < kD; ++c) {
        double qv[RI], kv[RJ];
#pragma unroll
        for (int a = 0; a < RI; ++a) qv[a] = sm.qs[c][ty + 16 * a];
#pragma unroll
        for (int b = 0; b < RJ; ++b) kv[b] = sm.ks[c][tx + 16 * b];
#pragma unroll
        for (int a = 0; a < RI; ++a)
#pragma unroll
          for (int b = 0; b < RJ; ++b) acc[a][b] = fma(qv[a], kv[b], acc[a][b]);
      }
#pragma unroll
      for (int a = 0; a < RI; ++a) {
        const int r = ty + 16 * a, i = i0 + r;
        const unsigned long long th = sm.thr[r];
        const int iy = sm.iy[r], ix = sm.ix[r];
        bool any = false;
#pragma unroll
        for (int b = 0; b < RJ; ++b) {
          const int jj = tx + 16 * b;
          int dx = sm.jx[jj] - ix;
          dx += dx < 0 ? g.nbw : 0;  // (jx - ix) mod nbw
          const bool local = abs(sm.jy[jj] - iy) <= g.rlat && (dx <= g.rlon || g.nbw - dx <= g.rlon);
          unsigned long long key = 0ull;
          if (jj < nj && i < g.m && !local) {
            key = score_key(acc[a][b]);
            if (key < th) key = 0ull;  // cannot enter the list (an equal key may: lower id wins)
          }
          sm.keys[r][jj] = key;
          any |= key != 0ull;
        }
        if (any) sm.flag[r] = 1;
      }
    }
    __syncthreads();
    // merge, all rows of this warp in lockstep: repeatedly take each row's best remaining chunk entry
    // while it still enters the row's list
    unsigned live = 0;
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) live |= (sm.flag[warp * RPW + rr] ? 1u : 0u) << rr;
    for (int round = 0; round < g.topk && live; ++round) {
      unsigned long long bk[RPW];
      int bj[RPW];
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        bk[rr] = 0ull;
        bj[rr] = 0x7fffffff;
        if ((live >> rr) & 1) {
          const unsigned long long* row = sm.keys[warp * RPW + rr];
#pragma unroll
          for (int s = 0; s < JT / 32; ++s) {
            const unsigned long long kk = row[lane + 32 * s];
            const int jj = j0 + lane + 32 * s;
            if (kk != 0ull && ranks_before(kk, jj, bk[rr], bj[rr])) { bk[rr] = kk; bj[rr] = jj; }
          }
        }
      }
      // warp-wide best of each row: maximum of the key's high word, then of the low word among the
      // lanes that hold that high word, then the lowest block id among the lanes that hold the key
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        if (!((live >> rr) & 1)) continue;  // warp-uniform
        const unsigned hi = (unsigned)(bk[rr] >> 32), lo = (unsigned)bk[rr];
        const unsigned mh = __reduce_max_sync(0xffffffffu, hi);
        const unsigned ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
        const bool mine = bk[rr] != 0ull && hi == mh && lo == ml;
        bj[rr] = __reduce_min_sync(0xffffffffu, mine ? bj[rr] : 0x7fffffff);
        bk[rr] = ((unsigned long long)mh << 32) | ml;
      }
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        // list is sorted best-first; its last wanted entry sits in lane topk-1
        if (!((live >> rr) & 1)) continue;
        const unsigned long long tk = __shfl_sync(0xffffffffu, lkey[rr], g.topk - 1);
        const int ti = __shfl_sync(0xffffffffu, lid[rr], g.topk - 1);
        const bool enters = bk[rr] != 0ull && (tk == 0ull || ranks_before(bk[rr], bj[rr], tk, ti));
        if (!enters) { live &= ~(1u << rr); continue; }  // chunk exhausted for this row
        // insert at position p = number of entries ranking before the new one
        const bool before = lkey[rr] != 0ull && ranks_before(lkey[rr], lid[rr], bk[rr], bj[rr]);
        const int p = __popc(__ballot_sync(0xffffffffu, before));
        const unsigned long long uk = __shfl_up_sync(0xffffffffu, lkey[rr], 1);
        const int ui = __shfl_up_sync(0xffffffffu, lid[rr], 1);
        if (lane == p) { lkey[rr] = bk[rr]; lid[rr] = bj[rr]; }
        else if (lane > p) { lkey[rr] = uk; lid[rr] = ui; }
        if (lane == ((bj[rr] - j0) & 31)) sm.keys[warp * RPW + rr][bj[rr] - j0] = 0ull;  // taken
      }
      __syncwarp();
    }
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) {
      const unsigned long long tk = __shfl_sync(0xffffffffu, lkey[rr], g.topk - 1);
      if (lane == 0) sm.thr[warp * RPW + rr] = tk;  // 0 until the list holds topk entries
    }
  }
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr) {
    const int i = i0 + warp * RPW + rr;
    if (i < g.m && lane < g.topk)
      block_idx[((long long)u * g.m + i) * g.topk + lane] = lkey[rr] != 0ull ? lid[rr] : -1;
  }
}

template <int TI, int JT>
int launch_topk(const HostCtx& c, const float* pooled_q, const float* pooled_k, int32_t* block_idx) {
  const Geo& g = c.g;
  const size_t smem = sizeof(TopkSmem<TI, JT>);
  if (cudaFuncSetAttribute(topk_kernel<TI, JT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return MOSAIC_E_CUDA;
  const int tiles = (g.m + TI - 1) / TI;
  topk_kernel<TI, JT><<<(unsigned)(g.U * tiles), 256, smem, c.stream>>>(g, pooled_q, pooled_k, block_idx);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_select(const HostCtx& c, const void* q, const void* k, int32_t* block_idx, float* pooled_q,
                  float* pooled_k) {
  const Geo& g = c.g;
  {
    const long long threads = 2ll * g.U * g.m * 8;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    if (g.bw == 8)
      pool_kernel<8><<<blocks, 256, 0, c.stream>>>(g, (const uint4*)q, (const uint4*)k, pooled_q, pooled_k);
    else
      pool_kernel<16><<<blocks, 256, 0, c.stream>>>(g, (const uint4*)q, (const uint4*)k, pooled_q, pooled_k);
    if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  }
  if (g.topk > 0) {
    // the most query blocks per CTA (64, 32, 16) that still gives every SM two CTAs; 16 otherwise
    auto ctas = [&](int ti) { return (long long)g.U * ((g.m + ti - 1) / ti); };
    // small problems (16 rows per CTA) take keys in chunks of 128 to halve the number of merge passes
    const int rc = ctas(64) >= 296 ? launch_topk<64, 64>(c, pooled_q, pooled_k, block_idx)
                 : ctas(32) >= 296 ? launch_topk<32, 64>(c, pooled_q, pooled_k, block_idx)
                                   : launch_topk<16, 128>(c, pooled_q, pooled_k, block_idx);
    if (rc) return rc;
  }
  return MOSAIC_OK;
}

}  // namespace mosaic
