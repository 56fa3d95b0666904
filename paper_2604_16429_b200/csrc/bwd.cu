// Backward of the block-sparse attention (selection held constant).
//
// Paper, appendix "Block-sparse attention implementation", paragraph "Kernel Design": gradients of
// keys and values are formed per key/value block by visiting only the query blocks connected to it;
// the attention matrix is never materialised (probabilities are recomputed from the saved
// log-sum-exp, following the memory-efficient formulation the paper adopts).
//
// With w = exp(scale*q.k - LSE), dP = dO.v, D = dO.O, dS = w*(dP - D):
//   dQ_l = scale * sum_t dS_lt k_t       (query-block stationary, same traversal as the forward;
//                                         tensor-core kernel in bwd_dq_tc.cu)
//   dV_t = sum_l w_lt dO_l ; dK_t = scale * sum_l dS_lt q_l   (key-block stationary over the
//          transposed pattern: local neighbours by geometry + a CSR list of selecting query blocks)
// Summation order is fixed (no floating-point atomics), so results are deterministic.
#include "mma_util.cuh"

namespace mosaic {

constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------
// D_l = sum_c dO_lc * O_lc.  HBM-bound: 8 lanes per token, 16 bytes of each tensor per lane.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rowdot_kernel(long long tokens, const uint4* __restrict__ o,
                                                     const uint4* __restrict__ d_o, float* __restrict__ D) {
  long long t = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  int part = threadIdx.x & 7;
  float acc = 0.f;
  if (t < tokens) {
    uint4 a = __ldg(o + t * 8 + part), b = __ldg(d_o + t * 8 + part);
    const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc += __uint_as_float(av[i] << 16) * __uint_as_float(bv[i] << 16);
      acc += __uint_as_float(av[i] & 0xffff0000u) * __uint_as_float(bv[i] & 0xffff0000u);
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  acc += __shfl_xor_sync(0xffffffffu, acc, 4);
  if (part == 0 && t < tokens) D[t] = acc;
}

// ------------------------------------------------------------------------------------------
// Transposed pattern: for every key block j the ascending list of query blocks that selected it.
// One CTA per unit: histogram, exclusive scan, then an ordered fill by a single warp so that
// each list comes out sorted by query block id (this fixes the dK/dV summation order).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) csr_kernel(Geo g, const int32_t* __restrict__ block_idx,
                                                  int32_t* __restrict__ csr_off, int32_t* __restrict__ csr_q) {
  extern __shared__ int cur[];  // [m] counts, then running cursors
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const int32_t* idx = block_idx + (long long)u * g.m * g.topk;
  int32_t* off = csr_off + (long long)u * (g.m + 1);
  int32_t* outq = csr_q + (long long)u * g.m * g.topk;
  const int E = g.m * g.topk;
  for (int j = tid; j < g.m; j += blockDim.x) cur[j] = 0;
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) {
    int j = idx[e];
    if (j >= 0 && j < g.m) atomicAdd(&cur[j], 1);
  }
  __syncthreads();
  if (tid < 32) {
    int carry = 0;
    for (int base = 0; base < g.m; base += 32) {
      int j = base + lane;
      int v = j < g.m ? cur[j] : 0, incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (j < g.m) { off[j] = carry + incl - v; cur[j] = carry + incl - v; }
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) off[g.m] = carry;
    __syncwarp();
    for (int e0 = 0; e0 < E; e0 += 32) {
      int e = e0 + lane;
      int j = e < E ? idx[e] : -1;
      if (j >= g.m) j = -1;
      int key = j < 0 ? -1 - lane : j;  // invalid entries never match each other
      unsigned mask = __match_any_sync(0xffffffffu, key);
      int rank = __popc(mask & ((1u << lane) - 1u));
      int base = j >= 0 ? cur[j] : 0;
      __syncwarp();
      if (j >= 0) {
        outq[base + rank] = e / g.topk;
        if (rank == 0) cur[j] = base + __popc(mask);
      }
      __syncwarp();
    }
  }
}

// ------------------------------------------------------------------------------------------
// dK/dV kernel: one CTA per 64-token key/value chunk; visits the connected query blocks in a
// fixed order (local neighbours by geometry -- the neighbourhood relation is symmetric -- then
// the ascending CSR list) and accumulates dK, dV in registers.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) dkdv_kernel(Geo g, const __nv_bfloat16* __restrict__ q,
                                                   const __nv_bfloat16* __restrict__ k,
                                                   const __nv_bfloat16* __restrict__ v,
                                                   const __nv_bfloat16* __restrict__ d_o,
                                                   const float* __restrict__ lse, const float* __restrict__ D,
                                                   const int32_t* __restrict__ csr_off,
                                                   const int32_t* __restrict__ csr_q,
                                                   __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv) {
  __shared__ __align__(128) unsigned char tiles[4 * kTileBytes];
  __shared__ float lse_s[kChunk], D_s[kChunk];
  __shared__ int loc[kMaxList];
  __shared__ int nloc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x % g.cpb;
  const int j = (blockIdx.x / g.cpb) % g.m;
  const int u = blockIdx.x / (g.cpb * g.m);
  const long long ubase = (long long)u * g.N;
  const uint32_t Ks = smem_u32(tiles), Vs = Ks + kTileBytes, Qs = Vs + kTileBytes, dOs = Qs + kTileBytes;

  if (tid == 0) nloc = local_set(g, j, loc);
  load_tile<128>(Ks, k + ubase * kD, g, j, c, tid);
  load_tile<128>(Vs, v + ubase * kD, g, j, c, tid);
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();
  uint32_t ka[4][4], va[4][4];
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    load_A(Ks, warp * 16, kk, lane, ka[kk]);
    load_A(Vs, warp * 16, kk, lane, va[kk]);
  }
  float acck[8][4], accv[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) { acck[n][e] = 0.f; accv[n][e] = 0.f; }

  const int32_t* offs = csr_off + (long long)u * (g.m + 1);
  const int s_beg = offs[j], s_end = offs[j + 1];
  const int32_t* sel = csr_q + (long long)u * g.m * g.topk;
  const int nq = nloc + (s_end - s_beg);

  for (int qi = 0; qi < nq; ++qi) {
    const int i = qi < nloc ? loc[qi] : sel[s_beg + qi - nloc];
    for (int qc = 0; qc < g.cpb; ++qc) {
      __syncthreads();
      load_tile<128>(Qs, q + ubase * kD, g, i, qc, tid);
      load_tile<128>(dOs, d_o + ubase * kD, g, i, qc, tid);
      cp_async_commit();
      if (tid < kChunk) {
        long long t = ubase + chunk_token(g, i, qc, tid);
        lse_s[tid] = lse[t] * kLog2e;
        D_s[tid] = D[t];
      }
      cp_async_wait<0>();
      __syncthreads();

      float st[8][4], dpt[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) { st[n][e] = 0.f; dpt[n][e] = 0.f; }
      gemm_nt(st, ka, Qs, lane);    // S^T = K Q^T : rows = keys, columns = queries
      gemm_nt(dpt, va, dOs, lane);  // dP^T = V dO^T
      uint32_t pa[4][4];
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        const int col = 8 * n + 2 * (lane & 3);
        const float l0 = lse_s[col], l1 = lse_s[col + 1], d0 = D_s[col], d1 = D_s[col + 1];
        float p0 = exp2f(st[n][0] * g.scale_log2 - l0), p1 = exp2f(st[n][1] * g.scale_log2 - l1);
        float p2 = exp2f(st[n][2] * g.scale_log2 - l0), p3 = exp2f(st[n][3] * g.scale_log2 - l1);
        dpt[n][0] = p0 * (dpt[n][0] - d0);
        dpt[n][1] = p1 * (dpt[n][1] - d1);
        dpt[n][2] = p2 * (dpt[n][2] - d0);
        dpt[n][3] = p3 * (dpt[n][3] - d1);
        st[n][0] = p0; st[n][1] = p1; st[n][2] = p2; st[n][3] = p3;
      }
      acc_to_A(st, pa);
      gemm_nn(accv, pa, dOs, lane);  // dV += P^T dO
      acc_to_A(dpt, pa);
      gemm_nn(acck, pa, Qs, lane);   // dK += dS^T Q
    }
  }
  const int r0 = warp * 16 + (lane >> 2);
  const long long tok0 = ubase + chunk_token(g, j, c, r0), tok1 = ubase + chunk_token(g, j, c, r0 + 8);
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    const int col = 8 * n + 2 * (lane & 3);
    *reinterpret_cast<uint32_t*>(dk + tok0 * kD + col) = pack_bf16(acck[n][0] * g.scale, acck[n][1] * g.scale);
    *reinterpret_cast<uint32_t*>(dk + tok1 * kD + col) = pack_bf16(acck[n][2] * g.scale, acck[n][3] * g.scale);
    *reinterpret_cast<uint32_t*>(dv + tok0 * kD + col) = pack_bf16(accv[n][0], accv[n][1]);
    *reinterpret_cast<uint32_t*>(dv + tok1 * kD + col) = pack_bf16(accv[n][2], accv[n][3]);
  }
}

int launch_bwd(const HostCtx& c, const void* q, const void* k, const void* v, const void* o, const float* lse,
               const void* d_o, const int32_t* block_idx, void* dq, void* dk, void* dv, float* Dbuf,
               int32_t* csr_off, int32_t* csr_cur, int32_t* csr_q) {
  (void)csr_cur;
  const Geo& g = c.g;
  const long long tokens = (long long)g.U * g.N;
  {
    long long threads = tokens * 8;
    rowdot_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, c.stream>>>(tokens, (const uint4*)o,
                                                                           (const uint4*)d_o, Dbuf);
    if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  }
  if (g.topk > 0) {
    size_t smem = sizeof(int) * (size_t)g.m;
    if (smem > 48 * 1024) {
      if (cudaFuncSetAttribute(csr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return MOSAIC_E_CUDA;
    }
    csr_kernel<<<g.U, 256, smem, c.stream>>>(g, block_idx, csr_off, csr_q);
  } else {
    if (cudaMemsetAsync(csr_off, 0, sizeof(int32_t) * (size_t)g.U * (g.m + 1), c.stream) != cudaSuccess)
      return MOSAIC_E_CUDA;
  }
  if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  const unsigned grid = (unsigned)((long long)g.U * g.m * g.cpb);
  {
    // dQ on the tcgen05 path; its work queue counts in the second word of the status block (zeroed when the
    // op started)
    const int rc = launch_dq_tc(c, q, k, v, d_o, lse, Dbuf, block_idx, dq, c.status + 1);
    if (rc) return rc;
  }
  dkdv_kernel<<<grid, 128, 0, c.stream>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                          (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, lse, Dbuf, csr_off,
                                          csr_q, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv);
  if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  return MOSAIC_OK;
}

}  // namespace mosaic
