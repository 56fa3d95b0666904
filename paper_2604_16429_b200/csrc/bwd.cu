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
//          transposed pattern: local neighbours by geometry + a CSR list of selecting query blocks;
//          tensor-core kernel in bwd_dkdv_tc.cu)
// Summation order is fixed (no floating-point atomics), so results are deterministic.
#include "common.cuh"

namespace mosaic {

constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------
// D_l = sum_c dO_lc * O_lc (also stored negated, with the negated base-2 log-sum-exp beside it).
// HBM-bound: 8 lanes per token, 16 bytes of each tensor per lane.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rowdot_kernel(long long tokens, const uint4* __restrict__ o,
                                                     const uint4* __restrict__ d_o, const float* __restrict__ lse,
                                                     float* __restrict__ D, float* __restrict__ neg_d,
                                                     float* __restrict__ neg_lse2, bool f16) {
  long long t = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  int part = threadIdx.x & 7;
  float acc = 0.f;
  if (t < tokens) {
    uint4 a = __ldg(o + t * 8 + part), b = __ldg(d_o + t * 8 + part);
    const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float a0, a1, b0, b1;
      unpack16x2(av[i], f16, a0, a1);
      unpack16x2(bv[i], f16, b0, b1);
      acc += a0 * b0;
      acc += a1 * b1;
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  acc += __shfl_xor_sync(0xffffffffu, acc, 4);
  if (part == 0 && t < tokens) {
    D[t] = acc;
    neg_d[t] = -acc;                     // the key-stationary kernel reads these per query column
    neg_lse2[t] = -lse[t] * kLog2e;      // log-sum-exp in base-2 units, negated
  }
}

// ------------------------------------------------------------------------------------------
// Transposed pattern: for every key block j the ascending list of query blocks that selected it.
// One CTA per unit.  The query blocks are cut into `nseg` contiguous segments:
//   1. one thread per query block validates its row of block_idx (ids outside [0, m), ids of the row's own
//      neighbourhood and repeats are dropped, exactly as the forward drops them), marks the valid entries in a
//      bit array and counts them per (segment, key block);
//   2. per key block, a running sum over the segments and an exclusive scan over the key blocks turn the counts
//      into the position where each segment's part of each list starts;
//   3. every warp fills its segments in entry order, so each list comes out sorted by query block id (this
//      fixes the dK/dV summation order).
// Shared memory: (nseg + 1) * m counters + m * topk bits.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) csr_kernel(Geo g, const int32_t* __restrict__ block_idx,
                                                  int32_t* __restrict__ csr_off, int32_t* __restrict__ csr_q, int nseg) {
  extern __shared__ int csr_sm[];
  int* tot = csr_sm;                        // [m] list lengths, then list starts
  int* seg = csr_sm + g.m;                  // [nseg][m] counts, then cursors
  unsigned* bits = reinterpret_cast<unsigned*>(seg + (long long)nseg * g.m);  // [ceil(m * topk / 32)] valid entries
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* idx = block_idx + (long long)u * g.m * g.topk;
  int32_t* off = csr_off + (long long)u * (g.m + 1);
  int32_t* outq = csr_q + (long long)u * g.m * g.topk;
  const int E = g.m * g.topk, rps = (g.m + nseg - 1) / nseg;  // rows per segment
  for (int x = tid; x < (nseg + 1) * g.m; x += blockDim.x) csr_sm[x] = 0;
  for (int x = tid; x < (E + 31) / 32; x += blockDim.x) bits[x] = 0u;
  __syncthreads();
  for (int i = tid; i < g.m; i += blockDim.x) {
    const int32_t* row = idx + (long long)i * g.topk;
    int* cnt = seg + (long long)(i / rps) * g.m;
    for (int r = 0; r < g.topk; ++r) {
      bool report;
      if (selected_entry_ok(g, row, i, r, &report)) {
        atomicAdd(&cnt[row[r]], 1);
        const int e = i * g.topk + r;
        atomicOr(&bits[e >> 5], 1u << (e & 31));
      }
    }
  }
  __syncthreads();
  for (int j = tid; j < g.m; j += blockDim.x) {
    int t = 0;
    for (int sgm = 0; sgm < nseg; ++sgm) {
      const int c = seg[(long long)sgm * g.m + j];
      seg[(long long)sgm * g.m + j] = t;
      t += c;
    }
    tot[j] = t;
  }
  __syncthreads();
  if (tid < 32) {
    int carry = 0;
    for (int base = 0; base < g.m; base += 32) {
      const int j = base + lane;
      const int v = j < g.m ? tot[j] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int nb = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += nb;
      }
      if (j < g.m) { off[j] = carry + incl - v; tot[j] = carry + incl - v; }
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) off[g.m] = carry;
  }
  __syncthreads();
  for (int sgm = warp; sgm < nseg; sgm += (int)(blockDim.x >> 5)) {
    int* cur = seg + (long long)sgm * g.m;  // only this warp touches this segment's cursors
    const int e_beg = sgm * rps * g.topk, e_end = min(E, (sgm + 1) * rps * g.topk);
    for (int e0 = e_beg; e0 < e_end; e0 += 32) {
      const int e = e0 + lane;
      int j = -1;
      if (e < e_end && ((bits[e >> 5] >> (e & 31)) & 1u)) j = idx[e];
      const int key = j < 0 ? -1 - lane : j;  // invalid entries never match each other
      const unsigned same = __match_any_sync(0xffffffffu, key);
      const int rank = __popc(same & ((1u << lane) - 1u));
      const int base = j >= 0 ? tot[j] + cur[j] : 0;
      __syncwarp();
      if (j >= 0) {
        outq[base + rank] = e / g.topk;
        if (rank == 0) cur[j] += __popc(same);
      }
      __syncwarp();
    }
  }
}

// segments of the transposed-pattern kernel that fit the shared memory (8 when possible: one per warp)
static int csr_segments(const Geo& g, size_t* smem) {
  const size_t budget = 200 * 1024, bits = 4 * (((size_t)g.m * g.topk + 31) / 32);
  int nseg = 8;
  while (nseg > 1 && (size_t)(nseg + 1) * g.m * sizeof(int) + bits > budget) --nseg;
  *smem = (size_t)(nseg + 1) * g.m * sizeof(int) + bits;
  return *smem <= budget ? nseg : 0;
}

int launch_bwd(const HostCtx& c, const void* q, const void* k, const void* v, const void* o, const float* lse,
               const void* d_o, const int32_t* block_idx, void* dq, void* dk, void* dv, float* Dbuf, float* neg_d,
               float* neg_lse2,
               int32_t* csr_off, int32_t* csr_q, int32_t* order, int* counters) {
  const Geo& g = c.g;
  const long long tokens = (long long)g.U * g.N;
  {
    long long threads = tokens * 8;
    rowdot_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, c.stream>>>(tokens, (const uint4*)o,
                                                                           (const uint4*)d_o, lse, Dbuf, neg_d, neg_lse2, g.f16 != 0);
    if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  }
  if (g.topk > 0) {
    size_t smem = 0;
    const int nseg = csr_segments(g, &smem);
    if (nseg == 0) return MOSAIC_E_UNSUPPORTED;
    static unsigned long long configured = 0;  // devices on which the kernel's shared-memory opt-in is set
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
    if (dev >= 0 && dev < 64 && !((configured >> dev) & 1ull)) {
      if (cudaFuncSetAttribute(csr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
        return MOSAIC_E_CUDA;
      configured |= 1ull << dev;
    }
    csr_kernel<<<g.U, 256, smem, c.stream>>>(g, block_idx, csr_off, csr_q, nseg);
  } else {
    if (cudaMemsetAsync(csr_off, 0, sizeof(int32_t) * (size_t)g.U * (g.m + 1), c.stream) != cudaSuccess)
      return MOSAIC_E_CUDA;
  }
  if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  {
    // dQ on the tcgen05 path; its work queue counts in a word of the status block (zeroed when the op started)
    const int rc = launch_dq_tc(c, q, k, v, d_o, lse, Dbuf, block_idx, dq, counters);
    if (rc) return rc;
  }
  {
    // dK, dV on the tcgen05 path; its work queue counts in the next word
    const int rc = launch_dkdv_tc(c, q, k, v, d_o, neg_lse2, neg_d, csr_off, csr_q, dk, dv, counters + 1, order);
    if (rc) return rc;
  }
  return MOSAIC_OK;
}

}  // namespace mosaic
