// Shared device/host definitions of the MOSAIC block-sparse attention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mosaic_bsa.h"

namespace mosaic {

constexpr int kD = 64;            // head dimension
constexpr int kChunk = 64;        // tokens per staged key/value chunk (and per mma.sync query tile)
constexpr int kMaxList = 64;      // most blocks one query block attends (local + top-k)
constexpr int kMaxTopk = 32;
constexpr int kStatusBytes = 256; // status block at the start of every workspace

// Geometry of one call, passed by value to the kernels.
struct Geo {
  int U;            // B*H independent units
  int H, Hkv;       // query heads, key/value heads (grouped-query attention: H / Hkv query heads share a key/value head)
  int Ukv;          // B*Hkv key/value units
  int nlat, nlon;   // grid
  int bh, bw;       // block shape
  int nbh, nbw, m;  // blocks per column / row / unit
  int b;            // tokens per block
  int cpb;          // 64-token chunks per block (b / 64)
  int crows;        // grid rows per chunk (64 / bw)
  int rlat, rlon, topk;
  int local_off;    // 1: the local neighbourhood is not attended (selection branch of the three-branch form)
  int local_groups; // 1: the local set is the aligned group of rlat x rlon blocks that holds the block
  int f16;          // 1: the 16-bit tensors are IEEE binary16, 0: bf16
  float scale;      // softmax scale
  float scale_log2; // scale * log2(e)
  long long N;      // tokens per unit
};

// key/value unit read by query unit u
__host__ __device__ __forceinline__ int kv_unit(const Geo& g, int u) {
  const int b = u / g.H;
  return b * g.Hkv + (u - b * g.H) / (g.H / g.Hkv);
}

// Two 16-bit elements of the problem's storage type (bf16 or binary16) packed in a word <-> two floats.
__device__ __forceinline__ void unpack16x2(uint32_t x, bool f16, float& lo, float& hi) {
  if (f16) {
    const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&x));
    lo = v.x;
    hi = v.y;
  } else {
    lo = __uint_as_float(x << 16);
    hi = __uint_as_float(x & 0xffff0000u);
  }
}
__device__ __forceinline__ uint32_t pack16x2(float lo, float hi, bool f16) {
  if (f16) {
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
  }
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Record the first device-side fault in the workspace status word (never traps).
__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

// Is key block j inside the local set of query block i (window: rows clamp(by+dy), columns (bx+dx) mod nbw;
// group mode: the same aligned group of rlat x rlon blocks)?
__device__ __forceinline__ bool is_local(const Geo& g, int i, int j) {
  int by = i / g.nbw, bx = i - by * g.nbw;
  int jy = j / g.nbw, jx = j - jy * g.nbw;
  if (g.local_groups) return by / g.rlat == jy / g.rlat && bx / g.rlon == jx / g.rlon;
  // clamping only folds an out-of-range row onto a row already in the window
  bool row_ok = abs(jy - by) <= g.rlat;
  int dx = jx - bx;
  dx += dx < 0 ? g.nbw : 0;                       // (jx - bx) mod nbw in [0, nbw)
  bool col_ok = dx <= g.rlon || g.nbw - dx <= g.rlon;
  return row_ok && col_ok;
}

// Is entry r of a row of block_idx (query block i) one the kernels use?  Ids outside [0, m), ids inside the
// row's local set (already attended through the neighbourhood) and repeats of an earlier entry of the row are
// not: they are skipped, and reported unless the entry is the padding value -1.
__device__ __forceinline__ bool selected_entry_ok(const Geo& g, const int32_t* __restrict__ idx_row, int i, int r,
                                                  bool* report) {
  const int j = idx_row[r];
  *report = false;
  if (j == -1) return false;
  *report = true;
  if (j < 0 || j >= g.m || is_local(g, i, j)) return false;
  for (int a = 0; a < r; ++a)
    if (idx_row[a] == j) return false;
  *report = false;
  return true;
}

// First token (row-major grid index inside the unit) of row `r` of chunk `c` of block j.
__device__ __forceinline__ long long chunk_row_token(const Geo& g, int j, int c, int r) {
  int by = j / g.nbw, bx = j - by * g.nbw;
  return (long long)(by * g.bh + c * g.crows + r) * g.nlon + bx * g.bw;
}

// Token of element e (0..63, row-major inside the chunk) of chunk c of block j.
__device__ __forceinline__ long long chunk_token(const Geo& g, int j, int c, int e) {
  int r = e / g.bw;
  return chunk_row_token(g, j, c, r) + (e - r * g.bw);
}

// Work items of 256 rows (four 64-row halves) per unit, as the tensor-core kernels cut a unit's blocks.
__host__ __device__ inline int items_per_unit(const Geo& g) {
  if (g.cpb == 1) return (g.nbh >> 1) * ((g.nbw + 1) >> 1) + (g.nbh & 1) * ((g.nbw + 3) >> 2);
  if (g.cpb == 2) return g.nbw > 1 ? g.nbh * ((g.nbw + 1) >> 1) : (g.nbh + 1) >> 1;
  return g.m * ((g.cpb + 3) >> 2);
}

// ---- host side ---------------------------------------------------------------------------
struct HostCtx {
  Geo g;
  cudaStream_t stream;
  int* status;  // device pointer to the workspace status word
};

int validate(const mosaic_bsa_params* p, Geo* g);
size_t align256(size_t x);

// kernel launchers (one per translation unit)
// Layout of the selection's scratch behind the status block: pooled sums of Q and of K ([U, m, d] fp32 each),
// then the norm bounds of the pooled vectors ([U, m] fp32 each).
struct SelectWs { size_t pq, pk, nq, nk, total; };
SelectWs select_layout(const Geo& g);
int launch_select(const HostCtx& c, const void* q, const void* k, int32_t* block_idx, float* pooled_q,
                  float* pooled_k, float* norm_q, float* norm_k);
int launch_fwd_tc(const HostCtx& c, const void* q, const void* k, const void* v, const int32_t* block_idx,
                  void* o, float* lse, int* work_counter);
// Layout of the three-branch forward's scratch behind the status block
struct BranchWs { size_t pq, pk, pv, nrm, ocg, ofg, ol, total; };
BranchWs branch_layout(const Geo& g);
int launch_pool_one(const HostCtx& c, const void* x, float* pooled, float* norm, int units);
// `lse2` (may be null): base-2 log-sum-exp of every query block's block-level logits, [U, m]
int launch_compress(const HostCtx& c, const float* pooled_q, const float* pooled_k, const float* pooled_v, float* ocg,
                    float* lse2);
// backward of the three-branch form (branches_bwd.cu)
int launch_gate(const HostCtx& c, const void* d_o, const void* o_fg, const void* o_l, const float* ocg,
                const float* gates, float* dgates, void* do_fg, void* do_l, float* dob);
int launch_compress_bwd(const HostCtx& c, const float* pq, const float* pk, const float* pv, const float* dob,
                        const float* ocg, const float* lse2, float* delta, float* dqm, float* dkm, float* dvm);
int launch_rope(const HostCtx& c, const void* q, const void* k, const float* pos, double theta, void* q_out, void* k_out);
int launch_grad_sum(const HostCtx& c, int units, const void* x_l, const void* x_fg, const float* xm, void* out);
int launch_combine(const HostCtx& c, const float* ocg, const void* o_fg, const void* o_l, const float* gates, void* o);
int launch_dq_tc(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* D, const int32_t* block_idx, void* dq, int* work_counter);
int launch_dkdv_tc(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o,
                   const float* neg_lse2, const float* neg_d, const int32_t* csr_off, const int32_t* csr_q, void* dk,
                   void* dv, int* work_counter, int32_t* order);
int launch_bwd(const HostCtx& c, const void* q, const void* k, const void* v, const void* o, const float* lse,
               const void* d_o, const int32_t* block_idx, void* dq, void* dk, void* dv, float* Dbuf, float* neg_d,
               float* neg_lse2, int32_t* csr_off, int32_t* csr_q, int32_t* order, int* counters);

}  // namespace mosaic
