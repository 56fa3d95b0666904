// Forward of the block-sparse attention on Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// Paper: fine-grained attention equation of the "Selection" paragraph (section "Block-Sparse
// Attention"), evaluated over the union of the local neighbourhood and the selected blocks with one
// softmax; streaming evaluation with the query tile resident on chip and key/value blocks streamed
// through, as the appendix paragraph "Kernel Design" describes.
//
// One CTA owns a tile of 128 query rows:
//   * 64-token blocks (8x8): two consecutive query blocks share the tile; the CTA walks the UNION of
//     their key lists and each 64-row half skips (P = 0) the blocks only the other half attends, so
//     every staged key/value block serves both halves.
//   * larger blocks (16x16): half of one query block (two 64-token chunks); one key list.
// Key/value data moves in 64-token chunks: one 4-D TMA box {d, bw, 64/bw, 1} of the [U, nlat, nlon, d]
// view lands as 64 rows x 128 B in 128-byte-swizzled shared memory, which is at once the K-major
// operand layout for S = Q K^T and the MN-major operand layout for O += P V.
//
// Warp roles (192 threads): warps 0-3 softmax (thread r owns query row r = TMEM lane r),
// warp 4 builds the key list and issues TMA, warp 5 allocates TMEM and issues tcgen05.mma.
// TMEM columns: [0,64) O accumulator, then SBUFS S buffers of 64 columns; P (bf16) overwrites the
// first 32 columns of its S buffer and is consumed from TMEM as the A operand of P V.
// Several CTAs are resident per SM, so one CTA's softmax overlaps another's tensor work.
// Every mbarrier wait is bounded; on expiry the CTA records MOSAIC_E_DEVICE_TIMEOUT and drains.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "common.cuh"

namespace mosaic {

namespace {

constexpr int kTile = 8192;                    // bytes of one 64 x 64 bf16 chunk
constexpr uint32_t kColO = 0, kColS = 64;
constexpr long long kSpinCycles = 4000000000ll;  // bound of a single wait (~2 s)
constexpr float kRescaleThreshold = 8.0f;      // log2 units: P stays below 2^8

template <int NST, int SBUFS>
struct SmemTC {
  unsigned char q[2 * kTile];
  unsigned char kv[NST][2][kTile];
  unsigned long long kv_full[NST], kv_empty[NST], q_full, s_full[SBUFS], p_full[SBUFS], pv_done[SBUFS];
  uint32_t tmem_base;
  int abort;
  int nlist;
  int ids[2 * kMaxList];
  unsigned char mask[2 * kMaxList];
};

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false after the limit (status recorded) or once another thread aborted.
// The clock and the abort flag are looked at only every 64 polls to keep the poll loop light.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
#pragma unroll 1
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 0u) {
      if (*abort) return false;
      if (clock64() - t0 > kSpinCycles) {
        set_status(status, MOSAIC_E_DEVICE_TIMEOUT);
        *abort = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, "
      "%6}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void umma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::
          "r"(d),
      "l"(a), "l"(b), "r"(idesc), "r"(acc)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::
          "r"(d),
      "r"(a), "l"(b), "r"(idesc), "r"(acc)
      : "memory");
}

#define MOSAIC_R32(r, o)                                                                                         \
  "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), \
      "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]), "=r"(r[o + 12]),          \
      "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15]), "=r"(r[o + 16]), "=r"(r[o + 17]), "=r"(r[o + 18]),       \
      "=r"(r[o + 19]), "=r"(r[o + 20]), "=r"(r[o + 21]), "=r"(r[o + 22]), "=r"(r[o + 23]), "=r"(r[o + 24]),       \
      "=r"(r[o + 25]), "=r"(r[o + 26]), "=r"(r[o + 27]), "=r"(r[o + 28]), "=r"(r[o + 29]), "=r"(r[o + 30]),       \
      "=r"(r[o + 31])
#define MOSAIC_W32(r, o)                                                                                      \
  "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]),     \
      "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), "r"(r[o + 12]),             \
      "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15]), "r"(r[o + 16]), "r"(r[o + 17]), "r"(r[o + 18]),          \
      "r"(r[o + 19]), "r"(r[o + 20]), "r"(r[o + 21]), "r"(r[o + 22]), "r"(r[o + 23]), "r"(r[o + 24]),          \
      "r"(r[o + 25]), "r"(r[o + 26]), "r"(r[o + 27]), "r"(r[o + 28]), "r"(r[o + 29]), "r"(r[o + 30]),          \
      "r"(r[o + 31])

// 32 consecutive 32-bit TMEM columns of this thread's lane -> registers r[o .. o+31]
template <int O, int N>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[N]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
      "%15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : MOSAIC_R32(r, O)
      : "r"(taddr)
      : "memory");
}
template <int O, int N>
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[N]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
      "%15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      MOSAIC_W32(r, O)
      : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two fp32 lanes in one 64-bit register (packed fp32 arithmetic of this architecture)
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Shared-memory operand descriptor: 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;               // leading byte offset (not used by these shapes)
  d |= (uint64_t)(1024 >> 4) << 32;     // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;               // descriptor version of this architecture
  d |= (uint64_t)2 << 61;               // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 64.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((64u >> 3) << 17) |
         ((128u >> 4) << 24);
}

}  // namespace

// Warp-cooperative attended list of query block i (local set, then valid selected ids), appended to
// ids[n0..); returns the new count.  Same order as attended_list().
__device__ __forceinline__ int warp_attended(const Geo& g, const int32_t* __restrict__ idx_row, int i, int* ids,
                                             int n0, int lane, int* status) {
  const int by = i / g.nbw, bx = i - by * g.nbw;
  const int wl = 2 * g.rlon + 1, nl = (2 * g.rlat + 1) * wl;
  int id = -1 - lane;
  if (lane < nl) {
    const int dy = lane / wl - g.rlat, dx = lane - (lane / wl) * wl - g.rlon;
    const int y = min(max(by + dy, 0), g.nbh - 1);
    int x = (bx + dx) % g.nbw;
    x += x < 0 ? g.nbw : 0;
    id = y * g.nbw + x;
  }
  const unsigned same = __match_any_sync(0xffffffffu, id);
  const bool keep = lane < nl && (__ffs(same) - 1) == lane;  // first occurrence of a block
  const unsigned km = __ballot_sync(0xffffffffu, keep);
  if (keep) ids[n0 + __popc(km & ((1u << lane) - 1u))] = id;
  int n = n0 + __popc(km);
  int j = lane < g.topk ? __ldg(idx_row + lane) : -1;
  if (j < -1 || j >= g.m) { set_status(status, MOSAIC_E_DEVICE_BAD_INDEX); j = -1; }
  const unsigned sm_ = __ballot_sync(0xffffffffu, j >= 0);
  if (j >= 0) ids[n + __popc(sm_ & ((1u << lane) - 1u))] = j;
  return n + __popc(sm_);
}

template <int NST, int SBUFS, int MINB>
__global__ void __launch_bounds__(192, MINB)
    fwd_tc_kernel(const Geo g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ block_idx,
                  __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int* status, int tiles_per_unit) {
  using Smem = SmemTC<NST, SBUFS>;
  constexpr uint32_t kTmemCols = SBUFS == 1 ? 128 : 256;
  extern __shared__ unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x / tiles_per_unit, t = blockIdx.x - u * tiles_per_unit;

  // the two 64-row halves of the tile: (block, chunk) each
  int hb0, hb1, hc0, hc1;
  bool hvalid1 = true;
  if (g.cpb == 1) {
    hb0 = 2 * t; hb1 = 2 * t + 1; hc0 = hc1 = 0;
    if (hb1 >= g.m) { hvalid1 = false; hb1 = hb0; }
  } else {
    const int hpb = g.cpb / 2;  // tiles per block
    hb0 = hb1 = t / hpb;
    hc0 = 2 * (t % hpb); hc1 = hc0 + 1;
  }

  if (tid == 0) {
    for (int s = 0; s < NST; ++s) { mbar_init(s32(&sm.kv_full[s]), 1); mbar_init(s32(&sm.kv_empty[s]), 1); }
    mbar_init(s32(&sm.q_full), 1);
    for (int s = 0; s < SBUFS; ++s) {
      mbar_init(s32(&sm.s_full[s]), 1);
      mbar_init(s32(&sm.p_full[s]), 128);
      mbar_init(s32(&sm.pv_done[s]), 1);
    }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 4) {
    if (lane == 0) {  // the query tile does not depend on the key list: start it first
      mbar_expect_tx(s32(&sm.q_full), 2 * kTile);
      int by = hb0 / g.nbw, bx = hb0 - by * g.nbw;
      tma_load_4d(s32(sm.q), &map_q, s32(&sm.q_full), 0, bx * g.bw, by * g.bh + hc0 * g.crows, u);
      by = hb1 / g.nbw; bx = hb1 - by * g.nbw;
      tma_load_4d(s32(sm.q + kTile), &map_q, s32(&sm.q_full), 0, bx * g.bw, by * g.bh + hc1 * g.crows, u);
    }
    // key list: entries of the first half's block, then what only the second half adds
    const int32_t* row0 = block_idx + ((long long)u * g.m + hb0) * g.topk;
    int n = warp_attended(g, row0, hb0, sm.ids, 0, lane, status);
    __syncwarp();
    const unsigned char m0 = g.cpb == 1 ? 1 : 3;
    for (int e = lane; e < n; e += 32) sm.mask[e] = m0;
    if (g.cpb == 1 && hvalid1) {
      const int32_t* row1 = block_idx + ((long long)u * g.m + hb1) * g.topk;
      const int n0 = n;
      const int n1 = warp_attended(g, row1, hb1, sm.ids, n0, lane, status) - n0;  // staged behind list 0
      __syncwarp();
      // entries of list 1 (at most 2 per lane): shared with list 0 -> mark, else keep (compacted)
      int mine[2], pos[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int e = lane + 32 * r;
        mine[r] = e < n1 ? sm.ids[n0 + e] : -1;
        pos[r] = -1;
      }
      for (int a = 0; a < n0; ++a) {
        const int id = sm.ids[a];
        pos[0] = id == mine[0] ? a : pos[0];
        pos[1] = id == mine[1] ? a : pos[1];
      }
      __syncwarp();
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const bool have = mine[r] >= 0, fresh = have && pos[r] < 0;
        if (have && pos[r] >= 0) sm.mask[pos[r]] |= 2;
        const unsigned fm = __ballot_sync(0xffffffffu, fresh);
        if (fresh) {
          const int at = n + __popc(fm & ((1u << lane) - 1u));
          sm.ids[at] = mine[r];
          sm.mask[at] = 2;
        }
        n += __popc(fm);
        __syncwarp();
      }
    }
    if (lane == 0) sm.nlist = n;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  const uint32_t tmem = sm.tmem_base;
  const int nch = sm.nlist * g.cpb;
  volatile int* abort = &sm.abort;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int it = 0; it < nch; ++it) {
        const int st = it % NST, j = sm.ids[it / g.cpb], c = it % g.cpb;
        if (!mbar_wait(s32(&sm.kv_empty[st]), ((it / NST) & 1) ^ 1, abort, status)) break;
        const int by = j / g.nbw, bx = j - by * g.nbw;
        mbar_expect_tx(s32(&sm.kv_full[st]), 2 * kTile);
        tma_load_4d(s32(sm.kv[st][0]), &map_k, s32(&sm.kv_full[st]), 0, bx * g.bw, by * g.bh + c * g.crows, u);
        tma_load_4d(s32(sm.kv[st][1]), &map_v, s32(&sm.kv_full[st]), 0, bx * g.bw, by * g.bh + c * g.crows, u);
      }
      if (*abort) {  // give copies in flight time to land before the CTA's memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) {}
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(false), idesc_pv = make_idesc(true);
      const uint64_t qdesc = smem_desc(s32(sm.q));
      bool ok = mbar_wait(s32(&sm.q_full), 0, abort, status);
      auto issue_qk = [&](int it) {
        const uint64_t kdesc = smem_desc(s32(sm.kv[it % NST][0]));
        const uint32_t d = tmem + kColS + (it % SBUFS) * 64;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma_ss(d, qdesc + 2 * kk, kdesc + 2 * kk, idesc_qk, kk > 0);
        tc_commit(s32(&sm.s_full[it % SBUFS]));
      };
      // S buffer of iteration `it` is free once P V of iteration it - SBUFS has completed
      auto wait_sbuf = [&](int it) {
        const int prev = it - SBUFS;
        return prev < 0 || mbar_wait(s32(&sm.pv_done[prev % SBUFS]), (prev / SBUFS) & 1, abort, status);
      };
      if (ok && nch > 0) {
        ok = mbar_wait(s32(&sm.kv_full[0]), 0, abort, status);
        if (ok) { tc_fence_after(); issue_qk(0); }
      }
      for (int it = 0; ok && it < nch; ++it) {
        if (SBUFS > 1 && it + 1 < nch) {
          ok = mbar_wait(s32(&sm.kv_full[(it + 1) % NST]), ((it + 1) / NST) & 1, abort, status) && wait_sbuf(it + 1);
          if (!ok) break;
          tc_fence_after();
          issue_qk(it + 1);
        }
        ok = mbar_wait(s32(&sm.p_full[it % SBUFS]), (it / SBUFS) & 1, abort, status);
        if (!ok) break;
        tc_fence_after();
        const uint64_t vdesc = smem_desc(s32(sm.kv[it % NST][1]));
        const uint32_t p = tmem + kColS + (it % SBUFS) * 64;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_ts(tmem + kColO, p + 8 * kk, vdesc + (uint64_t)((2048 * kk) >> 4), idesc_pv, (it > 0 || kk > 0));
        tc_commit(s32(&sm.kv_empty[it % NST]));
        tc_commit(s32(&sm.pv_done[it % SBUFS]));
        if (SBUFS == 1 && it + 1 < nch) {
          ok = mbar_wait(s32(&sm.kv_full[(it + 1) % NST]), ((it + 1) / NST) & 1, abort, status) && wait_sbuf(it + 1);
          if (!ok) break;
          tc_fence_after();
          issue_qk(it + 1);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax, then epilogue
    const int h = warp >> 1;  // which 64-row half this warp's rows belong to
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const uint64_t scale2 = pack2(g.scale_log2, g.scale_log2);
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int it = 0; it < nch; ++it) {
      const int sb = it % SBUFS;
      ok = mbar_wait(s32(&sm.s_full[sb]), (it / SBUFS) & 1, abort, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool attends = (sm.mask[it / g.cpb] >> h) & 1;
      const uint32_t ts = tmem + lane_off + kColS + sb * 64;
      bool need = false;
      float alpha = 1.f;
      uint32_t pk[32];
      if (attends) {
        uint32_t sr[64];
        tmem_ld32<0>(ts, sr);
        tmem_ld32<32>(ts + 32, sr);
        tmem_wait_ld();
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]), mx2 = __uint_as_float(sr[2]),
              mx3 = __uint_as_float(sr[3]);
#pragma unroll
        for (int c = 4; c < 64; c += 4) {
          mx0 = fmaxf(mx0, __uint_as_float(sr[c]));
          mx1 = fmaxf(mx1, __uint_as_float(sr[c + 1]));
          mx2 = fmaxf(mx2, __uint_as_float(sr[c + 2]));
          mx3 = fmaxf(mx3, __uint_as_float(sr[c + 3]));
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * g.scale_log2;  // scale > 0 commutes with max
        if (m_ref == -INFINITY) {
          m_ref = mx;
        } else if (mx > m_ref + kRescaleThreshold) {
          need = true;
          alpha = ex2(m_ref - mx);
          m_ref = mx;
          l *= alpha;
        }
        const uint64_t negm2 = pack2(-m_ref, -m_ref);
        uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
#pragma unroll
        for (int c = 0; c < 64; c += 4) {
          float x0, x1, x2, x3;
          unpack2(fma2(pack2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), scale2, negm2), x0, x1);
          unpack2(fma2(pack2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), scale2, negm2), x2, x3);
          const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
          sum_a = add2(sum_a, pack2(p0, p1));
          sum_b = add2(sum_b, pack2(p2, p3));
          __nv_bfloat162 pa = __floats2bfloat162_rn(p0, p1), pb = __floats2bfloat162_rn(p2, p3);
          pk[c >> 1] = *reinterpret_cast<uint32_t*>(&pa);
          pk[(c >> 1) + 1] = *reinterpret_cast<uint32_t*>(&pb);
        }
        float s0, s1;
        unpack2(add2(sum_a, sum_b), s0, s1);
        l += s0 + s1;
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) pk[c] = 0u;
      }
      tmem_st32<0>(ts, pk);
      if (__any_sync(0xffffffffu, need)) {
        // the accumulator may only be touched between P V products
        if (it > 0) {
          ok = mbar_wait(s32(&sm.pv_done[(it - 1) % SBUFS]), ((it - 1) / SBUFS) & 1, abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t to = tmem + lane_off + kColO;
        const uint64_t alpha2 = pack2(alpha, alpha);
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          uint32_t ov[32];
          tmem_ld32<0>(to + 32 * part, ov);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            float a, b;
            unpack2(mul2(pack2(__uint_as_float(ov[c]), __uint_as_float(ov[c + 1])), alpha2), a, b);
            ov[c] = __float_as_uint(a);
            ov[c + 1] = __float_as_uint(b);
          }
          tmem_st32<0>(to + 32 * part, ov);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(s32(&sm.p_full[sb]));
    }
    if (ok && nch > 0) {
      const int last = nch - 1;
      ok = mbar_wait(s32(&sm.pv_done[last % SBUFS]), (last / SBUFS) & 1, abort, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && nch > 0 && (h == 0 || hvalid1)) {
      tc_fence_after();
      const int e = tid & 63;
      const long long tok = (long long)u * g.N + chunk_token(g, h ? hb1 : hb0, h ? hc1 : hc0, e);
      const float inv = 1.f / l;
      const uint32_t to = tmem + lane_off + kColO;
      uint4* dst = reinterpret_cast<uint4*>(o + tok * kD);
#pragma unroll
      for (int part = 0; part < 2; ++part) {
        uint32_t ov[32];
        tmem_ld32<0>(to + 32 * part, ov);
        tmem_wait_ld();
        uint32_t w[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          __nv_bfloat162 pb =
              __floats2bfloat162_rn(__uint_as_float(ov[2 * c]) * inv, __uint_as_float(ov[2 * c + 1]) * inv);
          w[c] = *reinterpret_cast<uint32_t*>(&pb);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) dst[part * 4 + c] = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
      }
      lse[tok] = (m_ref + log2f(l)) * 0.6931471805599453f;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [U, nlat, nlon, d] bf16 view, box = one 64-token chunk {d, bw, 64/bw, 1}, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, const Geo& g) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)g.nlon, (cuuint64_t)g.nlat, (cuuint64_t)g.U};
  cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)g.nlon * kD * 2, (cuuint64_t)g.N * kD * 2};
  cuuint32_t box[4] = {(cuuint32_t)kD, (cuuint32_t)g.bw, (cuuint32_t)g.crows, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

template <int NST, int SBUFS, int MINB>
int launch_variant(const HostCtx& c, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                   const int32_t* block_idx, void* o, float* lse) {
  const Geo& g = c.g;
  auto kern = fwd_tc_kernel<NST, SBUFS, MINB>;
  const size_t smem = sizeof(SmemTC<NST, SBUFS>) + 1024;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return MOSAIC_E_CUDA;
  const int tiles_per_unit = g.cpb == 1 ? (g.m + 1) / 2 : g.m * (g.cpb / 2);
  const long long grid = (long long)g.U * tiles_per_unit;
  kern<<<(unsigned)grid, 192, smem, c.stream>>>(g, mq, mk, mv, block_idx, (__nv_bfloat16*)o, lse, c.status,
                                                tiles_per_unit);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_fwd_tc(const HostCtx& c, const void* q, const void* k, const void* v, const int32_t* block_idx, void* o,
                  float* lse) {
  const Geo& g = c.g;
  if (!(g.cpb == 1 || g.cpb % 2 == 0)) return MOSAIC_E_UNSUPPORTED;
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, q, g) || !make_map(&mk, k, g) || !make_map(&mv, v, g)) return MOSAIC_E_CUDA;
  const char* var = getenv("MOSAIC_BSA_FWD_VARIANT");  // tuning aid; default below
  const int which = var ? atoi(var) : 0;
  switch (which) {
    case 1: return launch_variant<3, 1, 3>(c, mq, mk, mv, block_idx, o, lse);
    case 2: return launch_variant<2, 1, 4>(c, mq, mk, mv, block_idx, o, lse);
    default: return launch_variant<4, 2, 2>(c, mq, mk, mv, block_idx, o, lse);
  }
}

}  // namespace mosaic
