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
// TMEM columns: [0,64) O accumulator, [64,128) and [128,192) two S buffers; P (bf16) overwrites
// the first 32 columns of its S buffer and is consumed from TMEM as the A operand of P V.
// Every mbarrier wait is bounded; on expiry the CTA records MOSAIC_E_DEVICE_TIMEOUT and drains.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"

namespace mosaic {

namespace {

constexpr int NSTAGE = 4;
constexpr int kTile = 8192;                    // bytes of one 64 x 64 bf16 chunk
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColO = 0, kColS = 64;
constexpr long long kSpinCycles = 4000000000ll;  // bound of a single wait (~2 s)
constexpr float kRescaleThreshold = 8.0f;      // log2 units: P stays below 2^8

struct SmemTC {
  unsigned char q[2 * kTile];
  unsigned char kv[NSTAGE][2][kTile];
  unsigned long long kv_full[NSTAGE], kv_empty[NSTAGE], q_full, s_full[2], p_full[2], pv_done[2];
  uint32_t tmem_base;
  int abort;
  int nlist;
  int ids[2 * kMaxList];
  unsigned char mask[2 * kMaxList];
  int tmp[kMaxList];
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
    if (clock64() - t0 > kSpinCycles) {
      set_status(status, MOSAIC_E_DEVICE_TIMEOUT);
      *abort = 1;
      return false;
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

__global__ void __launch_bounds__(192, 2)
    fwd_tc_kernel(const Geo g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ block_idx,
                  __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int* status, int tiles_per_unit) {
  extern __shared__ unsigned char smem_raw[];
  SmemTC& sm = *reinterpret_cast<SmemTC*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x / tiles_per_unit, t = blockIdx.x - u * tiles_per_unit;

  // the two 64-row halves of the tile: (block, chunk) each
  int hb[2], hc[2];
  bool hvalid1 = true;
  if (g.cpb == 1) {
    hb[0] = 2 * t; hb[1] = 2 * t + 1; hc[0] = hc[1] = 0;
    if (hb[1] >= g.m) { hvalid1 = false; hb[1] = hb[0]; }
  } else {
    const int hpb = g.cpb / 2;  // tiles per block
    hb[0] = hb[1] = t / hpb;
    hc[0] = 2 * (t % hpb); hc[1] = hc[0] + 1;
  }

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(s32(&sm.kv_full[s]), 1); mbar_init(s32(&sm.kv_empty[s]), 1); }
    mbar_init(s32(&sm.q_full), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(s32(&sm.s_full[s]), 1);
      mbar_init(s32(&sm.p_full[s]), 128);
      mbar_init(s32(&sm.pv_done[s]), 1);
    }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 4 && lane == 0) {
    // key list: entries of the first half's block, then what only the second half adds
    const int32_t* row0 = block_idx + ((long long)u * g.m + hb[0]) * g.topk;
    int n = attended_list(g, row0, hb[0], sm.ids, status);
    for (int e = 0; e < n; ++e) sm.mask[e] = g.cpb == 1 ? 1 : 3;
    if (g.cpb == 1 && hvalid1) {
      const int32_t* row1 = block_idx + ((long long)u * g.m + hb[1]) * g.topk;
      int n1 = attended_list(g, row1, hb[1], sm.tmp, status);
      const int n0 = n;
      for (int e = 0; e < n1; ++e) {
        int id = sm.tmp[e], pos = -1;
        for (int a = 0; a < n0; ++a) pos = sm.ids[a] == id ? a : pos;
        if (pos >= 0) sm.mask[pos] |= 2;
        else { sm.ids[n] = id; sm.mask[n] = 2; ++n; }
      }
    }
    sm.nlist = n;
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
      mbar_expect_tx(s32(&sm.q_full), 2 * kTile);
      for (int h = 0; h < 2; ++h) {
        int by = hb[h] / g.nbw, bx = hb[h] - by * g.nbw;
        tma_load_4d(s32(sm.q + h * kTile), &map_q, s32(&sm.q_full), 0, bx * g.bw, by * g.bh + hc[h] * g.crows, u);
      }
      for (int it = 0; it < nch; ++it) {
        const int st = it % NSTAGE, j = sm.ids[it / g.cpb], c = it % g.cpb;
        if (!mbar_wait(s32(&sm.kv_empty[st]), ((it / NSTAGE) & 1) ^ 1, abort, status)) break;
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
        const uint64_t kdesc = smem_desc(s32(sm.kv[it % NSTAGE][0]));
        const uint32_t d = tmem + kColS + (it & 1) * 64;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma_ss(d, qdesc + 2 * kk, kdesc + 2 * kk, idesc_qk, kk > 0);
        tc_commit(s32(&sm.s_full[it & 1]));
      };
      if (ok && nch > 0) {
        ok = mbar_wait(s32(&sm.kv_full[0]), 0, abort, status);
        if (ok) { tc_fence_after(); issue_qk(0); }
      }
      for (int it = 0; ok && it < nch; ++it) {
        if (it + 1 < nch) {
          ok = mbar_wait(s32(&sm.kv_full[(it + 1) % NSTAGE]), ((it + 1) / NSTAGE) & 1, abort, status);
          if (ok && it >= 1) ok = mbar_wait(s32(&sm.pv_done[(it + 1) & 1]), ((it - 1) >> 1) & 1, abort, status);
          if (!ok) break;
          tc_fence_after();
          issue_qk(it + 1);
        }
        ok = mbar_wait(s32(&sm.p_full[it & 1]), (it >> 1) & 1, abort, status);
        if (!ok) break;
        tc_fence_after();
        const uint64_t vdesc = smem_desc(s32(sm.kv[it % NSTAGE][1]));
        const uint32_t p = tmem + kColS + (it & 1) * 64;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_ts(tmem + kColO, p + 8 * kk, vdesc + (uint64_t)((2048 * kk) >> 4), idesc_pv, (it > 0 || kk > 0));
        tc_commit(s32(&sm.kv_empty[it % NSTAGE]));
        tc_commit(s32(&sm.pv_done[it & 1]));
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax, then epilogue
    const int h = warp >> 1;  // which 64-row half this warp's rows belong to
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int it = 0; it < nch; ++it) {
      const int sb = it & 1;
      ok = mbar_wait(s32(&sm.s_full[sb]), (it >> 1) & 1, abort, status);
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
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 64; ++c) mx = fmaxf(mx, __uint_as_float(sr[c]));
        mx *= g.scale_log2;  // scale > 0, so the maximum commutes with it
        if (m_ref == -INFINITY) {
          m_ref = mx;
        } else if (mx > m_ref + kRescaleThreshold) {
          need = true;
          alpha = ex2(m_ref - mx);
          m_ref = mx;
          l *= alpha;
        }
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 64; c += 2) {
          float p0 = ex2(fmaf(__uint_as_float(sr[c]), g.scale_log2, -m_ref));
          float p1 = ex2(fmaf(__uint_as_float(sr[c + 1]), g.scale_log2, -m_ref));
          sum += p0 + p1;
          __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
          pk[c >> 1] = *reinterpret_cast<uint32_t*>(&pb);
        }
        l += sum;
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) pk[c] = 0u;
      }
      tmem_st32<0>(ts, pk);
      if (__any_sync(0xffffffffu, need)) {
        // the accumulator may only be touched between P V products
        if (it > 0) {
          ok = mbar_wait(s32(&sm.pv_done[(it - 1) & 1]), ((it - 1) >> 1) & 1, abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t to = tmem + lane_off + kColO;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          uint32_t ov[32];
          tmem_ld32<0>(to + 32 * part, ov);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
          tmem_st32<0>(to + 32 * part, ov);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(s32(&sm.p_full[sb]));
    }
    if (ok && nch > 0) {
      const int last = nch - 1;
      ok = mbar_wait(s32(&sm.pv_done[last & 1]), (last >> 1) & 1, abort, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && nch > 0 && (h == 0 || hvalid1)) {
      tc_fence_after();
      const int e = tid & 63;
      const long long tok = (long long)u * g.N + chunk_token(g, hb[h], hc[h], e);
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

int launch_fwd_tc(const HostCtx& c, const void* q, const void* k, const void* v, const int32_t* block_idx, void* o,
                  float* lse) {
  const Geo& g = c.g;
  if (!(g.cpb == 1 || g.cpb % 2 == 0)) return MOSAIC_E_UNSUPPORTED;
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, q, g) || !make_map(&mk, k, g) || !make_map(&mv, v, g)) return MOSAIC_E_CUDA;
  const size_t smem = sizeof(SmemTC) + 1024;
  if (cudaFuncSetAttribute(fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return MOSAIC_E_CUDA;
  const int tiles_per_unit = g.cpb == 1 ? (g.m + 1) / 2 : g.m * (g.cpb / 2);
  const long long grid = (long long)g.U * tiles_per_unit;
  fwd_tc_kernel<<<(unsigned)grid, 192, smem, c.stream>>>(g, mq, mk, mv, block_idx, (__nv_bfloat16*)o, lse, c.status,
                                                         tiles_per_unit);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

}  // namespace mosaic
