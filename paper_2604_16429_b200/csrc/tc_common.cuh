// Device and host helpers shared by the tensor-core kernels (tcgen05 + TMEM + TMA): mbarrier waits with a
// bound, TMA loads, MMA issue, TMEM loads and stores, packed fp32 arithmetic, operand descriptors, and the
// planner routines that turn a 256-row work item into its merged, interleaved key list.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"

namespace mosaic {

namespace {

constexpr int kTile = 8192;                      // bytes of one 64 x 64 bf16 chunk
constexpr int kMaxUnion = 4 * kMaxList;          // most entries of an item's merged key list
constexpr int kLists = 4;                        // key lists in flight (the planner runs this far ahead)
#ifdef MOSAIC_TEST_SPIN_CYCLES                   // test build only: a short bound, so that a wait that nothing ends runs out quickly
constexpr long long kSpinCycles = MOSAIC_TEST_SPIN_CYCLES;
#else
constexpr long long kSpinCycles = 4000000000ll;  // bound of a single wait (~2 s)
#endif
constexpr uint32_t kSuspendHintNs = 20000;       // longest park of one mbarrier poll

struct ItemInfo {
  int n;        // entries of the merged list; -1 = no more work
  int unit;     // (batch, head) unit
  int hvalid;   // bit h: half h exists
  int hb[4];    // query block of half h
  int hc[4];    // 64-token chunk of that block
  int more;     // 1: the item's list continues in the next list buffer (lists longer than a buffer)
  int kvunit;   // key-stationary kernel: the key/value unit of the item's tile (`unit` is the query unit of this buffer's list)
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
// One poll.  The time hint lets the hardware park the thread for up to that long (it wakes as soon as the
// phase completes), so warps that wait do not take issue slots from warps that work.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
      : "memory");
  return ok != 0;
}
// Non-blocking test of a phase.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false after the limit (status recorded) or once another thread aborted.
// The clock and the abort flag are looked at only every 64 polls to keep the poll loop light.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort, status);
}

// Abort path only: a bounded wait for phase `parity` of `bar` that records nothing.  After a failed wait the roles
// leave their loops with copies and tensor-core work possibly still in flight; the producer waits on the barriers it
// armed and each MMA issuer commits and waits once more, so that shared memory and TMEM are released only after
// everything that was issued has landed or run out of this (second, shorter) bound.
constexpr long long kDrainCycles = 4000000;  // about 2 ms per barrier
__device__ __forceinline__ bool mbar_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > kDrainCycles) return false;
  return true;
}
// Warp-wide wait: lane 0 polls, the warp learns the outcome and synchronises (polls by all 32 lanes serialise on the
// barrier word and cost several times as much).  What lane 0 acquired is visible to the warp after the barrier.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort, int* status, int lane) {
  bool ok = true;
  if (lane == 0) ok = mbar_wait(bar, parity, abort, status);
  ok = __all_sync(0xffffffffu, ok);
  __syncwarp();
  return ok;
}
__device__ __forceinline__ bool warp_test(uint32_t bar, uint32_t parity, int lane) {
  bool ok = true;
  if (lane == 0) ok = mbar_test(bar, parity);
  ok = __all_sync(0xffffffffu, ok);
  __syncwarp();
  return ok;
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
// One thread's tensor-core work issued so far has completed (or the bound ran out): commit to a barrier of its
// own (count 1, never used before) and wait for it.
__device__ __forceinline__ void mma_drain(uint32_t bar) {
  tc_commit(bar);
  mbar_drain(bar, 0);
}
// CTA prologue and epilogue that the tensor-core kernels share.  After the barriers are initialised (by one thread,
// followed by `cta_publish_barriers`), `alloc_warp` takes the whole of the SM's tensor memory and every thread
// reads its base address; at the end the same warp gives it back once every role has left its loop.
__device__ __forceinline__ void cta_publish_barriers() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ uint32_t cta_tmem_alloc(bool alloc_warp, uint32_t* slot, uint32_t cols) {
  __syncthreads();  // barrier initialisation is visible to every thread
  if (alloc_warp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(slot)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  return *slot;
}
__device__ __forceinline__ void cta_tmem_free(bool alloc_warp, uint32_t tmem, uint32_t cols) {
  tc_fence_before();
  __syncthreads();
  if (alloc_warp) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
  }
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

#define MOSAIC_R16(r, o)                                                                                          \
  "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]),  \
      "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]), "=r"(r[o + 12]),           \
      "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15])
#define MOSAIC_W16(r, o)                                                                                     \
  "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]),    \
      "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), "r"(r[o + 12]),            \
      "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15])

// 32 consecutive 32-bit TMEM columns of this thread's lane -> registers r[0..31]
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
      "%15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : MOSAIC_R16(r, 0), MOSAIC_R16(r, 16)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
      "%15}, [%16];"
      : MOSAIC_R16(r, 0)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
      "%15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      MOSAIC_W16(r, 0), MOSAIC_W16(r, 16)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
      "%15, %16};" ::"r"(taddr),
      MOSAIC_W16(r, 0)
      : "memory");
}

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
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
// two floats -> two 16-bit operands in one word (bf16, or binary16 when F16)
template <bool F16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  uint32_t r;
  if (F16) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// 2^x for two values on the FMA pipe instead of the MUFU pipe (which caps the softmax at d = 64):
// x = n + f with n = round(x), |f| <= 1/2 (adding 1.5 * 2^23 leaves n in the low mantissa bits),
// 2^f by a cubic fitted to a maximum relative error of 1.0e-4 (P is rounded to bf16, 2^-9, afterwards),
// and 2^n by adding n to the exponent field.  Inputs are clamped at -125 so the exponent stays normal.
__device__ __forceinline__ void ex2_poly2(uint64_t x2, float& p0, float& p1) {
  float x0, x1;
  unpack2(x2, x0, x1);
  const uint64_t xc = pack2(fmaxf(x0, -125.f), fmaxf(x1, -125.f));
  const uint64_t t = add2(xc, pack2(12582912.f, 12582912.f));
  const uint64_t n = add2(t, pack2(-12582912.f, -12582912.f));
  const uint64_t f = fma2(n, pack2(-1.f, -1.f), xc);
  uint64_t p = fma2(f, pack2(0.05500893f, 0.05500893f), pack2(0.24221095f, 0.24221095f));
  p = fma2(p, f, pack2(0.6932829f, 0.6932829f));
  p = fma2(p, f, pack2(1.f, 1.f));
  float t0, t1, q0, q1;
  unpack2(t, t0, t1);
  unpack2(p, q0, q1);
  p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
  p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
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
// Instruction descriptor: 16-bit x 16-bit -> fp32 (both operands bf16, or both binary16 when f16), M = 128,
// N = 64 unless given.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major, uint32_t n = 64u, bool f16 = false) {
  return (1u << 4) | ((f16 ? 0u : 1u) << 7) | ((f16 ? 0u : 1u) << 10) | ((b_mn_major ? 1u : 0u) << 16) |
         ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// The four halves of work item `it` (index inside the unit).  Missing halves repeat half 0 (their rows
// are computed with every key masked and never stored).  Returns the bit set of existing halves.
__device__ __forceinline__ int item_halves(const Geo& g, int it, int (&hb)[4], int (&hc)[4]) {
  int valid = 0;
  if (g.cpb == 1) {
    const int ntx = (g.nbw + 1) >> 1, n_main = (g.nbh >> 1) * ntx;
    if (it < n_main) {  // 2 x 2 group
      const int gy = it / ntx, tx = it - gy * ntx;
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const int by = 2 * gy + (h >> 1), bx = 2 * tx + (h & 1);
        hb[h] = by * g.nbw + bx;
        hc[h] = 0;
        valid |= (bx < g.nbw) << h;
      }
    } else {            // odd last block row: 1 x 4 group
      const int bx0 = 4 * (it - n_main);
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        hb[h] = (g.nbh - 1) * g.nbw + bx0 + h;
        hc[h] = 0;
        valid |= (bx0 + h < g.nbw) << h;
      }
    }
  } else if (g.cpb == 2) {  // two neighbouring 128-token blocks: side by side, or one above the other in a one-column grid
    if (g.nbw > 1) {
      const int ntx = (g.nbw + 1) >> 1, by = it / ntx, tx = it - by * ntx;
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const int bx = 2 * tx + (h >> 1);
        hb[h] = by * g.nbw + bx;
        hc[h] = h & 1;
        valid |= (bx < g.nbw) << h;
      }
    } else {
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const int by = 2 * it + (h >> 1);
        hb[h] = by;
        hc[h] = h & 1;
        valid |= (by < g.nbh) << h;
      }
    }
  } else {                  // four chunks of one block
    const int ipb = (g.cpb + 3) >> 2, blk = it / ipb, c0 = 4 * (it - blk * ipb);
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      hb[h] = blk;
      hc[h] = c0 + h;
      valid |= (c0 + h < g.cpb) << h;
    }
  }
#pragma unroll
  for (int h = 1; h < 4; ++h)
    if (!((valid >> h) & 1)) { hb[h] = hb[0]; hc[h] = hc[0]; }
  return valid;
}

// Warp-cooperative attended list of query block i (local set, then valid selected ids) written to
// ids[n0..); returns the new count.  `j` is this lane's entry of the block's row of block_idx (-1 beyond top-k).
__device__ __forceinline__ int warp_attended(const Geo& g, int j, int i, int* ids, int n0, int lane, int* status) {
  const int by = i / g.nbw, bx = i - by * g.nbw;
  int id = -1 - lane;  // lanes without a block hold distinct negative values
  int nl;
  if (g.local_groups) {   // the aligned group of rlat x rlon blocks that holds block i (ragged at the grid's edge)
    nl = g.local_off ? 0 : g.rlat * g.rlon;
    if (lane < nl) {
      const int dy = lane / g.rlon, dx = lane - dy * g.rlon;
      const int y = (by / g.rlat) * g.rlat + dy, x = (bx / g.rlon) * g.rlon + dx;
      if (y < g.nbh && x < g.nbw) id = y * g.nbw + x;
    }
  } else {
    const int wl = 2 * g.rlon + 1;
    nl = g.local_off ? 0 : (2 * g.rlat + 1) * wl;
    if (lane < nl) {
      const int dy = lane / wl - g.rlat, dx = lane - (lane / wl) * wl - g.rlon;
      const int y = min(max(by + dy, 0), g.nbh - 1);
      int x = (bx + dx) % g.nbw;
      x += x < 0 ? g.nbw : 0;
      id = y * g.nbw + x;
    }
  }
  const unsigned same = __match_any_sync(0xffffffffu, id);
  const bool keep = id >= 0 && (__ffs(same) - 1) == lane;  // first occurrence of a block
  const unsigned km = __ballot_sync(0xffffffffu, keep);
  if (keep) ids[n0 + __popc(km & ((1u << lane) - 1u))] = id;
  int n = n0 + __popc(km);
  // selected ids outside [-1, m), inside the local set (attended already) or repeated in the row: skipped, reported
  const unsigned twins = __match_any_sync(0xffffffffu, j);
  if (j != -1 && (j < 0 || j >= g.m || is_local(g, i, j) || (__ffs(twins) - 1) != lane)) {
    set_status(status, MOSAIC_E_DEVICE_BAD_INDEX);
    j = -1;
  }
  const unsigned sm_ = __ballot_sync(0xffffffffu, j >= 0);
  if (j >= 0) ids[n + __popc(sm_ & ((1u << lane) - 1u))] = j;
  return n + __popc(sm_);
}

// Merge the attended list of query block `blk` into the item's list (ids/mask, n entries so far):
// entries already present get `bits` OR-ed into their mask, new ones are appended.  Returns the new n.
// `jsel` is this lane's entry of the block's row of block_idx (-1 beyond top-k).
__device__ __forceinline__ int merge_block(const Geo& g, int jsel, int blk, unsigned char bits, int* ids,
                                           unsigned char* mask, int n, int lane, int* status) {
  const int n0 = n;
  const int nb = warp_attended(g, jsel, blk, ids, n0, lane, status) - n0;  // staged behind the list
  __syncwarp();
  if (n0 == 0) {
    for (int e = lane; e < nb; e += 32) mask[e] = bits;
    __syncwarp();
    return nb;
  }
  int mine[2], pos[2];  // at most 64 entries per block: two per lane
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int e = lane + 32 * r;
    mine[r] = e < nb ? ids[n0 + e] : -1;
    pos[r] = -1;
  }
#pragma unroll 8
  for (int a = 0; a < n0; ++a) {
    const int id = ids[a];
    pos[0] = id == mine[0] ? a : pos[0];
    pos[1] = id == mine[1] ? a : pos[1];
  }
  __syncwarp();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const bool have = mine[r] >= 0, fresh = have && pos[r] < 0;
    if (have && pos[r] >= 0) mask[pos[r]] |= bits;
    const unsigned fm = __ballot_sync(0xffffffffu, fresh);
    if (fresh) {
      const int at = n + __popc(fm & ((1u << lane) - 1u));
      ids[at] = mine[r];
      mask[at] = bits;
    }
    n += __popc(fm);
    __syncwarp();
  }
  return n;
}

// One lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

// Reorder a merged key list so that both tiles, and both 64-row halves of a tile, find work all along it.
// Entries fall into seven classes by who attends them: tile 0 only (upper half, lower half, both halves), both
// tiles, tile 1 only (upper, lower, both).  The k-th entry of a class of n gets the fractional position
// (8k + class) / (8n), so every class is spread evenly; in particular products that only the upper half of a
// tile attends alternate with products only its lower half attends, and since S is double-buffered the idle
// half's warps run ahead into the next product.  The order of a softmax sum does not matter to the result
// beyond rounding; the order is a function of the list alone.
__device__ __forceinline__ int list_class(unsigned m) {
  const unsigned t0 = m & 3u, t1 = (m >> 2) & 3u;
  return t1 == 0u ? (int)t0 - 1 : t0 == 0u ? 3 + (int)t1 : 3;
}
__device__ __forceinline__ void interleave_tiles(const int* sid, const unsigned char* smask, int n, int* did,
                                                 unsigned char* dmask, int lane) {
  constexpr int NC = 7;
  int cnt[NC];
#pragma unroll
  for (int y = 0; y < NC; ++y) cnt[y] = 0;
  for (int e0 = 0; e0 < n; e0 += 32) {
    const int e = e0 + lane;
    const int cls = e < n ? list_class(smask[e]) : -1;
#pragma unroll
    for (int y = 0; y < NC; ++y) cnt[y] += __popc(__ballot_sync(0xffffffffu, cls == y));
  }
  int base[NC];
#pragma unroll
  for (int y = 0; y < NC; ++y) base[y] = 0;
  for (int e0 = 0; e0 < n; e0 += 32) {
    const int e = e0 + lane;
    const unsigned m = e < n ? smask[e] : 0u;
    const int cls = e < n ? list_class(m) : -1;
    const unsigned lower = (1u << lane) - 1u;
    int k = 0, nx = 1;
#pragma unroll
    for (int y = 0; y < NC; ++y) {
      const unsigned by = __ballot_sync(0xffffffffu, cls == y);
      if (cls == y) { k = base[y] + __popc(by & lower); nx = cnt[y]; }
      base[y] += __popc(by);
    }
    if (e < n) {
      int pos = k;
#pragma unroll
      for (int y = 0; y < NC; ++y) {
        const int ny = cnt[y];
        if (y == cls || ny == 0) continue;
        // entries j of class y that come first: (8j + y) nx < (8k + cls) ny, ties to the lower class
        const int R = (8 * k + cls) * ny - y * nx;
        int c = 0;
        if (y < cls) c = R >= 0 ? R / (8 * nx) + 1 : 0;
        else c = R > 0 ? (R + 8 * nx - 1) / (8 * nx) : 0;
        pos += min(c, ny);
      }
      did[pos] = sid[e];
      dmask[pos] = (unsigned char)m;
    }
  }
  __syncwarp();
}

// Planner warp: draws work items from the queue (the first item of a CTA is its own index) and builds each
// item's merged, interleaved key list one or more items ahead of the warps that consume it.  `SM` is the
// kernel's shared-memory struct (info, ids, mask, tmp_ids, tmp_mask, list_full, list_empty).
template <class SM>
__device__ __forceinline__ void planner_loop(SM& sm, const Geo& g, const int32_t* __restrict__ block_idx,
                                             int* work_counter, int ipu, int total_items, int lane,
                                             volatile int* abort, int* status) {
  for (int it = 0;; ++it) {
    const int buf = it % kLists;
    int item = 0;
    // the first item of a CTA is its own index; later ones come from the queue, which counts from 0
    if (lane == 0) item = it == 0 ? (int)blockIdx.x : atomicAdd(work_counter, 1) + (int)gridDim.x;
    item = __shfl_sync(0xffffffffu, item, 0);
    bool ok = true;
    if (lane == 0) ok = mbar_wait(s32(&sm.list_empty[buf]), ((it / kLists) & 1) ^ 1, abort, status);
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) break;
    if (item >= total_items) {
      if (lane == 0) { sm.info[buf].n = -1; mbar_arrive(s32(&sm.list_full[buf])); }
      break;
    }
    const int u = item / ipu;
    int hb[4], hc[4];
    const int valid = item_halves(g, item - u * ipu, hb, hc);
    int jsel[4];  // the four rows of block_idx, fetched together
#pragma unroll
    for (int h = 0; h < 4; ++h)
      jsel[h] = lane < g.topk ? __ldg(block_idx + ((long long)u * g.m + hb[h]) * g.topk + lane) : -1;
    int n = 0;
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      if (!((valid >> h) & 1)) continue;
      bool first = true;  // first half of its block: merge the block's list once, for all its halves
      unsigned char bits = 0;
#pragma unroll
      for (int h2 = 0; h2 < 4; ++h2) {
        if (((valid >> h2) & 1) && hb[h2] == hb[h]) {
          if (h2 < h) first = false;
          bits |= (unsigned char)(1 << h2);
        }
      }
      if (first) n = merge_block(g, jsel[h], hb[h], bits, sm.tmp_ids, sm.tmp_mask, n, lane, status);
    }
    if (g.cpb == 1 && valid == 0xF) {
      // Four different query blocks: which two share a 128-row tile is free.  Take the pairing whose tiles have
      // the most entries in common (fewest products with a masked half); ties keep the first pairing.
      int o01 = 0, o23 = 0, o02 = 0, o13 = 0, o03 = 0, o12 = 0;
      for (int e0 = 0; e0 < n; e0 += 32) {
        const unsigned mk = e0 + lane < n ? sm.tmp_mask[e0 + lane] : 0u;
        o01 += __popc(__ballot_sync(0xffffffffu, (mk & 3u) == 3u));
        o23 += __popc(__ballot_sync(0xffffffffu, (mk & 12u) == 12u));
        o02 += __popc(__ballot_sync(0xffffffffu, (mk & 5u) == 5u));
        o13 += __popc(__ballot_sync(0xffffffffu, (mk & 10u) == 10u));
        o03 += __popc(__ballot_sync(0xffffffffu, (mk & 9u) == 9u));
        o12 += __popc(__ballot_sync(0xffffffffu, (mk & 6u) == 6u));
      }
      const int s0 = o01 + o23, s1 = o02 + o13, s2 = o03 + o12;
      const int pick = (s1 > s0 && s1 >= s2) ? 1 : (s2 > s0 && s2 > s1) ? 2 : 0;
      if (pick != 0) {
        // new half k is old half perm[k]: (0,2,1,3) pairs the blocks vertically, (0,3,1,2) diagonally
        const int p1 = pick == 1 ? 2 : 3, p2 = 1, p3 = pick == 1 ? 3 : 2;
        for (int e = lane; e < n; e += 32) {
          const unsigned mk = sm.tmp_mask[e];
          sm.tmp_mask[e] = (unsigned char)((mk & 1u) | (((mk >> p1) & 1u) << 1) | (((mk >> p2) & 1u) << 2) |
                                           (((mk >> p3) & 1u) << 3));
        }
        const int b1 = hb[p1], b2 = hb[p2], b3 = hb[p3], c1 = hc[p1], c2 = hc[p2], c3 = hc[p3];
        hb[1] = b1; hb[2] = b2; hb[3] = b3;
        hc[1] = c1; hc[2] = c2; hc[3] = c3;
        __syncwarp();
      }
    }
    interleave_tiles(sm.tmp_ids, sm.tmp_mask, n, sm.ids[buf], sm.mask[buf], lane);
    if (lane == 0) {
      ItemInfo& inf = sm.info[buf];
      inf.n = n; inf.unit = u; inf.hvalid = valid; inf.more = 0;
#pragma unroll
      for (int h = 0; h < 4; ++h) { inf.hb[h] = hb[h]; inf.hc[h] = hc[h]; }
    }
    __syncwarp();
#ifdef MOSAIC_TEST_WITHHOLD_FIRST_LIST  // test build only: the CTA's first list is never published, so every consumer's wait runs out
    if (it == 0) continue;
#endif
    if (lane == 0) mbar_arrive(s32(&sm.list_full[buf]));
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], "
      "[%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
}  // namespace

// ---- host side (tmap.cu) -------------------------------------------------------------------
// TMA descriptors are cached per (device, base pointer, geometry), so a call that sees the same tensors
// again encodes nothing.
// [units, nlat, nlon, d] bf16 view, box = one 64-token chunk {d, bw, 64/bw, 1}, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, const Geo& g, int units);
// [U, nlat, nlon] fp32 view (one value per token), box = the 64 tokens of one chunk {bw, 64/bw, 1}, no swizzle.
bool make_map_rows(CUtensorMap* map, const void* base, const Geo& g);
// Current device, its SM count (cached), and the opt-in to `smem` bytes of dynamic shared memory for `func`
// (set once per device; `done` is the caller's per-kernel bit set of devices already configured).
int launch_setup(const void* func, size_t smem, unsigned long long* done, int* sms);

}  // namespace mosaic
