// dK and dV of the block-sparse attention backward on Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// Paper, appendix "Block-sparse attention implementation", paragraph "Kernel Design": the gradients of
// keys and values are formed per key/value block by visiting only the query blocks connected to it.
// With P = exp(scale * Q K^T - LSE), dP = dO V^T, D = rowsum(dO o O), dS = P o (dP - D):
//   dV_j = sum_i P_ij^T dO_i ,   dK_j = scale * sum_i dS_ij^T Q_i      (i over the query blocks connected to j)
// The connected query blocks of key block j are its local neighbours (the neighbourhood relation is
// symmetric, so they follow from geometry) and the query blocks that selected j (transposed pattern, CSR).
//
// Key/value-stationary: a persistent CTA per SM draws items of 128 KEY rows (one tile = two 64-row halves,
// each half one 64-token chunk of a key block; tile t of the 256-row items the other kernels use).  The K
// and V tiles stay in shared memory; query-side chunks (Q, dO, and per query row -LSE*log2(e) and -D)
// stream through a ring of slots, two chunks (a pair of products) per slot.  Per pair:  S^T = K Q^T and
// dP^T = V dO^T for both chunks at once (eight MMAs with N = 128: the two chunks' Q tiles lie back to back in
// the slot, their S^T buffers side by side in TMEM); two groups of row threads (TMEM lane = key row, two threads
// per row and group, each half of the query columns; the backward has no reduction along a row, so they never
// talk), one group per chunk, pull their share into registers and hand the buffers back at once, so the next
// pair's S^T and dP^T are computed while they form P^T and dS^T (bf16, own TMEM columns per group); then
// dV += P^T dO and dK += dS^T Q (TMEM A operands, the staged dO and Q chunks as MN-major B operands), issued by
// a second thread as each group finishes.  A list with an odd number of chunks ends in a pair of one.
// Lists: the planner merges the local neighbourhoods of the tile's key blocks (entries carry a mask of the
// halves they are connected to) and appends each block's CSR list; a list longer than a list buffer
// continues in the next buffer (ItemInfo::more).  The order of a list is a function of the pattern alone,
// so the summation order, and with it the result, is deterministic.
// Every mbarrier wait is bounded; on expiry the CTA records MOSAIC_E_DEVICE_TIMEOUT and drains.
#include "tc_common.cuh"

namespace mosaic {

namespace {

constexpr int kSlots = 4;        // ring depth in pairs of query-side chunks
constexpr int kRowWarps = 16;    // two groups of eight: two threads per key row in each
constexpr int kGroupWarps = kRowWarps / 2;
constexpr int kThreads = 32 * (kRowWarps + 4);  // row threads, then TMA producer, two MMA issuers, planner
constexpr int kWProd = kRowWarps, kWMma0 = kRowWarps + 1, kWMma1 = kRowWarps + 2, kWPlan = kRowWarps + 3;
constexpr uint32_t kTmemCols = 512;
// dK, dV accumulators; per chunk of a pair S^T and dP^T (fp32, 64 columns) and P^T and dS^T (bf16 pairs, 32 columns)
constexpr uint32_t kColDK = 0, kColDV = 64, kColS = 128, kColDP = 256, kColP = 384, kColDS = 448;
constexpr uint32_t kChunkBytes = 2 * kTile + 2 * 64 * 4;

struct Slot {
  unsigned char q[2][kTile];     // per chunk 64 query rows x 128 B, swizzled; the two tiles form one 128-row operand
  unsigned char d_o[2][kTile];
  float neg_lse2[2][64];         // -LSE * log2(e) of the chunks' query rows
  float neg_d[2][64];            // -D of the chunks' query rows
};
static_assert(sizeof(Slot) % 1024 == 0, "slots keep the 1024-byte alignment of the swizzled tiles");

struct Smem {
  unsigned char k[2 * kTile];              // 128 key rows x 128 B
  unsigned char v[2 * kTile];
  Slot ring[kSlots];
  unsigned long long ring_full[kSlots], ring_empty[kSlots];
  unsigned long long kv_full, kv_empty, s_full, sdp_free, p_full[2], pv_done, acc_done, acc_free;
  unsigned long long mma_drain_bar[2];  // abort path: completion of each issuer's outstanding products
  unsigned long long list_full[kLists], list_empty[kLists];
  uint32_t tmem_base;
  int abort;
  ItemInfo info[kLists];             // hb/hc/hvalid entries 0 and 1 describe the tile's two halves
  int ids[kLists][kMaxUnion];
  unsigned char mask[kLists][kMaxUnion];
};

// Planner of the key-stationary kernel: per item (tile), the merged local neighbourhoods of its key blocks,
// then each block's list of selecting query blocks, cut into list buffers.
__device__ __forceinline__ void planner_kv_loop(Smem& sm, const Geo& g, const int32_t* __restrict__ csr_off,
                                                const int32_t* __restrict__ csr_q,
                                                const int32_t* __restrict__ order, int* work_counter, int ipu,
                                                int total_items, int lane, volatile int* abort, int* status) {
  int lb = 0;  // list buffers handed out so far
  for (int it = 0;; ++it) {
    int item = 0;
    if (lane == 0) {  // the queue hands out positions of the longest-first order
      const int pos = it == 0 ? (int)blockIdx.x : atomicAdd(work_counter, 1) + (int)gridDim.x;
      item = pos < total_items ? __ldg(order + pos) : total_items;
    }
    item = __shfl_sync(0xffffffffu, item, 0);
    bool ok = true;
    auto acquire = [&]() {  // wait until list buffer lb % kLists is free
      if (lane == 0) ok = mbar_wait(s32(&sm.list_empty[lb % kLists]), ((lb / kLists) & 1) ^ 1, abort, status);
      ok = __shfl_sync(0xffffffffu, ok, 0);
    };
    acquire();
    if (!ok) break;
    if (item >= total_items) {
      if (lane == 0) { sm.info[lb % kLists].n = -1; mbar_arrive(s32(&sm.list_full[lb % kLists])); }
      break;
    }
    // item = 2 * (256-row item) + tile of a key/value unit
    const int i256 = item >> 1, t = item & 1;
    const int u = i256 / ipu;  // key/value unit
    int hb4[4], hc4[4];
    const int valid4 = item_halves(g, i256 - u * ipu, hb4, hc4);
    const int hb[2] = {hb4[2 * t], hb4[2 * t + 1]}, hc[2] = {hc4[2 * t], hc4[2 * t + 1]};
    const int valid = (valid4 >> (2 * t)) & 3;
    const int ratio = g.H / g.Hkv, qu0 = (u / g.Hkv) * g.H + (u - (u / g.Hkv) * g.Hkv) * ratio;
    int n = 0, qu = qu0;  // qu: the query unit whose connected query blocks are being listed
    auto publish = [&](int more) {
      const int buf = lb % kLists;
      if (lane == 0) {
        ItemInfo& inf = sm.info[buf];
        inf.n = n; inf.unit = qu; inf.kvunit = u; inf.hvalid = valid; inf.more = more;
        inf.hb[0] = hb[0]; inf.hb[1] = hb[1]; inf.hc[0] = hc[0]; inf.hc[1] = hc[1];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(s32(&sm.list_full[buf]));
      ++lb;
      n = 0;
    };
    // the two halves are either two key blocks (one bit each) or two chunks of one block (both bits)
    const bool same = (valid == 3) && hb[0] == hb[1];
    const unsigned char bits0 = same ? 3 : 1, bits1 = 2;
    const bool use0 = (valid & 1) != 0, use1 = (valid & 2) != 0 && !same;
    // One pass per query head of the group (grouped-query attention: the tile's dK and dV sum over them); the
    // passes are list buffers of the same item, chained by `more`.
    for (int r = 0; r < ratio && ok; ++r) {
      qu = qu0 + r;
      if (r > 0) {
        acquire();
        if (!ok) break;
      }
      // local neighbourhoods (at most 64 entries per block, merged with masks), straight into the list buffer
      if (use0) n = merge_block(g, -1, hb[0], bits0, sm.ids[lb % kLists], sm.mask[lb % kLists], n, lane, status);
      if (use1) n = merge_block(g, -1, hb[1], bits1, sm.ids[lb % kLists], sm.mask[lb % kLists], n, lane, status);
      // query blocks that selected the key block (ascending ids), appended 32 at a time
      const int32_t* off = csr_off + (long long)qu * (g.m + 1);
      const int32_t* sel = csr_q + (long long)qu * g.m * g.topk;
#pragma unroll
      for (int hh = 0; hh < 2 && ok; ++hh) {
        if (!(hh == 0 ? use0 : use1)) continue;
        const unsigned char bits = hh == 0 ? bits0 : bits1;
        const int s_beg = __ldg(off + hb[hh]), s_end = __ldg(off + hb[hh] + 1);
        for (int base = s_beg; base < s_end && ok; base += 32) {
          if (n + 32 > kMaxUnion) {
            publish(1);
            acquire();
            if (!ok) break;
          }
          const int e = base + lane;
          if (e < s_end) {
            sm.ids[lb % kLists][n + lane] = __ldg(sel + e);
            sm.mask[lb % kLists][n + lane] = bits;
          }
          n += min(32, s_end - base);
          __syncwarp();
        }
      }
      if (!ok) break;
      publish(r + 1 < ratio ? 1 : 0);
    }
    if (!ok) break;
  }
}

}  // namespace

// The items' lists differ in length (a key block that many query blocks selected has a long one), and a long item
// drawn late leaves the other SMs idle at the end.  This kernel orders the items by the number of selecting query
// blocks, longest first, inside windows of consecutive key/value units (the windows keep their order, so that items
// in flight at the same time read the same few units; a window holds at least sixteen items per SM).  One CTA per
// window, counting sort; the place inside a class of equal length is arbitrary, which changes no result: an item
// writes only its own tile, in the order of its own list.
constexpr int kCostBins = 2048;
__global__ void __launch_bounds__(1024) dkdv_order_kernel(const Geo g, const int32_t* __restrict__ csr_off, int ipu,
                                                          int total_items, int window_items,
                                                          int32_t* __restrict__ order, int32_t* __restrict__ bins) {
  __shared__ int hist[kCostBins];
  const int tid = threadIdx.x, lane = tid & 31;
  const int first_item = (int)blockIdx.x * window_items;
  const int end_item = min(total_items, first_item + window_items);
  for (int i = tid; i < kCostBins; i += (int)blockDim.x) hist[i] = 0;
  __syncthreads();
  const int ratio = g.H / g.Hkv;
  for (int item = first_item + tid; item < end_item; item += (int)blockDim.x) {
    const int i256 = item >> 1, t = item & 1, u = i256 / ipu;
    int hb4[4], hc4[4];
    const int valid = (item_halves(g, i256 - u * ipu, hb4, hc4) >> (2 * t)) & 3;
    const int b0 = hb4[2 * t], b1 = hb4[2 * t + 1];
    const bool use0 = (valid & 1) != 0, use1 = (valid & 2) != 0 && !(valid == 3 && b0 == b1);
    const int qu0 = (u / g.Hkv) * g.H + (u - (u / g.Hkv) * g.Hkv) * ratio;
    int cost = 0;
    for (int r = 0; r < ratio; ++r) {
      const int32_t* off = csr_off + (long long)(qu0 + r) * (g.m + 1);
      if (use0) cost += __ldg(off + b0 + 1) - __ldg(off + b0);
      if (use1) cost += __ldg(off + b1 + 1) - __ldg(off + b1);
    }
    const int bin = cost < 0 ? 0 : (cost < kCostBins ? cost : kCostBins - 1);
    bins[item] = bin;
    atomicAdd(&hist[bin], 1);
  }
  __syncthreads();
  if (tid < 32) {  // first place of each class, classes in descending order
    int carry = 0;
    for (int base = kCostBins - 32; base >= 0; base -= 32) {
      const int b = base + 31 - lane;  // lane 0 takes the highest class of the chunk
      const int v = hist[b];
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int nb = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += nb;
      }
      hist[b] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
  }
  __syncthreads();
  for (int item = first_item + tid; item < end_item; item += (int)blockDim.x)
    order[first_item + atomicAdd(&hist[bins[item]], 1)] = item;
}

template <bool F16>
__global__ void __launch_bounds__(kThreads, 1)
    dkdv_tc_kernel(const Geo g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                   const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const __grid_constant__ CUtensorMap map_nlse, const __grid_constant__ CUtensorMap map_nd,
                   const int32_t* __restrict__ csr_off, const int32_t* __restrict__ csr_q,
                   const int32_t* __restrict__ order, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, int* status, int* work_counter,
                   int ipu, int total_items) {
  extern __shared__ unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(s32(&sm.ring_full[s]), 1); mbar_init(s32(&sm.ring_empty[s]), 1); }
    mbar_init(s32(&sm.kv_full), 1);
    mbar_init(s32(&sm.kv_empty), 1);
    mbar_init(s32(&sm.s_full), 1);
    mbar_init(s32(&sm.sdp_free), 32 * kRowWarps);
    mbar_init(s32(&sm.p_full[0]), 32 * kGroupWarps);
    mbar_init(s32(&sm.p_full[1]), 32 * kGroupWarps);
    mbar_init(s32(&sm.pv_done), 1);
    mbar_init(s32(&sm.acc_done), 1);
    mbar_init(s32(&sm.acc_free), kRowWarps);
    mbar_init(s32(&sm.mma_drain_bar[0]), 1);
    mbar_init(s32(&sm.mma_drain_bar[1]), 1);
    for (int i = 0; i < kLists; ++i) {
      mbar_init(s32(&sm.list_full[i]), 1);
      mbar_init(s32(&sm.list_empty[i]), kRowWarps + 3);  // row-thread warps + 2 MMA issuers + TMA producer
    }
    sm.abort = 0;
    cta_publish_barriers();
  }
  const uint32_t tmem = cta_tmem_alloc(warp == kWMma0, &sm.tmem_base, kTmemCols);
  volatile int* abort = &sm.abort;

  // Every role walks the same sequence: list buffers, and inside a buffer its n * cpb chunks two at a time.
  // `pr` counts pairs (ring slot pr % kSlots, phase of the per-pair barriers).
  if (warp == kWPlan) {
    planner_kv_loop(sm, g, csr_off, csr_q, order, work_counter, ipu, total_items, lane, abort, status);
  } else if (warp == kWProd) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      long long pr = 0;
      int items = 0;       // items started so far (phase of kv_full / kv_empty)
      bool ok = true, fresh = true;  // fresh: the next list buffer starts a new item
      for (int lb = 0; ok; ++lb) {
        const int buf = lb % kLists;
        ok = mbar_wait(s32(&sm.list_full[buf]), (lb / kLists) & 1, abort, status);
        if (!ok) break;
        const ItemInfo& inf = sm.info[buf];
        const int n = inf.n, u = inf.unit;
        if (n < 0) break;
        if (fresh) {
          // K and V tiles: free once every product of the previous item has completed
          ok = mbar_wait(s32(&sm.kv_empty), (items & 1) ^ 1, abort, status);
          if (!ok) break;
          mbar_expect_tx(s32(&sm.kv_full), 4 * kTile);
          for (int hh = 0; hh < 2; ++hh) {
            const int by = inf.hb[hh] / g.nbw, bx = inf.hb[hh] - by * g.nbw;
            tma_load_4d(s32(sm.k + hh * kTile), &map_k, s32(&sm.kv_full), 0, bx * g.bw,
                        by * g.bh + inf.hc[hh] * g.crows, inf.kvunit);
            tma_load_4d(s32(sm.v + hh * kTile), &map_v, s32(&sm.kv_full), 0, bx * g.bw,
                        by * g.bh + inf.hc[hh] * g.crows, inf.kvunit);
          }
          ++items;
        }
        fresh = inf.more == 0;
        const int chunks = n * g.cpb;
        for (int p0 = 0; p0 < chunks && ok; p0 += 2, ++pr) {
          const int slot = (int)(pr % kSlots), np = min(2, chunks - p0);
          ok = mbar_wait(s32(&sm.ring_empty[slot]), (uint32_t)((pr / kSlots) & 1) ^ 1, abort, status);
          if (!ok) break;
          Slot& sl = sm.ring[slot];
          const uint32_t bar = s32(&sm.ring_full[slot]);
          mbar_expect_tx(bar, np * kChunkBytes);
          for (int h = 0; h < np; ++h) {
            const int e = (p0 + h) / g.cpb, c = (p0 + h) - e * g.cpb;
            const int i = sm.ids[buf][e], by = i / g.nbw, bx = i - by * g.nbw;
            const int x0 = bx * g.bw, y0 = by * g.bh + c * g.crows;
            tma_load_4d(s32(sl.q[h]), &map_q, bar, 0, x0, y0, u);
            tma_load_4d(s32(sl.d_o[h]), &map_do, bar, 0, x0, y0, u);
            tma_load_3d(s32(sl.neg_lse2[h]), &map_nlse, bar, x0, y0, u);
            tma_load_3d(s32(sl.neg_d[h]), &map_nd, bar, x0, y0, u);
          }
        }
        if (ok) mbar_arrive(s32(&sm.list_empty[buf]));
      }
      if (*abort) {  // copies this thread issued must land before the CTA's memory is released
        const long long first = pr > kSlots ? pr - kSlots : 0;
        for (long long s = first; s < pr; ++s) mbar_drain(s32(&sm.ring_full[s % kSlots]), (uint32_t)((s / kSlots) & 1));
        if (items > 0) mbar_drain(s32(&sm.kv_full), (uint32_t)((items - 1) & 1));
      } else {       // drain: the last uses of every ring slot have been released
        const long long first = pr > kSlots ? pr - kSlots : 0;
        for (long long s = first; s < pr; ++s)
          if (!mbar_wait(s32(&sm.ring_empty[s % kSlots]), (uint32_t)((s / kSlots) & 1), abort, status)) break;
      }
    }
  } else if (warp == kWMma0) {
    // ------------------------------------------------------------- issuer of S^T = K Q^T and dP^T = V dO^T (one thread)
    // The buffers may be overwritten once the row threads hold the previous pair in registers, so this thread runs
    // one pair ahead of their arithmetic.
    if (lane == 0) {
      constexpr uint32_t idesc1 = make_idesc(false, 64u, F16), idesc2 = make_idesc(false, 128u, F16);
      const uint64_t kdesc = smem_desc(s32(sm.k)), vdesc = smem_desc(s32(sm.v));
      long long pr = 0;
      int items = 0;
      bool ok = true, fresh = true;
      for (int lb = 0; ok; ++lb) {
        const int buf = lb % kLists;
        ok = mbar_wait(s32(&sm.list_full[buf]), (lb / kLists) & 1, abort, status);
        if (!ok) break;
        const int n = sm.info[buf].n;
        if (n < 0) break;
        const bool more = sm.info[buf].more != 0;
        if (fresh) {
          ok = mbar_wait(s32(&sm.kv_full), items & 1, abort, status);
          if (!ok) break;
          ++items;
        }
        fresh = !more;
        const int chunks = n * g.cpb;
        for (int p0 = 0; p0 < chunks && ok; p0 += 2, ++pr) {
          const int slot = (int)(pr % kSlots);
          ok = mbar_wait(s32(&sm.ring_full[slot]), (uint32_t)((pr / kSlots) & 1), abort, status);
          if (ok && pr > 0) ok = mbar_wait(s32(&sm.sdp_free), (uint32_t)((pr - 1) & 1), abort, status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t idesc = chunks - p0 >= 2 ? idesc2 : idesc1;
          const uint64_t qdesc = smem_desc(s32(sm.ring[slot].q[0])), dodesc = smem_desc(s32(sm.ring[slot].d_o[0]));
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) umma_ss(tmem + kColS, kdesc + 2 * kk, qdesc + 2 * kk, idesc, kk > 0);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) umma_ss(tmem + kColDP, vdesc + 2 * kk, dodesc + 2 * kk, idesc, kk > 0);
          tc_commit(s32(&sm.s_full));
        }
        // the K and V tiles are read by this thread's products only: all of the item's are behind this commit
        if (ok && !more) tc_commit(s32(&sm.kv_empty));
        if (ok) mbar_arrive(s32(&sm.list_empty[buf]));
      }
      if (*abort) mma_drain(s32(&sm.mma_drain_bar[0]));  // products already issued must finish before the release
    }
  } else if (warp == kWMma1) {
    // ------------------------------------------------------------- issuer of dV += P^T dO and dK += dS^T Q (one thread)
    if (lane == 0) {
      constexpr uint32_t idesc_nn = make_idesc(true, 64u, F16);
      long long pr = 0;
      uint32_t jg[2] = {0u, 0u};  // products each group of row threads has handed over (phase of p_full)
      uint32_t items = 0;         // items whose accumulators have been handed to the row threads
      bool ok = true, first = true;
      for (int lb = 0; ok; ++lb) {
        const int buf = lb % kLists;
        ok = mbar_wait(s32(&sm.list_full[buf]), (lb / kLists) & 1, abort, status);
        if (!ok) break;
        const int n = sm.info[buf].n;
        if (n < 0) break;
        const bool more = sm.info[buf].more != 0;
        const int chunks = n * g.cpb;
        for (int p0 = 0; p0 < chunks && ok; p0 += 2, ++pr) {
          const int slot = (int)(pr % kSlots), np = min(2, chunks - p0);
          // the slot landed before S^T could be produced; this wait makes the copied Q and dO visible here too
          ok = mbar_wait(s32(&sm.ring_full[slot]), (uint32_t)((pr / kSlots) & 1), abort, status);
          for (int h = 0; h < np && ok; ++h) {
            ok = mbar_wait(s32(&sm.p_full[h]), jg[h] & 1, abort, status);
            // a new accumulation overwrites dK and dV: every row thread must have read the previous item's
            if (ok && first && items > 0) ok = mbar_wait(s32(&sm.acc_free), (items - 1) & 1, abort, status);
            if (!ok) break;
            ++jg[h];
            tc_fence_after();
            const uint64_t qmn = smem_desc(s32(sm.ring[slot].q[h])), domn = smem_desc(s32(sm.ring[slot].d_o[h]));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_ts(tmem + kColDV, tmem + kColP + 32 * h + 8 * kk, domn + (uint64_t)((2048 * kk) >> 4), idesc_nn,
                      (!first || kk > 0));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_ts(tmem + kColDK, tmem + kColDS + 32 * h + 8 * kk, qmn + (uint64_t)((2048 * kk) >> 4), idesc_nn,
                      (!first || kk > 0));
            first = false;
          }
          if (!ok) break;
          // the pair's S^T and dP^T completed before P^T could be formed, so this thread's completion frees the slot
          tc_commit(s32(&sm.ring_empty[slot]));
          tc_commit(s32(&sm.pv_done));
        }
        if (ok && !more && !first) {  // the item's accumulators are complete behind this commit
          tc_commit(s32(&sm.acc_done));
          ++items;
          first = true;
        }
        if (ok) mbar_arrive(s32(&sm.list_empty[buf]));
      }
      if (*abort) mma_drain(s32(&sm.mma_drain_bar[1]));
    }
  } else if (warp < kRowWarps) {
    // ------------------------------------------------------------- row threads (TMEM lane = key row)
    // Group 0 takes the first chunk of every pair, group 1 the second, so the two work side by side.  Inside a
    // group two threads share a key row, each with half of the query columns.
    const int grp = warp >> 3;        // chunk of a pair this thread works on
    const int ch = (warp >> 2) & 1;   // half of the query columns
    const int cq = warp >> 2;         // quarter of the output channels (epilogue)
    const int quad = warp & 3;        // TMEM lane quadrant
    const int hh = quad >> 1;         // 64-row half of the tile this warp's rows belong to
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    const uint32_t tb = tmem + lane_off;
    const uint32_t hbit = 1u << hh;
    const uint64_t scale2 = pack2(g.scale_log2, g.scale_log2);
    const uint32_t col_s = kColS + 64 * grp + 32 * ch, col_dp = kColDP + 64 * grp + 32 * ch;
    const uint32_t col_p = kColP + 32 * grp + 16 * ch, col_ds = kColDS + 32 * grp + 16 * ch;
    long long pr = 0;    // pairs seen so far
    uint32_t item_chunks = 0, items = 0;
    bool ok = true;
    for (int lb = 0; ok; ++lb) {
      const int buf = lb % kLists;
      ok = mbar_wait(s32(&sm.list_full[buf]), (lb / kLists) & 1, abort, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int n = sm.info[buf].n;
      if (n < 0) break;
      const bool more = sm.info[buf].more != 0;
      const int chunks = n * g.cpb;
      item_chunks += (uint32_t)chunks;
      for (int p0 = 0; p0 < chunks; p0 += 2, ++pr) {
        ok = mbar_wait(s32(&sm.s_full), (uint32_t)(pr & 1), abort, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const int p = p0 + grp;
        if (p >= chunks) {  // a pair of one: nothing for group 1, the buffers go back at once
          tc_fence_before();
          mbar_arrive(s32(&sm.sdp_free));
          continue;
        }
        const bool connected = (sm.mask[buf][p / g.cpb] & hbit) != 0;
        uint32_t pp[16], ds[16];
        if (connected) {
          const int slot = (int)(pr % kSlots);
          // the slot landed before the MMA warp could produce this S^T; waiting on its barrier here as well
          // makes the copied -LSE and -D visible to this thread
          ok = mbar_wait(s32(&sm.ring_full[slot]), (uint32_t)((pr / kSlots) & 1), abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const Slot& sl = sm.ring[slot];
          uint32_t sv[32], dp[32];
          tmem_ld32(tb + col_s, sv);
          tmem_ld32(tb + col_dp, dp);
          tmem_wait_ld();
          tc_fence_before();
          mbar_arrive(s32(&sm.sdp_free));  // S^T and dP^T go back to the tensor core
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            // -LSE*log2(e) and -D of four query columns (the same for every thread: broadcast loads)
            const float4 nl = *reinterpret_cast<const float4*>(&sl.neg_lse2[grp][32 * ch + i]);
            const float4 nd = *reinterpret_cast<const float4*>(&sl.neg_d[grp][32 * ch + i]);
            float x0, x1, x2, x3, d0, d1, d2, d3;
            unpack2(fma2(pack2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), scale2, pack2(nl.x, nl.y)), x0, x1);
            unpack2(fma2(pack2(__uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3])), scale2, pack2(nl.z, nl.w)), x2, x3);
            const float e0 = ex2(x0), e1 = ex2(x1), e2 = ex2(x2), e3 = ex2(x3);
            const uint64_t t01 = add2(pack2(__uint_as_float(dp[i]), __uint_as_float(dp[i + 1])), pack2(nd.x, nd.y));
            const uint64_t t23 = add2(pack2(__uint_as_float(dp[i + 2]), __uint_as_float(dp[i + 3])), pack2(nd.z, nd.w));
            unpack2(mul2(pack2(e0, e1), t01), d0, d1);
            unpack2(mul2(pack2(e2, e3), t23), d2, d3);
            pp[i >> 1] = pack2<F16>(e0, e1);
            pp[(i >> 1) + 1] = pack2<F16>(e2, e3);
            ds[i >> 1] = pack2<F16>(d0, d1);
            ds[(i >> 1) + 1] = pack2<F16>(d2, d3);
          }
        } else {
          tc_fence_before();
          mbar_arrive(s32(&sm.sdp_free));
#pragma unroll
          for (int i = 0; i < 16; ++i) { pp[i] = 0u; ds[i] = 0u; }
        }
        // P^T and dS^T have one buffer per group: the previous pair's dV / dK updates must have consumed them
        if (pr > 0) {
          ok = mbar_wait(s32(&sm.pv_done), (uint32_t)((pr - 1) & 1), abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        tmem_st16(tb + col_p, pp);
        tmem_st16(tb + col_ds, ds);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(s32(&sm.p_full[grp]));
      }
      if (!ok) break;
      if (!more) {
        if (item_chunks > 0) {
          ok = mbar_wait(s32(&sm.acc_done), items & 1, abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          if ((sm.info[buf].hvalid >> hh) & 1) {
            const long long tok = (long long)sm.info[buf].kvunit * g.N +
                                  chunk_token(g, sm.info[buf].hb[hh], sm.info[buf].hc[hh], (quad & 1) * 32 + lane);
#pragma unroll
            for (int which = 0; which < 2; ++which) {  // 0: dK (scaled), 1: dV
              uint4* dst = reinterpret_cast<uint4*>((which ? dv : dk) + tok * kD + 16 * cq);
              const float f = which ? 1.f : g.scale;
              uint32_t ov[16];
              tmem_ld16(tb + (which ? kColDV : kColDK) + 16 * cq, ov);
              tmem_wait_ld();
              uint32_t w[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                w[i] = pack2<F16>(__uint_as_float(ov[2 * i]) * f, __uint_as_float(ov[2 * i + 1]) * f);
              dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
              dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
          }
          // the accumulators may be overwritten by the next item's first products
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(s32(&sm.acc_free));
          ++items;
        } else if ((sm.info[buf].hvalid >> hh) & 1) {
          // a tile that no query block is connected to (possible when the local set is switched off): zero gradients
          const long long tok = (long long)sm.info[buf].kvunit * g.N +
                                chunk_token(g, sm.info[buf].hb[hh], sm.info[buf].hc[hh], (quad & 1) * 32 + lane);
          const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
          uint4* dst_k = reinterpret_cast<uint4*>(dk + tok * kD + 16 * cq);
          uint4* dst_v = reinterpret_cast<uint4*>(dv + tok * kD + 16 * cq);
          dst_k[0] = zero; dst_k[1] = zero;
          dst_v[0] = zero; dst_v[1] = zero;
        }
        item_chunks = 0;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s32(&sm.list_empty[buf]));
    }
  }
  cta_tmem_free(warp == kWMma0, tmem, kTmemCols);
}

// `work_counter` must be zero when the kernel starts (a word of the workspace status block).
template <bool F16>
static int launch_dkdv_tc_t(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o,
                   const float* neg_lse2, const float* neg_d, const int32_t* csr_off, const int32_t* csr_q, void* dk,
                   void* dv, int* work_counter, int32_t* order) {
  const Geo& g = c.g;
  CUtensorMap mq, mdo, mk, mv, mnl, mnd;
  if (!make_map(&mq, q, g, g.U) || !make_map(&mdo, d_o, g, g.U) || !make_map(&mk, k, g, g.Ukv) || !make_map(&mv, v, g, g.Ukv) ||
      !make_map_rows(&mnl, neg_lse2, g) || !make_map_rows(&mnd, neg_d, g))
    return MOSAIC_E_CUDA;
  const size_t smem = sizeof(Smem) + 1024;
  static unsigned long long configured = 0;  // devices on which the kernel's shared-memory opt-in is set
  int sms = 0;
  if (const int rc = launch_setup(reinterpret_cast<const void*>(dkdv_tc_kernel<F16>), smem, &configured, &sms)) return rc;
  const int ipu = items_per_unit(g);
  const long long total = 2ll * g.Ukv * ipu;  // one item per 128-row tile of a key/value unit
  if (total > 0x7fffff00ll) return MOSAIC_E_UNSUPPORTED;
  const long long grid = total < (long long)sms ? total : (long long)sms;
  // window: the key/value units whose Q and dO (all query heads of the group) take about 48 MB, widened to
  // sixteen items per SM
  const size_t unit_bytes = (size_t)(g.H / g.Hkv) * g.N * kD * 2 * 2;
  long long win_units = unit_bytes >= (48u << 20) ? 1 : (long long)((48u << 20) / unit_bytes);
  const long long min_units = (16ll * sms + 2 * ipu - 1) / (2 * ipu);
  if (win_units < min_units) win_units = min_units;
  const long long win_items = win_units * 2 * ipu;
  dkdv_order_kernel<<<(unsigned)((total + win_items - 1) / win_items), 1024, 0, c.stream>>>(
      g, csr_off, ipu, (int)total, (int)win_items, order, order + total);
  if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  dkdv_tc_kernel<F16><<<(unsigned)grid, kThreads, smem, c.stream>>>(g, mq, mdo, mk, mv, mnl, mnd, csr_off, csr_q, order,
                                                               (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, c.status,
                                                               work_counter, ipu, (int)total);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_dkdv_tc(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o,
                   const float* neg_lse2, const float* neg_d, const int32_t* csr_off, const int32_t* csr_q, void* dk,
                   void* dv, int* work_counter, int32_t* order) {
  return c.g.f16 ? launch_dkdv_tc_t<true>(c, q, k, v, d_o, neg_lse2, neg_d, csr_off, csr_q, dk, dv, work_counter, order) : launch_dkdv_tc_t<false>(c, q, k, v, d_o, neg_lse2, neg_d, csr_off, csr_q, dk, dv, work_counter, order);
}

}  // namespace mosaic
