// dK and dV of the block-sparse attention backward on Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// Paper, appendix "Block-sparse attention implementation", paragraph "Kernel Design": the gradients of
// keys and values are formed per key/value block by visiting only the query blocks connected to it.
// With P = exp(scale * Q K^T - LSE), dP = dO V^T, D = rowsum(dO o O), dS = P o (dP - D):
//   dV_j = sum_i P_ij^T dO_i ,   dK_j = scale * sum_i dS_ij^T Q_i      (i over the query blocks connected to j)
// The connected query blocks of key block j are its local neighbours (the neighbourhood relation is
// symmetric, so they follow from geometry) and the query blocks that selected j (transposed pattern, CSR).
//
// Key/value-stationary mirror of the forward kernel: a persistent CTA per SM draws 256-row items of KEY
// rows (two 128-row tiles, four 64-row halves, each half one 64-token chunk of a key block); the K and V
// tiles stay in shared memory, query-side chunks (Q, dO, and per query row -LSE*log2(e) and -D) stream
// through a ring.  Per product and tile:  S^T = K Q^T and dP^T = V dO^T (eight MMAs into two 64-column TMEM
// buffers), the row threads (thread = key row = TMEM lane) write P^T over the start of the S^T buffer and
// dS^T over the start of the dP^T buffer (bf16), then dV += P^T dO and dK += dS^T Q with those buffers as
// TMEM A operands and the staged dO and Q chunks as MN-major B operands.
// Lists: the planner merges the local neighbourhoods of the item's key blocks (entries carry a mask of
// the halves they are connected to) and appends each block's CSR list; a list longer than a list buffer
// continues in the next buffer (ItemInfo::more).  The order of a list is a function of the pattern alone,
// so the summation order, and with it the result, is deterministic.
// Every mbarrier wait is bounded; on expiry the CTA records MOSAIC_E_DEVICE_TIMEOUT and drains.
#include "tc_common.cuh"

namespace mosaic {

namespace {

constexpr int kStages = 6;       // ring depth of query-side chunks
constexpr int kThreads = 384;
constexpr uint32_t kTmemCols = 512;
// tile t: dK at 256 t, dV at 256 t + 64, S^T (then P^T) at 256 t + 128, dP^T (then dS^T) at 256 t + 192
constexpr uint32_t kColDK = 0, kColDV = 64, kColS = 128, kColDP = 192, kTileCols = 256;
constexpr uint32_t kStageBytes = 2 * kTile + 2 * 64 * 4;

struct Stage {
  unsigned char q[kTile];     // 64 query rows x 128 B, swizzled
  unsigned char d_o[kTile];
  float neg_lse2[64];         // -LSE * log2(e) of the chunk's query rows
  float neg_d[64];            // -D of the chunk's query rows
  unsigned char pad[1024 - 512];
};

struct Smem {
  unsigned char k[2][2 * kTile];           // [tile][128 key rows x 128 B]
  unsigned char v[2][2 * kTile];
  Stage ring[kStages];
  unsigned long long ring_full[kStages], ring_empty[kStages];
  unsigned long long kv_full[2], kv_empty[2], s_full[2], p_full[2], pv_done[2];  // [tile]
  unsigned long long list_full[kLists], list_empty[kLists];
  uint32_t tmem_base;
  int abort;
  ItemInfo info[kLists];
  int ids[kLists][kMaxUnion];
  unsigned char mask[kLists][kMaxUnion];
  int tmp_ids[kMaxUnion];            // planner scratch: merged list before reordering
  unsigned char tmp_mask[kMaxUnion];
};

// Planner of the key-stationary kernel: per item, the merged local neighbourhoods of its key blocks, then
// each block's list of selecting query blocks, cut into list buffers.
__device__ __forceinline__ void planner_kv_loop(Smem& sm, const Geo& g, const int32_t* __restrict__ csr_off,
                                                const int32_t* __restrict__ csr_q, int* work_counter, int ipu,
                                                int total_items, int lane, volatile int* abort, int* status) {
  int lb = 0;  // list buffers handed out so far
  for (int it = 0;; ++it) {
    int item = 0;
    if (lane == 0) item = it == 0 ? (int)blockIdx.x : atomicAdd(work_counter, 1) + (int)gridDim.x;
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
    const int u = item / ipu;
    int hb[4], hc[4];
    const int valid = item_halves(g, item - u * ipu, hb, hc);
    int n = 0;
    auto publish = [&](int more) {  // reorder the scratch list into buffer lb and hand it over
      const int buf = lb % kLists;
      interleave_tiles(sm.tmp_ids, sm.tmp_mask, n, sm.ids[buf], sm.mask[buf], lane);
      if (lane == 0) {
        ItemInfo& inf = sm.info[buf];
        inf.n = n; inf.unit = u; inf.hvalid = valid; inf.more = more;
#pragma unroll
        for (int h = 0; h < 4; ++h) { inf.hb[h] = hb[h]; inf.hc[h] = hc[h]; }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(s32(&sm.list_full[buf]));
      ++lb;
      n = 0;
    };
    // the halves of one key block are merged once, with all their bits
    unsigned char bits_of[4];
    bool first_of[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      first_of[h] = ((valid >> h) & 1) != 0;
      bits_of[h] = 0;
#pragma unroll
      for (int h2 = 0; h2 < 4; ++h2) {
        if (((valid >> h2) & 1) && ((valid >> h) & 1) && hb[h2] == hb[h]) {
          if (h2 < h) first_of[h] = false;
          bits_of[h] |= (unsigned char)(1 << h2);
        }
      }
    }
    // local neighbourhoods (at most 64 entries per block, merged with masks)
#pragma unroll
    for (int h = 0; h < 4; ++h)
      if (first_of[h]) n = merge_block(g, -1, hb[h], bits_of[h], sm.tmp_ids, sm.tmp_mask, n, lane, status);
    // query blocks that selected the key block (ascending ids), appended 32 at a time
    const int32_t* off = csr_off + (long long)u * (g.m + 1);
    const int32_t* sel = csr_q + (long long)u * g.m * g.topk;
#pragma unroll
    for (int h = 0; h < 4 && ok; ++h) {
      if (!first_of[h]) continue;
      const int s_beg = __ldg(off + hb[h]), s_end = __ldg(off + hb[h] + 1);
      for (int base = s_beg; base < s_end && ok; base += 32) {
        if (n + 32 > kMaxUnion) {
          publish(1);
          acquire();
          if (!ok) break;
        }
        const int e = base + lane;
        if (e < s_end) {
          sm.tmp_ids[n + lane] = __ldg(sel + e);
          sm.tmp_mask[n + lane] = bits_of[h];
        }
        n += min(32, s_end - base);
        __syncwarp();
      }
    }
    if (!ok) break;
    publish(0);
  }
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
    dkdv_tc_kernel(const Geo g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                   const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const __grid_constant__ CUtensorMap map_nlse, const __grid_constant__ CUtensorMap map_nd,
                   const int32_t* __restrict__ csr_off, const int32_t* __restrict__ csr_q,
                   __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, int* status, int* work_counter,
                   int ipu, int total_items) {
  extern __shared__ unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(s32(&sm.ring_full[s]), 1); mbar_init(s32(&sm.ring_empty[s]), 2); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(s32(&sm.kv_full[t]), 1);
      mbar_init(s32(&sm.kv_empty[t]), 1);
      mbar_init(s32(&sm.s_full[t]), 1);
      mbar_init(s32(&sm.p_full[t]), 128);
      mbar_init(s32(&sm.pv_done[t]), 1);
    }
    for (int i = 0; i < kLists; ++i) {
      mbar_init(s32(&sm.list_full[i]), 1);
      mbar_init(s32(&sm.list_empty[i]), 11);  // 8 row-thread warps + 2 MMA warps + TMA producer
    }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm.tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  const uint32_t tmem = sm.tmem_base;
  volatile int* abort = &sm.abort;

  if (warp == 11) {
    planner_kv_loop(sm, g, csr_off, csr_q, work_counter, ipu, total_items, lane, abort, status);
  } else if (warp == 8) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      long long step = 0;  // query-side chunks issued so far (ring position)
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
          for (int t = 0; t < 2 && ok; ++t) {
            ok = mbar_wait(s32(&sm.kv_empty[t]), (items & 1) ^ 1, abort, status);
            if (!ok) break;
            mbar_expect_tx(s32(&sm.kv_full[t]), 4 * kTile);
            for (int hh = 0; hh < 2; ++hh) {
              const int h = 2 * t + hh, by = inf.hb[h] / g.nbw, bx = inf.hb[h] - by * g.nbw;
              tma_load_4d(s32(sm.k[t] + hh * kTile), &map_k, s32(&sm.kv_full[t]), 0, bx * g.bw,
                          by * g.bh + inf.hc[h] * g.crows, u);
              tma_load_4d(s32(sm.v[t] + hh * kTile), &map_v, s32(&sm.kv_full[t]), 0, bx * g.bw,
                          by * g.bh + inf.hc[h] * g.crows, u);
            }
          }
          ++items;
        }
        fresh = inf.more == 0;
        for (int e = 0; e < n && ok; ++e) {
          const int i = sm.ids[buf][e], by = i / g.nbw, bx = i - by * g.nbw;
          for (int c = 0; c < g.cpb; ++c, ++step) {
            const int st = (int)(step % kStages);
            ok = mbar_wait(s32(&sm.ring_empty[st]), (uint32_t)((step / kStages) & 1) ^ 1, abort, status);
            if (!ok) break;
            Stage& sg = sm.ring[st];
            const uint32_t bar = s32(&sm.ring_full[st]);
            const int x0 = bx * g.bw, y0 = by * g.bh + c * g.crows;
            mbar_expect_tx(bar, kStageBytes);
            tma_load_4d(s32(sg.q), &map_q, bar, 0, x0, y0, u);
            tma_load_4d(s32(sg.d_o), &map_do, bar, 0, x0, y0, u);
            tma_load_3d(s32(sg.neg_lse2), &map_nlse, bar, x0, y0, u);
            tma_load_3d(s32(sg.neg_d), &map_nd, bar, x0, y0, u);
          }
        }
        if (ok) mbar_arrive(s32(&sm.list_empty[buf]));
      }
      if (*abort) {  // give copies in flight time to land before the CTA's memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) {}
      } else {       // drain: the last uses of every ring stage have been released by both tiles
        const long long first = step > kStages ? step - kStages : 0;
        for (long long s = first; s < step; ++s)
          if (!mbar_wait(s32(&sm.ring_empty[s % kStages]), (uint32_t)((s / kStages) & 1), abort, status)) break;
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------------------------------------- MMA issuer of tile t
    // The whole warp walks the loop; one elected lane issues the tensor-core instructions.
    const int t = warp - 9;
    constexpr uint32_t idesc_nt = make_idesc(false), idesc_nn = make_idesc(true);
    const uint64_t kdesc = smem_desc(s32(sm.k[t])), vdesc = smem_desc(s32(sm.v[t]));
    const uint32_t tbase = tmem + kTileCols * t;
    const uint32_t tbits = 3u << (2 * t);
    long long step = 0;   // ring position (all chunks, connected to this tile or not)
    uint32_t nt = 0;      // products issued by this tile so far (phase of s_full / p_full / pv_done)
    int items = 0;
    bool ok = true, fresh = true, first = true;
    for (int lb = 0; ok; ++lb) {
      const int buf = lb % kLists;
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.list_full[buf]), (lb / kLists) & 1, abort, status));
      if (!ok) break;
      const int n = sm.info[buf].n;
      if (n < 0) break;
      const bool more = sm.info[buf].more != 0;
      if (fresh) {
        ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.kv_full[t]), items & 1, abort, status));
        if (!ok) break;
        ++items;
        first = true;
      }
      fresh = !more;
      for (int e = 0; e < n && ok; ++e) {
        const bool act = (sm.mask[buf][e] & tbits) != 0;
        for (int c = 0; c < g.cpb && ok; ++c, ++step) {
          const int st = (int)(step % kStages);
          ok = __all_sync(0xffffffffu,
                          mbar_wait(s32(&sm.ring_full[st]), (uint32_t)((step / kStages) & 1), abort, status));
          if (!ok) break;
          if (!act) {
            if (elect_one()) mbar_arrive(s32(&sm.ring_empty[st]));
            continue;
          }
          // S^T and dP^T were last read by this warp's previous dV / dK products (P^T and dS^T alias them)
          // and before that by the row threads, which arrived on p_full: in-order execution makes
          // overwriting them safe
          tc_fence_after();
          const uint64_t qdesc = smem_desc(s32(sm.ring[st].q)), dodesc = smem_desc(s32(sm.ring[st].d_o));
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_ss(tbase + kColS, kdesc + 2 * kk, qdesc + 2 * kk, idesc_nt, kk > 0);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_ss(tbase + kColDP, vdesc + 2 * kk, dodesc + 2 * kk, idesc_nt, kk > 0);
            tc_commit(s32(&sm.s_full[t]));
          }
          __syncwarp();
          ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.p_full[t]), nt & 1, abort, status));
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_ts(tbase + kColDV, tbase + kColS + 8 * kk, dodesc + (uint64_t)((2048 * kk) >> 4), idesc_nn,
                      (!first || kk > 0));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_ts(tbase + kColDK, tbase + kColDP + 8 * kk, qdesc + (uint64_t)((2048 * kk) >> 4), idesc_nn,
                      (!first || kk > 0));
            tc_commit(s32(&sm.ring_empty[st]));
            tc_commit(s32(&sm.pv_done[t]));
          }
          __syncwarp();
          first = false;
          ++nt;
        }
      }
      if (ok && !more && elect_one()) tc_commit(s32(&sm.kv_empty[t]));  // all products of the item are behind it
      if (ok && elect_one()) mbar_arrive(s32(&sm.list_empty[buf]));
    }
  } else {
    // ------------------------------------------------------------- row threads of tile t (thread = key row)
    const int t = warp >> 2;        // tile
    const int hh = (warp >> 1) & 1; // 64-row half of the tile this warp's rows belong to
    const int h = 2 * t + hh;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tbase = tmem + lane_off + kTileCols * t;
    const uint32_t tbits = 3u << (2 * t), hbit = 1u << h;
    const uint64_t scale2 = pack2(g.scale_log2, g.scale_log2);
    uint32_t nt = 0;
    long long step = 0;  // ring position, to find the stage that holds the query rows' -LSE and -D
    uint32_t item_done = 0;
    bool ok = true;
    for (int lb = 0; ok; ++lb) {
      const int buf = lb % kLists;
      ok = mbar_wait(s32(&sm.list_full[buf]), (lb / kLists) & 1, abort, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int n = sm.info[buf].n;
      if (n < 0) break;
      const bool more = sm.info[buf].more != 0;
      for (int e = 0; e < n && ok; ++e) {
        const uint32_t mk = sm.mask[buf][e];
        if (!(mk & tbits)) { step += g.cpb; continue; }
        const bool connected = (mk & hbit) != 0;
        for (int c = 0; c < g.cpb; ++c, ++step) {
          ok = mbar_wait(s32(&sm.s_full[t]), nt & 1, abort, status);  // implies the ring stage has landed
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          if (connected) {
            const int st = (int)(step % kStages);
            // the stage landed before the MMA warp could produce this S^T; waiting on its barrier here as well
            // makes the copied -LSE and -D visible to this thread
            ok = mbar_wait(s32(&sm.ring_full[st]), (uint32_t)((step / kStages) & 1), abort, status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const Stage& sg = sm.ring[st];
            // two pieces of 32 query columns; piece p writes P^T and dS^T (bf16 pairs) over columns
            // 16p .. 16p+15 of the S^T and dP^T buffers, which hold values this thread has already consumed
#pragma unroll
            for (int piece = 0; piece < 2; ++piece) {
              uint32_t sv[32], dp[32], pp[16], ds[16];
              tmem_ld32(tbase + kColS + 32 * piece, sv);
              tmem_ld32(tbase + kColDP + 32 * piece, dp);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                // -LSE*log2(e) and -D of four query columns (the same for every thread: broadcast loads)
                const float4 nl = *reinterpret_cast<const float4*>(&sg.neg_lse2[32 * piece + i]);
                const float4 nd = *reinterpret_cast<const float4*>(&sg.neg_d[32 * piece + i]);
                float x0, x1, x2, x3, d0, d1, d2, d3;
                unpack2(fma2(pack2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), scale2, pack2(nl.x, nl.y)), x0, x1);
                unpack2(fma2(pack2(__uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3])), scale2, pack2(nl.z, nl.w)), x2, x3);
                const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
                const uint64_t t01 = add2(pack2(__uint_as_float(dp[i]), __uint_as_float(dp[i + 1])), pack2(nd.x, nd.y));
                const uint64_t t23 = add2(pack2(__uint_as_float(dp[i + 2]), __uint_as_float(dp[i + 3])), pack2(nd.z, nd.w));
                unpack2(mul2(pack2(p0, p1), t01), d0, d1);
                unpack2(mul2(pack2(p2, p3), t23), d2, d3);
                pp[i >> 1] = bf16x2(p0, p1);
                pp[(i >> 1) + 1] = bf16x2(p2, p3);
                ds[i >> 1] = bf16x2(d0, d1);
                ds[(i >> 1) + 1] = bf16x2(d2, d3);
              }
              tmem_st16(tbase + kColS + 16 * piece, pp);
              tmem_st16(tbase + kColDP + 16 * piece, ds);
            }
          } else {
            uint32_t z[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) z[i] = 0u;
            tmem_st32(tbase + kColS, z);
            tmem_st32(tbase + kColDP, z);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(s32(&sm.p_full[t]));
          ++nt;
          ++item_done;
        }
      }
      if (!ok) break;
      if (!more) {
        if (item_done > 0) {
          ok = mbar_wait(s32(&sm.pv_done[t]), (nt - 1) & 1, abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          if ((sm.info[buf].hvalid >> h) & 1) {
            const long long tok = (long long)sm.info[buf].unit * g.N +
                                  chunk_token(g, sm.info[buf].hb[h], sm.info[buf].hc[h], tid & 63);
#pragma unroll
            for (int which = 0; which < 2; ++which) {  // 0: dK (scaled), 1: dV
              uint4* dst = reinterpret_cast<uint4*>((which ? dv : dk) + tok * kD);
              const float f = which ? 1.f : g.scale;
#pragma unroll
              for (int part = 0; part < 2; ++part) {
                uint32_t ov[32];
                tmem_ld32(tbase + (which ? kColDV : kColDK) + 32 * part, ov);
                tmem_wait_ld();
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                  w[i] = bf16x2(__uint_as_float(ov[2 * i]) * f, __uint_as_float(ov[2 * i + 1]) * f);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                  dst[part * 4 + i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
              }
            }
          }
        }
        item_done = 0;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s32(&sm.list_empty[buf]));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// `work_counter` must be zero when the kernel starts (a word of the workspace status block).
int launch_dkdv_tc(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o,
                   const float* neg_lse2, const float* neg_d, const int32_t* csr_off, const int32_t* csr_q, void* dk,
                   void* dv, int* work_counter) {
  const Geo& g = c.g;
  CUtensorMap mq, mdo, mk, mv, mnl, mnd;
  if (!make_map(&mq, q, g) || !make_map(&mdo, d_o, g) || !make_map(&mk, k, g) || !make_map(&mv, v, g) ||
      !make_map_rows(&mnl, neg_lse2, g) || !make_map_rows(&mnd, neg_d, g))
    return MOSAIC_E_CUDA;
  const size_t smem = sizeof(Smem) + 1024;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MOSAIC_E_CUDA;
  if (cudaFuncSetAttribute(dkdv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return MOSAIC_E_CUDA;
  const int ipu = items_per_unit(g);
  const long long total = (long long)g.U * ipu;
  if (total > 0x7fffff00ll) return MOSAIC_E_UNSUPPORTED;
  const long long grid = total < (long long)sms ? total : (long long)sms;
  dkdv_tc_kernel<<<(unsigned)grid, kThreads, smem, c.stream>>>(g, mq, mdo, mk, mv, mnl, mnd, csr_off, csr_q,
                                                               (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, c.status,
                                                               work_counter, ipu, (int)total);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

}  // namespace mosaic
