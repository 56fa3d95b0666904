// dQ of the block-sparse attention backward on Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// Paper, appendix "Block-sparse attention implementation", paragraph "Kernel Design": the backward
// recomputes the probabilities from the saved log-sum-exp instead of storing the attention matrix, and
// the query gradient is query-block stationary with the same traversal as the forward.
//   P = exp(scale * Q K^T - LSE),  dP = dO V^T,  dS = P o (dP - D),  dQ = scale * dS K,
// D = rowsum(dO o O) from the preprocessing kernel; the selection is a constant of the backward.
//
// Same work decomposition as the forward kernel: a persistent CTA per SM draws 256-row items (two
// 128-row tiles, four 64-row halves) from a queue; a planner warp merges the key lists of the item's
// query blocks; a producer warp streams 64-token K and V chunks through a ring; one warp per tile issues
// the tensor-core work; two groups of four warps (thread = query row = TMEM lane) turn S and dP into dS.
// Per product and tile: S = Q K^T and dP = dO V^T (eight MMAs into two 64-column TMEM buffers); the row
// threads pull both into registers and hand the buffers back at once, so the next product's S and dP are
// computed while they form dS (bf16, its own 32 TMEM columns); then dQ += dS K (dS is the TMEM A operand,
// the K chunk in shared memory is read as the MN-major B operand), issued one product behind.
// Every mbarrier wait is bounded; on expiry the CTA records MOSAIC_E_DEVICE_TIMEOUT and drains.
#include "tc_common.cuh"

namespace mosaic {

namespace {

constexpr int kStages = 6;       // key/value ring depth (K + V chunk per stage)
constexpr int kThreads = 384;
constexpr uint32_t kTmemCols = 512;
// dQ of tile t at 64 t; S of tile t at 128 + 128 t, dP right after it; dS (bf16) of tile t at 384 + 32 t
constexpr uint32_t kColDQ = 0, kColS = 128, kColDS = 384;

struct Smem {
  unsigned char q[2][2 * kTile];           // [tile][128 rows x 128 B]
  unsigned char d_o[2][2 * kTile];         // [tile][128 rows x 128 B]
  unsigned char kv[kStages][2][kTile];     // [stage][K, V]
  unsigned long long kv_full[kStages], kv_empty[kStages];
  unsigned long long q_full[2], q_empty[2], s_full[2], sdp_free[2], p_full[2], pv_done[2];  // [tile]
  unsigned long long mma_drain_bar[2];  // abort path: completion of each issuer's outstanding products
  unsigned long long list_full[kLists], list_empty[kLists];
  uint32_t tmem_base;
  int abort;
  ItemInfo info[kLists];
  int ids[kLists][kMaxUnion];
  unsigned char mask[kLists][kMaxUnion];
  int tmp_ids[kMaxUnion];            // planner scratch: merged list before reordering
  unsigned char tmp_mask[kMaxUnion];
};

}  // namespace

template <bool F16>
__global__ void __launch_bounds__(kThreads, 1)
    dq_tc_kernel(const Geo g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                 const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const int32_t* __restrict__ block_idx, const float* __restrict__ lse, const float* __restrict__ D,
                 __nv_bfloat16* __restrict__ dq, int* status, int* work_counter, int ipu, int total_items) {
  extern __shared__ unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(s32(&sm.kv_full[s]), 1); mbar_init(s32(&sm.kv_empty[s]), 2); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(s32(&sm.q_full[t]), 1);
      mbar_init(s32(&sm.q_empty[t]), 1);
      mbar_init(s32(&sm.mma_drain_bar[t]), 1);
      mbar_init(s32(&sm.s_full[t]), 1);
      mbar_init(s32(&sm.sdp_free[t]), 128);
      mbar_init(s32(&sm.p_full[t]), 128);
      mbar_init(s32(&sm.pv_done[t]), 1);
    }
    for (int i = 0; i < kLists; ++i) {
      mbar_init(s32(&sm.list_full[i]), 1);
      mbar_init(s32(&sm.list_empty[i]), 11);  // 8 row-thread warps + 2 MMA warps + TMA producer
    }
    sm.abort = 0;
    cta_publish_barriers();
  }
  const uint32_t tmem = cta_tmem_alloc(warp == 9, &sm.tmem_base, kTmemCols);
  volatile int* abort = &sm.abort;

  if (warp == 11) {
    planner_loop(sm, g, block_idx, work_counter, ipu, total_items, lane, abort, status);
  } else if (warp == 8) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      long long step = 0;  // key/value chunks issued so far (ring position)
      int q_armed[2] = {-1, -1};  // phase parity of the last load into each tile's Q / dO buffer
      bool ok = true;
      for (int it = 0; ok; ++it) {
        const int buf = it % kLists;
        ok = mbar_wait(s32(&sm.list_full[buf]), (it / kLists) & 1, abort, status);
        if (!ok) break;
        const ItemInfo& inf = sm.info[buf];
        const int n = inf.n, u = inf.unit;
        if (n < 0) break;
        const int ukv = kv_unit(g, u);  // key/value head of this query head's group
        // Q and dO tiles: free once the tile's last S / dP products of the previous item have completed
        for (int t = 0; t < 2 && ok; ++t) {
          ok = mbar_wait(s32(&sm.q_empty[t]), (it & 1) ^ 1, abort, status);
          if (!ok) break;
          mbar_expect_tx(s32(&sm.q_full[t]), 4 * kTile);
          q_armed[t] = it & 1;
          for (int hh = 0; hh < 2; ++hh) {
            const int h = 2 * t + hh, by = inf.hb[h] / g.nbw, bx = inf.hb[h] - by * g.nbw;
            tma_load_4d(s32(sm.q[t] + hh * kTile), &map_q, s32(&sm.q_full[t]), 0, bx * g.bw,
                        by * g.bh + inf.hc[h] * g.crows, u);
            tma_load_4d(s32(sm.d_o[t] + hh * kTile), &map_do, s32(&sm.q_full[t]), 0, bx * g.bw,
                        by * g.bh + inf.hc[h] * g.crows, u);
          }
        }
        for (int e = 0; e < n && ok; ++e) {
          const int j = sm.ids[buf][e], by = j / g.nbw, bx = j - by * g.nbw;
          for (int c = 0; c < g.cpb; ++c, ++step) {
            const int st = (int)(step % kStages);
            ok = mbar_wait(s32(&sm.kv_empty[st]), (uint32_t)((step / kStages) & 1) ^ 1, abort, status);
            if (!ok) break;
            mbar_expect_tx(s32(&sm.kv_full[st]), 2 * kTile);
            tma_load_4d(s32(sm.kv[st][0]), &map_k, s32(&sm.kv_full[st]), 0, bx * g.bw, by * g.bh + c * g.crows, ukv);
            tma_load_4d(s32(sm.kv[st][1]), &map_v, s32(&sm.kv_full[st]), 0, bx * g.bw, by * g.bh + c * g.crows, ukv);
          }
        }
        if (ok) mbar_arrive(s32(&sm.list_empty[buf]));
      }
      if (*abort) {  // copies this thread issued must land before the CTA's memory is released
        const long long first = step > kStages ? step - kStages : 0;
        for (long long s = first; s < step; ++s) mbar_drain(s32(&sm.kv_full[s % kStages]), (uint32_t)((s / kStages) & 1));
        for (int t = 0; t < 2; ++t)
          if (q_armed[t] >= 0) mbar_drain(s32(&sm.q_full[t]), (uint32_t)q_armed[t]);
      } else {       // drain: the last uses of every ring stage have been released by both tiles
        const long long first = step > kStages ? step - kStages : 0;
        for (long long s = first; s < step; ++s)
          if (!mbar_wait(s32(&sm.kv_empty[s % kStages]), (uint32_t)((s / kStages) & 1), abort, status)) break;
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------------------------------------- MMA issuer of tile t
    // The whole warp walks the loop; one elected lane issues the tensor-core instructions.
    const int t = warp - 9;
    constexpr uint32_t idesc_nt = make_idesc(false, 64u, F16), idesc_nn = make_idesc(true, 64u, F16);
    const uint64_t qdesc = smem_desc(s32(sm.q[t])), dodesc = smem_desc(s32(sm.d_o[t]));
    const uint32_t tcol_dq = tmem + kColDQ + 64 * t, tcol_s = tmem + kColS + 128 * t, tcol_dp = tcol_s + 64;
    const uint32_t tcol_ds = tmem + kColDS + 32 * t;
    const uint32_t tbits = 3u << (2 * t);
    long long step = 0;   // ring position (all chunks, attended by this tile or not)
    uint32_t nt = 0;      // products started by this tile so far (phase of the per-product barriers)
    bool ok = true;
    // dQ += dS K of the product whose K chunk sits in ring stage `pst` (the previous product of this tile)
    auto issue_dq = [&](int pst, bool pfirst) {
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.p_full[t]), (nt - 1) & 1, abort, status));
      if (!ok) return;
      tc_fence_after();
      const uint64_t kmn = smem_desc(s32(sm.kv[pst][0]));
      if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_ts(tcol_dq, tcol_ds + 8 * kk, kmn + (uint64_t)((2048 * kk) >> 4), idesc_nn, (!pfirst || kk > 0));
        tc_commit(s32(&sm.kv_empty[pst]));
        tc_commit(s32(&sm.pv_done[t]));
      }
      __syncwarp();
    };
    for (int it = 0; ok; ++it) {
      const int buf = it % kLists;
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.list_full[buf]), (it / kLists) & 1, abort, status));
      if (!ok) break;
      const int n = sm.info[buf].n;
      if (n < 0) break;
      int last = -1;
      for (int e = 0; e < n; ++e)
        if (sm.mask[buf][e] & tbits) last = e;
      // the tiles are loaded for every item; they must have landed before their buffers are handed back
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.q_full[t]), it & 1, abort, status));
      if (!ok) break;
      if (last < 0 && elect_one()) mbar_arrive(s32(&sm.q_empty[t]));
      bool first = true, pend = false, pend_first = false;
      int pend_st = 0;
      for (int e = 0; e < n && ok; ++e) {
        const bool act = (sm.mask[buf][e] & tbits) != 0;
        for (int c = 0; c < g.cpb && ok; ++c, ++step) {
          const int st = (int)(step % kStages);
          ok = __all_sync(0xffffffffu,
                          mbar_wait(s32(&sm.kv_full[st]), (uint32_t)((step / kStages) & 1), abort, status));
          if (!ok) break;
          if (!act) {
            if (elect_one()) mbar_arrive(s32(&sm.kv_empty[st]));
            continue;
          }
          // S and dP may be overwritten once the row threads hold the previous product's values in registers
          if (nt > 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.sdp_free[t]), (nt - 1) & 1, abort, status));
            if (!ok) break;
          }
          tc_fence_after();
          const uint64_t kdesc = smem_desc(s32(sm.kv[st][0])), vdesc = smem_desc(s32(sm.kv[st][1]));
          const bool release_q = e == last && c == g.cpb - 1;
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_ss(tcol_s, qdesc + 2 * kk, kdesc + 2 * kk, idesc_nt, kk > 0);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_ss(tcol_dp, dodesc + 2 * kk, vdesc + 2 * kk, idesc_nt, kk > 0);
            tc_commit(s32(&sm.s_full[t]));
            if (release_q) tc_commit(s32(&sm.q_empty[t]));
          }
          __syncwarp();
          if (pend) issue_dq(pend_st, pend_first);  // previous product: its dS is ready or about to be
          if (!ok) break;
          pend = true; pend_st = st; pend_first = first;
          first = false;
          ++nt;
        }
      }
      if (ok && pend) issue_dq(pend_st, pend_first);  // the item's last product
      if (ok && elect_one()) mbar_arrive(s32(&sm.list_empty[buf]));
    }
    if (*abort) {  // products already issued must finish before TMEM and shared memory are released
      if (elect_one()) mma_drain(s32(&sm.mma_drain_bar[t]));
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------- row threads of tile t: S, dP -> dS; then epilogue
    const int t = warp >> 2;        // tile
    const int hh = (warp >> 1) & 1; // 64-row half of the tile this warp's rows belong to
    const int h = 2 * t + hh;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t ts = tmem + lane_off + kColS + 128 * t, tdp = ts + 64, tdq = tmem + lane_off + kColDQ + 64 * t;
    const uint32_t tds = tmem + lane_off + kColDS + 32 * t;
    const uint32_t tbits = 3u << (2 * t), hbit = 1u << h;
    const uint64_t scale2 = pack2(g.scale_log2, g.scale_log2);
    uint32_t nt = 0;
    bool ok = true;
    for (int it = 0; ok; ++it) {
      const int buf = it % kLists;
      ok = mbar_wait(s32(&sm.list_full[buf]), (it / kLists) & 1, abort, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int n = sm.info[buf].n;
      if (n < 0) break;
      const bool valid = (sm.info[buf].hvalid >> h) & 1;
      const long long tok =
          (long long)sm.info[buf].unit * g.N + chunk_token(g, sm.info[buf].hb[h], sm.info[buf].hc[h], tid & 63);
      // log-sum-exp (in base-2 units) and D of this thread's query row
      const float lse2 = valid ? __ldg(lse + tok) * 1.4426950408889634f : 0.f;
      const float dv = valid ? __ldg(D + tok) : 0.f;
      const uint64_t neg_lse2 = pack2(-lse2, -lse2), neg_d2 = pack2(-dv, -dv);
      uint32_t done = 0;
      for (int e = 0; e < n && ok; ++e) {
        const uint32_t mk = sm.mask[buf][e];
        if (!(mk & tbits)) continue;
        const bool attends = (mk & hbit) != 0;
        for (int c = 0; c < g.cpb; ++c) {
          ok = mbar_wait(s32(&sm.s_full[t]), nt & 1, abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          uint32_t pk[32];
          if (attends) {
            // all 64 + 64 values into registers, then S and dP are handed back to the tensor core at once
            uint32_t sv[64], dp[64];
            tmem_ld32(ts, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
            tmem_ld32(ts + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
            tmem_ld32(tdp, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
            tmem_ld32(tdp + 32, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(s32(&sm.sdp_free[t]));
#pragma unroll
            for (int i = 0; i < 64; i += 2) {
              float x0, x1, d0, d1;
              unpack2(fma2(pack2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), scale2, neg_lse2), x0, x1);
              const uint64_t dmd = add2(pack2(__uint_as_float(dp[i]), __uint_as_float(dp[i + 1])), neg_d2);
              unpack2(mul2(pack2(ex2(x0), ex2(x1)), dmd), d0, d1);
              pk[i >> 1] = pack2<F16>(d0, d1);
            }
          } else {
            tc_fence_before();
            mbar_arrive(s32(&sm.sdp_free[t]));
#pragma unroll
            for (int i = 0; i < 32; ++i) pk[i] = 0u;
          }
          // dS has one buffer: the previous product's dQ += dS K must have consumed it
          if (done > 0) {
            ok = mbar_wait(s32(&sm.pv_done[t]), (nt - 1) & 1, abort, status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
          }
          tmem_st32(tds, pk);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(s32(&sm.p_full[t]));
          ++nt;
          ++done;
        }
      }
      if (!ok) break;
      if (done > 0) {
        ok = mbar_wait(s32(&sm.pv_done[t]), (nt - 1) & 1, abort, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (valid) {
          uint4* dst = reinterpret_cast<uint4*>(dq + tok * kD);
#pragma unroll
          for (int part = 0; part < 2; ++part) {
            uint32_t ov[32];
            tmem_ld32(tdq + 32 * part, ov);
            tmem_wait_ld();
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
              w[i] = pack2<F16>(__uint_as_float(ov[2 * i]) * g.scale, __uint_as_float(ov[2 * i + 1]) * g.scale);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[part * 4 + i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          }
        }
      } else if (valid) {
        // a tile whose rows attend nothing (possible when the local set is switched off): zero gradient
        uint4* dst = reinterpret_cast<uint4*>(dq + tok * kD);
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s32(&sm.list_empty[buf]));
    }
  }
  cta_tmem_free(warp == 9, tmem, kTmemCols);
}

// `work_counter` must be zero when the kernel starts (a word of the workspace status block).
template <bool F16>
static int launch_dq_tc_t(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* D, const int32_t* block_idx, void* dq, int* work_counter) {
  const Geo& g = c.g;
  CUtensorMap mq, mdo, mk, mv;
  if (!make_map(&mq, q, g, g.U) || !make_map(&mdo, d_o, g, g.U) || !make_map(&mk, k, g, g.Ukv) || !make_map(&mv, v, g, g.Ukv))
    return MOSAIC_E_CUDA;
  const size_t smem = sizeof(Smem) + 1024;
  static unsigned long long configured = 0;  // devices on which the kernel's shared-memory opt-in is set
  int sms = 0;
  if (const int rc = launch_setup(reinterpret_cast<const void*>(dq_tc_kernel<F16>), smem, &configured, &sms)) return rc;
  const int ipu = items_per_unit(g);
  const long long total = (long long)g.U * ipu;
  if (total > 0x7fffff00ll) return MOSAIC_E_UNSUPPORTED;
  const long long grid = total < (long long)sms ? total : (long long)sms;
  dq_tc_kernel<F16><<<(unsigned)grid, kThreads, smem, c.stream>>>(g, mq, mdo, mk, mv, block_idx, lse, D,
                                                             (__nv_bfloat16*)dq, c.status, work_counter, ipu,
                                                             (int)total);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_dq_tc(const HostCtx& c, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* D, const int32_t* block_idx, void* dq, int* work_counter) {
  return c.g.f16 ? launch_dq_tc_t<true>(c, q, k, v, d_o, lse, D, block_idx, dq, work_counter) : launch_dq_tc_t<false>(c, q, k, v, d_o, lse, D, block_idx, dq, work_counter);
}

}  // namespace mosaic
