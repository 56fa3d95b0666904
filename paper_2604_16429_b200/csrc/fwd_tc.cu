// Forward of the block-sparse attention on Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// Paper: fine-grained attention equation of the "Selection" paragraph (section "Block-Sparse
// Attention"), evaluated over the union of the local neighbourhood and the selected blocks with one
// softmax; streaming evaluation with the query tile resident on chip and key/value blocks streamed
// through, as the appendix paragraph "Kernel Design" describes.
//
// Work item = 256 query rows = two 128-row tiles = four 64-row "halves", each half one 64-token chunk
// of a query block:
//   * 64-token blocks (8x8): a 2x2 group of query blocks (a 1x4 group on an odd last block row); the
//     CTA walks the UNION of the four key lists, every entry carrying a 4-bit mask of the halves that
//     attend it.  A tile skips entries none of its halves attends; a half that does not attend an entry
//     its tile computes writes P = 0.
//   * 128-token blocks: two neighbouring query blocks; larger blocks: four chunks of one block.
// Key/value data moves in 64-token chunks: one 4-D TMA box {d, bw, 64/bw, 1} of the [U, nlat, nlon, d]
// view lands as 64 rows x 128 B in 128-byte-swizzled shared memory, which is at once the K-major
// operand layout for S = Q K^T and the MN-major operand layout for O += P V.  A staged chunk serves
// both tiles of the item.
//
// The kernel is persistent: one CTA per SM draws items from a counter in the workspace.
// Warp roles (384 threads): warps 0-3 softmax of tile 0, warps 4-7 softmax of tile 1 (thread = query
// row = TMEM lane), warp 8 issues TMA, warps 9 and 10 issue tcgen05.mma for tile 0 and tile 1 (the whole
// warp walks the loop, one elected lane issues), warp 11 draws items from the queue and builds their key
// lists one item ahead, interleaved so that both tiles find work all along a list.
// TMEM (512 columns): O of tile t at 64 t (fp32, 64 columns); two S buffers per tile at 128 + 128 t + 64 b
// (fp32, 64 columns each); the query tile of tile t (bf16, 32 columns) at 384 + 32 t.  P (bf16) overwrites
// the first 32 columns of its S buffer and is the TMEM A operand of PV.  The query tile is a TMEM A operand
// too: the softmax threads copy their rows there once per item, so QK^T reads only the key chunk from shared
// memory (with both operands in shared memory an N = 64 product is bound by shared-memory bandwidth, not by
// the tensor core).  QK^T of product n+1 is issued before P V of product n, so the tensor core fills one S
// buffer while the softmax warps work on the other.
// Softmax: fp32, base-2 exponentials with the scale folded in, running maximum moved only when it grows by
// more than 2^8 (then O is rescaled, between two P V products), packed two-lane fp32 arithmetic, and a
// quarter of the exponentials evaluated by a cubic on the FMA pipe because at d = 64 the MUFU pipe
// (16 ex2 per clock per SM against 8192 tensor FLOP per clock) is the limiter, not the tensor core.
// Every mbarrier wait is bounded; on expiry the CTA records MOSAIC_E_DEVICE_TIMEOUT and drains.


#include "tc_common.cuh"

namespace mosaic {

namespace {

constexpr int kStages = 8;                       // key/value ring depth (K + V chunk per stage)
constexpr int kThreads = 384;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 0, kColS = 128;       // O of tile t at 64 t; S buffer b of tile t at 128 + 128 t + 64 b
constexpr uint32_t kColQ = 384;                  // query tile of tile t (bf16 pairs) at 384 + 32 t
constexpr int kPolyEvery = 2;                   // one pair in every kPolyEvery groups of four logits takes the FMA-pipe exp2
constexpr float kRescaleThreshold = 8.0f;        // log2 units: P stays below 2^8

struct Smem {
  unsigned char q[2][2][2 * kTile];        // [item parity][tile][128 rows x 128 B]
  unsigned char kv[kStages][2][kTile];     // [stage][K, V]
  unsigned long long kv_full[kStages], kv_empty[kStages];
  unsigned long long q_full[2][2], q_empty[2][2];  // [item parity][tile]
  unsigned long long mma_drain_bar[2];             // abort path: completion of each issuer's outstanding products
  unsigned long long q_ready[2];                   // [tile]: the item's query rows are in TMEM
  unsigned long long s_full[2][2], p_full[2][2], pv_done[2][2];  // [tile][S buffer]
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
    fwd_tc_kernel(const Geo g, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ block_idx,
                  __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int* status, int* work_counter,
                  int ipu, int total_items) {
  extern __shared__ unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(s32(&sm.kv_full[s]), 1); mbar_init(s32(&sm.kv_empty[s]), 2); }
    for (int t = 0; t < 2; ++t) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(s32(&sm.q_full[b][t]), 1);
        if (t == 0) mbar_init(s32(&sm.mma_drain_bar[b]), 1);
        mbar_init(s32(&sm.q_empty[b][t]), 128);
      }
      mbar_init(s32(&sm.q_ready[t]), 128);
      for (int b = 0; b < 2; ++b) {
        mbar_init(s32(&sm.s_full[t][b]), 1);
        mbar_init(s32(&sm.p_full[t][b]), 128);
        mbar_init(s32(&sm.pv_done[t][b]), 1);
      }
    }
    for (int i = 0; i < kLists; ++i) {
      mbar_init(s32(&sm.list_full[i]), 1);
      mbar_init(s32(&sm.list_empty[i]), 11);  // 8 softmax warps + 2 MMA warps + TMA producer
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
      int q_armed[2][2] = {{-1, -1}, {-1, -1}};  // phase parity of the last load into each query-tile buffer
      bool ok = true;
      for (int it = 0; ok; ++it) {
        const int buf = it % kLists, qb = it & 1;
        ok = mbar_wait(s32(&sm.list_full[buf]), (it / kLists) & 1, abort, status);
        if (!ok) break;
        const ItemInfo& inf = sm.info[buf];
        const int n = inf.n, u = inf.unit;
        if (n < 0) break;
        const int ukv = kv_unit(g, u);  // key/value head of this query head's group
        // query tiles (double-buffered by item parity): free once the softmax threads have copied the rows of
        // the item before the previous one to TMEM, so this load runs while the previous item still computes
        for (int t = 0; t < 2 && ok; ++t) {
          ok = mbar_wait(s32(&sm.q_empty[qb][t]), ((it >> 1) & 1) ^ 1, abort, status);
          if (!ok) break;
          mbar_expect_tx(s32(&sm.q_full[qb][t]), 2 * kTile);
          q_armed[qb][t] = (it >> 1) & 1;
          for (int hh = 0; hh < 2; ++hh) {
            const int h = 2 * t + hh, by = inf.hb[h] / g.nbw, bx = inf.hb[h] - by * g.nbw;
            tma_load_4d(s32(sm.q[qb][t] + hh * kTile), &map_q, s32(&sm.q_full[qb][t]), 0, bx * g.bw,
                        by * g.bh + inf.hc[h] * g.crows, u);
          }
        }
        for (int e = 0; e < n && ok; ++e) {
          const int j = sm.ids[buf][e], by = j / g.nbw, bx = j - by * g.nbw;
          const uint32_t mk = sm.mask[buf][e];
          for (int c = 0; c < g.cpb; ++c, ++step) {
            const int st = (int)(step % kStages);
            ok = mbar_wait(s32(&sm.kv_empty[st]), (uint32_t)((step / kStages) & 1) ^ 1, abort, status);
            if (!ok) break;
            mbar_expect_tx(s32(&sm.kv_full[st]), 2 * kTile);
            tma_load_4d(s32(sm.kv[st][0]), &map_k, s32(&sm.kv_full[st]), 0, bx * g.bw, by * g.bh + c * g.crows, ukv);
            tma_load_4d(s32(sm.kv[st][1]), &map_v, s32(&sm.kv_full[st]), 0, bx * g.bw, by * g.bh + c * g.crows, ukv);
            // a tile that does not attend this entry never looks at the stage: its release is given here (the other
            // tile's release, after its P V, is what lets the stage be reused)
            if (!(mk & 3u)) mbar_arrive(s32(&sm.kv_empty[st]));
            if (!(mk & 12u)) mbar_arrive(s32(&sm.kv_empty[st]));
          }
        }
        if (ok) mbar_arrive(s32(&sm.list_empty[buf]));
      }
      if (*abort) {  // copies this thread issued must land before the CTA's memory is released
        const long long first = step > kStages ? step - kStages : 0;
        for (long long s = first; s < step; ++s) mbar_drain(s32(&sm.kv_full[s % kStages]), (uint32_t)((s / kStages) & 1));
        for (int i = 0; i < 4; ++i)
          if (q_armed[i >> 1][i & 1] >= 0) mbar_drain(s32(&sm.q_full[i >> 1][i & 1]), (uint32_t)q_armed[i >> 1][i & 1]);
      } else {       // drain: the last uses of every ring stage have been released by both tiles
        const long long first = step > kStages ? step - kStages : 0;
        for (long long s = first; s < step; ++s)
          if (!mbar_wait(s32(&sm.kv_empty[s % kStages]), (uint32_t)((s / kStages) & 1), abort, status)) break;
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------------------------------------- MMA issuer of tile t
    // The whole warp walks the loop (waits are cheap polls); one elected lane issues the tensor-core
    // instructions, so operands that are the same for the warp stay in uniform registers.
    // S is double-buffered: QK^T of product n+1 is issued before P V of product n, so the tensor core
    // fills the next S while the softmax warps work on the current one.
    const int t = warp - 9;
    constexpr uint32_t idesc_qk = make_idesc(false, 64u, F16), idesc_pv = make_idesc(true, 64u, F16);
    const uint32_t tcol_o = tmem + kColO + 64 * t, tcol_s = tmem + kColS + 128 * t, tcol_q = tmem + kColQ + 32 * t;
    const uint32_t tbits = 3u << (2 * t);
    long long step = 0;   // ring position (all chunks, attended by this tile or not)
    uint32_t nt = 0;      // products issued by this tile so far: buffer nt & 1, phase (nt >> 1) & 1
    bool ok = true;
    // P V of product `pn` (its V chunk sits in ring stage `pst`); `pfirst` starts a new accumulation
    auto issue_pv = [&](uint32_t pn, int pst, bool pfirst) {
      const uint32_t b = pn & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.p_full[t][b]), (pn >> 1) & 1, abort, status));
      if (!ok) return;
      tc_fence_after();
      const uint64_t vdesc = smem_desc(s32(sm.kv[pst][1]));
      const uint32_t pcol = tcol_s + 64 * b;
      if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_ts(tcol_o, pcol + 8 * kk, vdesc + (uint64_t)((2048 * kk) >> 4), idesc_pv, (!pfirst || kk > 0));
        tc_commit(s32(&sm.kv_empty[pst]));
        tc_commit(s32(&sm.pv_done[t][b]));
      }
      __syncwarp();
    };
    for (int it = 0; ok; ++it) {
      const int buf = it % kLists;
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.list_full[buf]), (it / kLists) & 1, abort, status));
      if (!ok) break;
      const int n = sm.info[buf].n;
      if (n < 0) break;
      // the item's query rows are in TMEM (copied there by the softmax threads)
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.q_ready[t]), it & 1, abort, status));
      if (!ok) break;
      bool first = true, pend = false, pend_first = false;
      uint32_t pend_n = 0;
      int pend_st = 0;
      for (int e = 0; e < n && ok; ++e) {
        if (!(sm.mask[buf][e] & tbits)) { step += g.cpb; continue; }  // not attended: the producer released the stages
        for (int c = 0; c < g.cpb && ok; ++c, ++step) {
          const int st = (int)(step % kStages);
          ok = __all_sync(0xffffffffu,
                          mbar_wait(s32(&sm.kv_full[st]), (uint32_t)((step / kStages) & 1), abort, status));
          if (!ok) break;
          // S buffer nt & 1 (aliased by P) was last read by P V of product nt - 2, which this warp issued
          // earlier: tensor-core operations of one thread execute in issue order, so this QK^T cannot
          // overwrite the buffer before that product has consumed it, and no wait is needed here
          const uint32_t b = nt & 1;
          tc_fence_after();
          const uint64_t kdesc = smem_desc(s32(sm.kv[st][0]));
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_ts(tcol_s + 64 * b, tcol_q + 8 * kk, kdesc + 2 * kk, idesc_qk, kk > 0);
            tc_commit(s32(&sm.s_full[t][b]));
          }
          __syncwarp();
          if (pend) issue_pv(pend_n, pend_st, pend_first);
          pend = true; pend_n = nt; pend_st = st; pend_first = first;
          first = false;
          ++nt;
        }
      }
      if (ok && pend) issue_pv(pend_n, pend_st, pend_first);  // the item's last product
      if (ok && elect_one()) mbar_arrive(s32(&sm.list_empty[buf]));
    }
    if (*abort) {  // products already issued must finish before TMEM and shared memory are released
      if (elect_one()) mma_drain(s32(&sm.mma_drain_bar[t]));
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------- softmax of tile t, then epilogue
    const int t = warp >> 2;        // tile
    const int hh = (warp >> 1) & 1; // 64-row half of the tile this warp's rows belong to
    const int h = 2 * t + hh;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t ts = tmem + lane_off + kColS + 128 * t, to = tmem + lane_off + kColO + 64 * t;
    const uint32_t tq = tmem + lane_off + kColQ + 32 * t;
    const uint32_t tbits = 3u << (2 * t), hbit = 1u << h;
    const uint64_t scale2 = pack2(g.scale_log2, g.scale_log2);
    uint32_t nt = 0;
    bool ok = true;
    // Copies this thread's query row of item `it2` from shared memory (128-byte swizzled rows) to TMEM, where it is
    // the A operand of the item's QK^T products.  Called when every QK^T of the previous item has completed.
    // Returns the item's list length (-1: no more work).
    auto stage_q = [&](int it2) -> int {
      const int buf2 = it2 % kLists, qb2 = it2 & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.list_full[buf2]), (it2 / kLists) & 1, abort, status));
      if (!ok) return -1;
      const int n2 = sm.info[buf2].n;
      if (n2 < 0) return -1;
      ok = __all_sync(0xffffffffu, mbar_wait(s32(&sm.q_full[qb2][t]), (it2 >> 1) & 1, abort, status));
      if (!ok) return -1;
      const int r = tid & 127;  // row of the tile; rows 0-63 and 64-127 are two 8 KB chunks
      const unsigned char* rowp = sm.q[qb2][t] + (r >> 6) * kTile + (r & 63) * 128;
      uint32_t qv[32];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(rowp + ((c ^ (r & 7)) << 4));
        qv[4 * c] = v.x; qv[4 * c + 1] = v.y; qv[4 * c + 2] = v.z; qv[4 * c + 3] = v.w;
      }
      tmem_st32(tq, qv);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(s32(&sm.q_ready[t]));
      mbar_arrive(s32(&sm.q_empty[qb2][t]));
      return n2;
    };
    int n = stage_q(0);
    for (int it = 0; ok && n >= 0; ++it) {
      const int buf = it % kLists;
      float m_ref = -INFINITY, l = 0.f;
      uint32_t done = 0;
      for (int e = 0; e < n && ok; ++e) {
        const uint32_t mk = sm.mask[buf][e];
        if (!(mk & tbits)) continue;
        const bool attends = (mk & hbit) != 0;
        for (int c = 0; c < g.cpb; ++c) {
          const uint32_t b = nt & 1, tsb = ts + 64 * b;
          ok = mbar_wait(s32(&sm.s_full[t][b]), (nt >> 1) & 1, abort, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          if (attends) {
            uint32_t sa[32], sb[32];
            tmem_ld32(tsb, sa);
            tmem_ld32(tsb + 32, sb);
            tmem_wait_ld();
            float mx0 = __uint_as_float(sa[0]), mx1 = __uint_as_float(sa[1]), mx2 = __uint_as_float(sb[0]),
                  mx3 = __uint_as_float(sb[1]);
#pragma unroll
            for (int i = 2; i < 32; i += 2) {
              if (i & 2) {
                mx0 = max3(mx0, __uint_as_float(sa[i]), __uint_as_float(sa[i + 1]));
                mx2 = max3(mx2, __uint_as_float(sb[i]), __uint_as_float(sb[i + 1]));
              } else {
                mx1 = max3(mx1, __uint_as_float(sa[i]), __uint_as_float(sa[i + 1]));
                mx3 = max3(mx3, __uint_as_float(sb[i]), __uint_as_float(sb[i + 1]));
              }
            }
            const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * g.scale_log2;  // scale > 0 commutes with max
            bool need = false;
            float alpha = 1.f;
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
            uint32_t pk[32];
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              float x0, x1, x2, x3;
              const uint64_t y01 = fma2(pack2(__uint_as_float(sa[i]), __uint_as_float(sa[i + 1])), scale2, negm2);
              const uint64_t y23 = fma2(pack2(__uint_as_float(sa[i + 2]), __uint_as_float(sa[i + 3])), scale2, negm2);
              unpack2(y01, x0, x1);
              unpack2(y23, x2, x3);
              float p0 = ex2(x0), p1 = ex2(x1), p2, p3;
              if ((i >> 2) % kPolyEvery == kPolyEvery - 1) { ex2_poly2(y23, p2, p3); } else { p2 = ex2(x2); p3 = ex2(x3); }
              sum_a = add2(sum_a, pack2(p0, p1));
              sum_b = add2(sum_b, pack2(p2, p3));
              pk[i >> 1] = pack2<F16>(p0, p1);
              pk[(i >> 1) + 1] = pack2<F16>(p2, p3);
            }
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              float x0, x1, x2, x3;
              const uint64_t y01 = fma2(pack2(__uint_as_float(sb[i]), __uint_as_float(sb[i + 1])), scale2, negm2);
              const uint64_t y23 = fma2(pack2(__uint_as_float(sb[i + 2]), __uint_as_float(sb[i + 3])), scale2, negm2);
              unpack2(y01, x0, x1);
              unpack2(y23, x2, x3);
              float p0 = ex2(x0), p1 = ex2(x1), p2, p3;
              if ((i >> 2) % kPolyEvery == kPolyEvery - 1) { ex2_poly2(y23, p2, p3); } else { p2 = ex2(x2); p3 = ex2(x3); }
              sum_a = add2(sum_a, pack2(p0, p1));
              sum_b = add2(sum_b, pack2(p2, p3));
              pk[16 + (i >> 1)] = pack2<F16>(p0, p1);
              pk[16 + (i >> 1) + 1] = pack2<F16>(p2, p3);
            }
            tmem_st32(tsb, pk);  // P (bf16 pairs) over the first 32 columns of this S buffer
            float s0, s1;
            unpack2(add2(sum_a, sum_b), s0, s1);
            l += s0 + s1;
            if (__any_sync(0xffffffffu, need)) {
              // the accumulator may only be touched between P V products: wait for the previous one
              if (done > 0) {
                ok = mbar_wait(s32(&sm.pv_done[t][b ^ 1]), ((nt - 1) >> 1) & 1, abort, status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
              }
              const uint64_t alpha2 = pack2(alpha, alpha);
#pragma unroll
              for (int part = 0; part < 2; ++part) {
                uint32_t ov[32];
                tmem_ld32(to + 32 * part, ov);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                  float a, bb;
                  unpack2(mul2(pack2(__uint_as_float(ov[i]), __uint_as_float(ov[i + 1])), alpha2), a, bb);
                  ov[i] = __float_as_uint(a);
                  ov[i + 1] = __float_as_uint(bb);
                }
                tmem_st32(to + 32 * part, ov);
              }
            }
          } else {
            uint32_t z[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) z[i] = 0u;
            tmem_st32(tsb, z);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(s32(&sm.p_full[t][b]));
          ++nt;
          ++done;
        }
      }
      if (!ok) break;
      // every QK^T of this item has completed (its S was received): the next item's query rows can go to TMEM,
      // and its first products run while this item's output is written
      const int n_next = stage_q(it + 1);
      if (!ok) break;
      if (done > 0) {
        ok = mbar_wait(s32(&sm.pv_done[t][(nt - 1) & 1]), ((nt - 1) >> 1) & 1, abort, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if ((sm.info[buf].hvalid >> h) & 1) {
          const int e = tid & 63;
          const long long tok =
              (long long)sm.info[buf].unit * g.N + chunk_token(g, sm.info[buf].hb[h], sm.info[buf].hc[h], e);
          const float inv = l > 0.f ? 1.f / l : 0.f;  // a row that attends nothing (empty selection): O = 0
          uint4* dst = reinterpret_cast<uint4*>(o + tok * kD);
#pragma unroll
          for (int part = 0; part < 2; ++part) {
            uint32_t ov[32];
            tmem_ld32(to + 32 * part, ov);
            tmem_wait_ld();
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
              w[i] = pack2<F16>(__uint_as_float(ov[2 * i]) * inv, __uint_as_float(ov[2 * i + 1]) * inv);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[part * 4 + i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          }
          lse[tok] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
        }
      } else if ((sm.info[buf].hvalid >> h) & 1) {
        // the tile attends nothing in this item (selection branch with empty rows): O = 0, log-sum-exp = -inf
        const long long tok =
            (long long)sm.info[buf].unit * g.N + chunk_token(g, sm.info[buf].hb[h], sm.info[buf].hc[h], tid & 63);
        uint4* dst = reinterpret_cast<uint4*>(o + tok * kD);
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        lse[tok] = -INFINITY;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s32(&sm.list_empty[buf]));
      n = n_next;
    }
  }
  cta_tmem_free(warp == 9, tmem, kTmemCols);
}

// ---------------------------------------------------------------------------------------------
namespace {
template <bool F16>
int launch_fwd_tc_t(const HostCtx& c, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                    const int32_t* block_idx, void* o, float* lse, int* work_counter) {
  const Geo& g = c.g;
  const size_t smem = sizeof(Smem) + 1024;
  static unsigned long long configured = 0;  // devices on which the kernel's shared-memory opt-in is set
  int sms = 0;
  if (const int rc = launch_setup(reinterpret_cast<const void*>(fwd_tc_kernel<F16>), smem, &configured, &sms)) return rc;
  const int ipu = items_per_unit(g);
  const long long total = (long long)g.U * ipu;
  if (total > 0x7fffff00ll) return MOSAIC_E_UNSUPPORTED;
  const long long grid = total < (long long)sms ? total : (long long)sms;
  fwd_tc_kernel<F16><<<(unsigned)grid, kThreads, smem, c.stream>>>(g, mq, mk, mv, block_idx, (__nv_bfloat16*)o, lse,
                                                                  c.status, work_counter, ipu, (int)total);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}
}  // namespace

// `work_counter` must be zero when the kernel starts (a word of the workspace status block).
int launch_fwd_tc(const HostCtx& c, const void* q, const void* k, const void* v, const int32_t* block_idx, void* o,
                  float* lse, int* work_counter) {
  const Geo& g = c.g;
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, q, g, g.U) || !make_map(&mk, k, g, g.Ukv) || !make_map(&mv, v, g, g.Ukv)) return MOSAIC_E_CUDA;
  return g.f16 ? launch_fwd_tc_t<true>(c, mq, mk, mv, block_idx, o, lse, work_counter)
               : launch_fwd_tc_t<false>(c, mq, mk, mv, block_idx, o, lse, work_counter);
}

}  // namespace mosaic
