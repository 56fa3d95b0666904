// Selection: block pooling, block-level scores, per-query-block top-k.
//
// Paper, section "Block-Sparse Attention": paragraph "Compression" defines the pooled block
// representations (phi = mean pooling) and the block-level score; paragraph "Selection" takes the
// top-n key blocks per query block.  The mean's 1/b, the 1/sqrt(d_k) and the row softmax are
// strictly increasing, so ranking the raw dot product of block SUMS gives the same blocks.
//
// Arithmetic is fixed so that the chosen ids are unique and reproducible bit for bit:
//   pooled sum  = fp64 accumulation over the block's tokens in row-major order, one rounding to fp32
//   score       = fp64 accumulation over channels 0..d-1 of the exact products of two fp32 values
//   order       = (score descending, block id ascending); +0 == -0; a NaN ranks last
#include "common.cuh"

namespace mosaic {

// ------------------------------------------------------------------------------------------
// pool_kernel: eight lanes per (tensor, unit, block), four blocks per warp; a lane owns eight
// consecutive channels (one 16-byte load per token) and adds them in token order, row-major inside
// the block, so every channel is one sequential fp64 chain.  HBM-bound: reads 2*U*N*d*2 bytes once;
// the loads of a whole block row are in flight together.  Beside the pooled sums it writes an upper
// bound of each pooled vector's Euclidean norm, which the ranking kernel's screening pass needs.
// ------------------------------------------------------------------------------------------
template <int BW>
__global__ void __launch_bounds__(256) pool_kernel(Geo g, const uint4* __restrict__ q, const uint4* __restrict__ k,
                                                   float* __restrict__ pq, float* __restrict__ pk,
                                                   float* __restrict__ nq, float* __restrict__ nk, int ntens, int units) {
  const int sub = threadIdx.x & 7;  // which 8 channels
  const long long grp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  const long long per_tensor = (long long)units * g.m;
  const bool live = grp < ntens * per_tensor;  // the last warp may be partly idle; it still takes part in the shuffles
  const int which = live && grp >= per_tensor;
  const long long w = live ? grp - which * per_tensor : 0;
  const int u = (int)(w / g.m), j = (int)(w - (long long)u * g.m);
  const uint4* src = (which ? k : q) + (long long)u * g.N * (kD / 8) + sub;
  const int by = j / g.nbw, bx = j - by * g.nbw;
  double acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.0;
  for (int r = 0; r < g.bh && live; ++r) {
    const uint4* row = src + ((long long)(by * g.bh + r) * g.nlon + bx * BW) * (kD / 8);
    uint4 v[BW];
#pragma unroll
    for (int c = 0; c < BW; ++c) v[c] = __ldg(row + c * (kD / 8));
#pragma unroll
    for (int c = 0; c < BW; ++c) {
      const uint32_t x[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float lo, hi;
        unpack16x2(x[e], g.f16 != 0, lo, hi);
        acc[2 * e] += (double)lo;
        acc[2 * e + 1] += (double)hi;
      }
    }
  }
  float p[8];
  double ss = 0.0;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    p[c] = (float)acc[c];
    ss += (double)p[c] * (double)p[c];
  }
  ss += __shfl_xor_sync(0xffffffffu, ss, 1);
  ss += __shfl_xor_sync(0xffffffffu, ss, 2);
  ss += __shfl_xor_sync(0xffffffffu, ss, 4);
  if (!live) return;
  float4* dst = reinterpret_cast<float4*>((which ? pk : pq) + ((long long)u * g.m + j) * kD + 8 * sub);
  dst[0] = make_float4(p[0], p[1], p[2], p[3]);
  dst[1] = make_float4(p[4], p[5], p[6], p[7]);
  // rounded up twice, so that it is never below the norm of the fp32 vector (NaN and inf pass through)
  if (sub == 0) (which ? nk : nq)[(long long)u * g.m + j] = __fmul_ru(__double2float_ru(sqrt(ss)), 1.000001f);
}

// ------------------------------------------------------------------------------------------
// topk_kernel<NW, RI, CAP>: ranking of the key blocks of NW * RI query blocks of one unit (warp w owns RI
// rows; a lane owns the keys lane, lane + 32, ... of every 128-key chunk that streams through shared memory).
//
// The ids must be those of the exact fp64 scores, but almost all of the m scores of a row are irrelevant,
// so the kernel screens in fp32 and scores exactly only what survives:
//   1. screening score  s~ = fp32 FMA chain over the channels.  |s~ - s| <= gamma_64 * sum|a_c||b_c|
//      <= 2^-18 (1 + 1e-5) |a||b|  (standard bound of a length-64 dot product, any order, FMA or not;
//      Cauchy-Schwarz).  The kernel uses eps = 2^-16 * na * nb + 1e-37 with the norm bounds of the pooling
//      kernel: four times the bound, which also covers the rounding of s~ -+ eps and subnormal products.
//      A non-finite s~ or eps makes the candidate's interval (-inf, +inf).
//   2. every lane tracks the two largest lower bounds s~ - eps among its own keys; the k-th largest of
//      those 64 values is a lower bound thr of the row's k-th best exact score (they belong to k distinct
//      candidates).  A candidate with s~ + eps < thr is worse than k others whatever the ties: dropped.
//      Chunks are visited from the CTA's own neighbourhood outwards (on smooth fields the best keys are
//      near, so the threshold is tight at once); the first chunk is screened twice, first for a threshold only.
//   3. survivors (id and upper bound) collect in shared memory, pruned when thr has risen; a row whose
//      survivors overflow (massive ties) falls back to scoring every key exactly.
//   4. exact phase: the fp64 chain of the selection's definition for every survivor of the warp's rows
//      (lanes take survivors, two chains in flight each), then each row ranks its survivors by
//      (score descending, id ascending) by counting, and ranks 0..k-1 are written.
// ------------------------------------------------------------------------------------------

// Total-order key: larger key = better score.  0 = not a candidate, 1 = NaN.
__device__ __forceinline__ unsigned long long score_key(double s) {
  if (s != s) return 1ull;
  s += 0.0;  // -0 -> +0
  unsigned long long b = (unsigned long long)__double_as_longlong(s);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

// does (ka, ia) rank before (kb, ib)?
__device__ __forceinline__ bool ranks_before(unsigned long long ka, int ia, unsigned long long kb, int ib) {
  return ka > kb || (ka == kb && ia < ib);
}

// order-preserving map of non-NaN floats to unsigned integers
__device__ __forceinline__ unsigned ordered_bits(float f) {
  const unsigned b = __float_as_uint(f);
  return (b >> 31) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(unsigned o) {
  return __uint_as_float((o >> 31) ? (o & 0x7fffffffu) : ~o);
}

constexpr int kKStr = kD + 4;   // padded row of the staged vectors (floats): 16-byte reads of one row per lane hit every bank once

template <int NW, int RI, int CAP, int JT>
struct TopkSmem {
  union {
    struct {
      float ks[2][JT][kKStr];  // pooled keys of two chunks (one being read, one in flight)
      float nk[2][JT];         // their norm bounds
    } scr;
    unsigned long long ekey[NW * RI][CAP];  // exact phase: score keys of the rows' survivors (every row that did not overflow)
  };
  float qs[NW * RI][kKStr];     // pooled queries of this CTA
  int surv[NW * RI][CAP];       // surviving key ids per row ...
  float surv_ub[NW * RI][CAP];  // ... and the upper bound of their score
};

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
  const unsigned n = valid ? 16u : 0u;  // 0 source bytes: the destination is filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((unsigned)__cvta_generic_to_shared(dst)),
               "l"(src), "r"(n)
               : "memory");
}
__device__ __forceinline__ void cp_async4(void* dst, const void* src, bool valid) {
  const unsigned n = valid ? 4u : 0u;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((unsigned)__cvta_generic_to_shared(dst)),
               "l"(src), "r"(n)
               : "memory");
}

// The warp's sorted list of the best candidates so far holds one entry per lane (lane r = rank r).  Offers this
// lane's candidate (key 0 = none) together with those of the other lanes; every candidate that belongs to the k
// best is inserted.
__device__ __forceinline__ void insert_batch(unsigned long long key, int id, unsigned long long& lkey, int& lid, int k,
                                             int lane) {
  while (true) {
    // warp-wide best remaining candidate: maximum of the key's high word, then of the low word among the lanes
    // that hold that high word, then the lowest id among the lanes that hold the key
    const unsigned hi = (unsigned)(key >> 32), lo = (unsigned)key;
    const unsigned mh = __reduce_max_sync(0xffffffffu, hi);
    const unsigned ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    const unsigned long long bk = ((unsigned long long)mh << 32) | ml;
    if (bk == 0ull) return;
    const int bj = (int)__reduce_min_sync(0xffffffffu, key == bk ? (unsigned)id : 0x7fffffffu);
    const unsigned long long tk = __shfl_sync(0xffffffffu, lkey, k - 1);
    const int ti = __shfl_sync(0xffffffffu, lid, k - 1);
    if (!(tk == 0ull || ranks_before(bk, bj, tk, ti))) return;  // the batch's best does not enter: nothing does
    const bool before = lkey != 0ull && ranks_before(lkey, lid, bk, bj);
    const int p = __popc(__ballot_sync(0xffffffffu, before));
    const unsigned long long uk = __shfl_up_sync(0xffffffffu, lkey, 1);
    const int ui = __shfl_up_sync(0xffffffffu, lid, 1);
    if (lane == p) { lkey = bk; lid = bj; }
    else if (lane > p) { lkey = uk; lid = ui; }
    if (key == bk && id == bj) key = 0ull;  // taken
  }
}

// exact score of (pooled query row in shared memory, pooled key row j in global memory) as a sortable key
__device__ __forceinline__ unsigned long long exact_key(const float* qrow, const float* __restrict__ pk_u, int j) {
  const float4* krow = reinterpret_cast<const float4*>(pk_u + (long long)j * kD);
  double s = 0.0;
#pragma unroll
  for (int half = 0; half < 2; ++half) {  // eight 16-byte loads in flight, then their 32 sequential FMAs
    float4 kv[kD / 8];
#pragma unroll
    for (int c4 = 0; c4 < kD / 8; ++c4) kv[c4] = __ldg(krow + half * (kD / 8) + c4);
#pragma unroll
    for (int c4 = 0; c4 < kD / 8; ++c4) {
      const float4 qv = *reinterpret_cast<const float4*>(qrow + 4 * (half * (kD / 8) + c4));
      s = fma((double)qv.x, (double)kv[c4].x, s);
      s = fma((double)qv.y, (double)kv[c4].y, s);
      s = fma((double)qv.z, (double)kv[c4].z, s);
      s = fma((double)qv.w, (double)kv[c4].w, s);
    }
  }
  return score_key(s);
}

template <int NW, int RI, int CAP, int JT, int MB>
__global__ void __launch_bounds__(NW * 32, MB) topk_kernel(Geo g, const float* __restrict__ pq,
                                                       const float* __restrict__ pk, const float* __restrict__ nq,
                                                       const float* __restrict__ nk, int32_t* __restrict__ block_idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  using SM = TopkSmem<NW, RI, CAP, JT>;
  SM& sm = *reinterpret_cast<SM*>(smem_raw);
  constexpr int TI = NW * RI, NT = NW * 32, KB = JT / 32;  // KB: keys of a chunk per lane
  const float kInf = __int_as_float(0x7f800000);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tiles = (g.m + TI - 1) / TI;
  const int u = blockIdx.x / tiles, i0 = (blockIdx.x - u * tiles) * TI;
  const float* pq_u = pq + (long long)u * g.m * kD;
  const float* pk_u = pk + (long long)kv_unit(g, u) * g.m * kD;   // grouped-query attention: the group's key head
  const float* nk_u = nk + (long long)kv_unit(g, u) * g.m;
  const int nchunks = (g.m + JT - 1) / JT;

  auto load_chunk = [&](int ch, int buf) {
    const int j0 = ch * JT;
    for (int e = tid; e < JT * (kD / 4); e += NT) {
      const int jj = e / (kD / 4), c4 = e - jj * (kD / 4);
      const bool valid = j0 + jj < g.m;
      cp_async16(&sm.scr.ks[buf][jj][4 * c4], pk_u + (long long)(valid ? j0 + jj : 0) * kD + 4 * c4, valid);
    }
    for (int jj = tid; jj < JT; jj += NT) {
      const bool valid = j0 + jj < g.m;
      cp_async4(&sm.scr.nk[buf][jj], nk_u + (valid ? j0 + jj : 0), valid);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // visiting order: the chunk that holds the middle of this CTA's rows, then alternately the next one above and
  // below (every chunk once).  seq_next() hands out that sequence.
  const int c_home = min((i0 + TI / 2) / JT, nchunks - 1);
  int seq_lo = c_home - 1, seq_hi = c_home + 1, seq_n = 0;
  auto seq_next = [&]() {
    int c;
    if (seq_n == 0) c = c_home;
    else if (seq_hi < nchunks && (seq_lo < 0 || (seq_n & 1))) c = seq_hi++;
    else c = seq_lo--;
    ++seq_n;
    return c;
  };

  int ch_cur = seq_next();  // visit 0 (threshold only) and visit 1 both take the home chunk
  load_chunk(ch_cur, 0);
  for (int e = tid; e < TI * (kD / 4); e += NT) {
    const int r = e / (kD / 4), c4 = e - r * (kD / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + r < g.m) v = __ldg(reinterpret_cast<const float4*>(pq_u + (long long)(i0 + r) * kD + 4 * c4));
    *reinterpret_cast<float4*>(&sm.qs[r][4 * c4]) = v;
  }

  // per row of this warp: block coordinates, norm bound, the lane's two best lower bounds, threshold, survivors
  int iy[RI], ix[RI], cnt[RI], cnt_upd[RI];
  float nqv[RI], m1[RI], m2[RI], thr[RI];
#pragma unroll
  for (int a = 0; a < RI; ++a) {
    const int i = min(i0 + warp * RI + a, g.m - 1);
    iy[a] = i / g.nbw;
    ix[a] = i - iy[a] * g.nbw;
    nqv[a] = __ldg(nq + (long long)u * g.m + i);
    m1[a] = -kInf; m2[a] = -kInf; thr[a] = -kInf;
    cnt[a] = 0; cnt_upd[a] = 0;
  }
  const unsigned lower = (1u << lane) - 1u;

  // thr <- k-th largest of the warp's tracked lower bounds, for the rows in `rows` (bit a = row a), all of them in
  // lockstep so that the latencies of their warp-wide steps overlap.  A pop takes the largest out of its lane's pair.
  auto update_thresholds = [&](unsigned rows) {
    float t1[RI], t2[RI];
#pragma unroll
    for (int a = 0; a < RI; ++a) { t1[a] = m1[a]; t2[a] = m2[a]; }
    for (int r = 0; r + 1 < g.topk; ++r) {
#pragma unroll
      for (int a = 0; a < RI; ++a) {
        if (!((rows >> a) & 1u)) continue;  // warp-uniform
        const unsigned o = ordered_bits(t1[a]);
        const unsigned best = __reduce_max_sync(0xffffffffu, o);
        const unsigned who = __ballot_sync(0xffffffffu, o == best);
        if (lane == __ffs(who) - 1) { t1[a] = t2[a]; t2[a] = -kInf; }
      }
    }
#pragma unroll
    for (int a = 0; a < RI; ++a)
      if ((rows >> a) & 1u) thr[a] = from_ordered_bits(__reduce_max_sync(0xffffffffu, ordered_bits(t1[a])));
  };
  // drop the survivors of row a that the current threshold rules out (order kept)
  auto prune = [&](int a) {
    const int row = warp * RI + a, n = min(cnt[a], CAP);
    if (cnt[a] > CAP) return;  // overflowed: the row is rescored in full anyway
    int kept = 0;
    for (int e0 = 0; e0 < n; e0 += 32) {
      const int e = e0 + lane;
      const int j = e < n ? sm.surv[row][e] : 0;
      const float ub = e < n ? sm.surv_ub[row][e] : 0.f;
      const bool keep = e < n && !(ub < thr[a]);
      const unsigned km = __ballot_sync(0xffffffffu, keep);
      __syncwarp();
      if (keep) {
        const int at = kept + __popc(km & lower);
        sm.surv[row][at] = j;
        sm.surv_ub[row][at] = ub;
      }
      kept += __popc(km);
      __syncwarp();
    }
    cnt[a] = kept;
  };

  // visit 0 screens the home chunk for a threshold only; visits 1 .. nchunks screen every chunk, the home chunk first
  for (int v = 0; v <= nchunks; ++v) {
    const int ch = ch_cur, buf = v & 1;
    if (v < nchunks) {  // the next visit's chunk streams in while this one is screened
      ch_cur = v == 0 ? ch : seq_next();
      load_chunk(ch_cur, buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const int j0 = ch * JT;
    float acc[RI][KB];
#pragma unroll
    for (int a = 0; a < RI; ++a)
#pragma unroll
      for (int b = 0; b < KB; ++b) acc[a][b] = 0.f;
#pragma unroll 4
    for (int c4 = 0; c4 < kD / 4; ++c4) {
      float4 kv[KB];
#pragma unroll
      for (int b = 0; b < KB; ++b) kv[b] = *reinterpret_cast<const float4*>(&sm.scr.ks[buf][lane + 32 * b][4 * c4]);
#pragma unroll
      for (int a = 0; a < RI; ++a) {
        const float4 qv = *reinterpret_cast<const float4*>(&sm.qs[warp * RI + a][4 * c4]);
#pragma unroll
        for (int b = 0; b < KB; ++b) {
          acc[a][b] = fmaf(qv.x, kv[b].x, acc[a][b]);
          acc[a][b] = fmaf(qv.y, kv[b].y, acc[a][b]);
          acc[a][b] = fmaf(qv.z, kv[b].z, acc[a][b]);
          acc[a][b] = fmaf(qv.w, kv[b].w, acc[a][b]);
        }
      }
    }
    float nkc[KB];  // norm bound of the lane's keys times 2^-16
#pragma unroll
    for (int b = 0; b < KB; ++b) nkc[b] = sm.scr.nk[buf][lane + 32 * b] * 1.52587890625e-5f;
    unsigned stale = 0;  // rows whose threshold should be recomputed
    // One candidate: bounds of its exact score, filter against the row's threshold, tracking of the lower bounds.
    // A non-finite screening score gives the interval (-inf, +inf); a non-finite eps does so by itself (s + eps is
    // then +inf or NaN, which the filter keeps, and s - eps is -inf or NaN, which the tracking ignores).
    auto candidate = [&](int a, int b, bool cand) {
      const float sc = acc[a][b], eps = fmaf(nqv[a], nkc[b], 1e-37f);
      const bool fin = fabsf(sc) <= 1e38f;
      const float lb = fin ? sc - eps : -kInf, ub = fin ? sc + eps : kInf;
      if (v >= 1) {
        const bool keep = cand && !(ub < thr[a]);
        const unsigned km = __ballot_sync(0xffffffffu, keep);
        if (km) {  // warp-uniform
          if (keep) {
            const int at = cnt[a] + __popc(km & lower);
            if (at < CAP) { sm.surv[warp * RI + a][at] = j0 + lane + 32 * b; sm.surv_ub[warp * RI + a][at] = ub; }
          }
          cnt[a] += __popc(km);
        }
      }
      if (v != 1 && cand) {  // the home chunk's bounds were tracked in the threshold-only visit
        if (lb > m1[a]) { m2[a] = m1[a]; m1[a] = lb; }
        else m2[a] = fmaxf(m2[a], lb);
      }
    };
    // Plain chunk for this warp (the common case): wholly inside the grid, every row of the warp exists, and no key of
    // the chunk can be local to any of the warp's rows, so every (row, key) pair is a candidate.
    const int i_lo = i0 + warp * RI, i_hi = i_lo + RI - 1;
    bool plain = j0 + JT <= g.m && i_hi < g.m;
    if (plain) {
      const int jy_lo = j0 / g.nbw, jy_hi = (j0 + JT - 1) / g.nbw, iy_lo = i_lo / g.nbw, iy_hi = i_hi / g.nbw;
      plain = g.local_groups ? (jy_lo / g.rlat > iy_hi / g.rlat || jy_hi / g.rlat < iy_lo / g.rlat)
                             : (jy_lo > iy_hi + g.rlat || jy_hi < iy_lo - g.rlat);
    }
    if (plain) {
#pragma unroll
      for (int a = 0; a < RI; ++a)
#pragma unroll
        for (int b = 0; b < KB; ++b) candidate(a, b, true);
    } else {
      int jy[KB], jx[KB];
#pragma unroll
      for (int b = 0; b < KB; ++b) {
        const int j = min(j0 + lane + 32 * b, g.m - 1);
        jy[b] = j / g.nbw;
        jx[b] = j - jy[b] * g.nbw;
      }
#pragma unroll
      for (int a = 0; a < RI; ++a) {
        const bool row_ok = i_lo + a < g.m;  // warp-uniform
#pragma unroll
        for (int b = 0; b < KB; ++b) {
          int dx = jx[b] - ix[a];
          dx += dx < 0 ? g.nbw : 0;  // (jx - ix) mod nbw
          const bool local = g.local_groups ? (jy[b] / g.rlat == iy[a] / g.rlat && jx[b] / g.rlon == ix[a] / g.rlon)
                                            : (abs(jy[b] - iy[a]) <= g.rlat && (dx <= g.rlon || g.nbw - dx <= g.rlon));
          candidate(a, b, row_ok && j0 + lane + 32 * b < g.m && !local);
        }
      }
    }
#pragma unroll
    for (int a = 0; a < RI; ++a) {
      // recompute when the row has no threshold yet, gathered enough new survivors to suggest it is stale, fills
      // up, or is about to be scored
      const bool due = v <= 1 || v == nchunks || cnt[a] - cnt_upd[a] >= g.topk / 2 + 4 || cnt[a] > CAP / 2;
      if (i_lo + a < g.m && due && cnt[a] <= CAP) stale |= 1u << a;
    }
    if (stale) {  // warp-uniform
      __syncwarp();
      update_thresholds(stale);
#pragma unroll
      for (int a = 0; a < RI; ++a)
        if ((stale >> a) & 1u) {
          if (v >= 1) prune(a);
          cnt_upd[a] = cnt[a];
        }
    }
    __syncthreads();  // everyone is done with this buffer before the chunk after next lands in it
  }

  // ---- exact phase (the staging buffers are free now and hold the survivors' score keys)
  // rows whose survivors fit the counting rank: flatten (row, entry) pairs over the lanes, two chains in flight
  int base_of[RI + 1];
  base_of[0] = 0;
  unsigned slow = 0;  // rows that take the insertion path (their survivors overflowed)
#pragma unroll
  for (int a = 0; a < RI; ++a) {
    const bool row_ok = i0 + warp * RI + a < g.m;
    const bool fast = row_ok && cnt[a] <= CAP;
    if (row_ok && !fast) slow |= 1u << a;
    base_of[a + 1] = base_of[a] + (fast ? cnt[a] : 0);
  }
  __syncwarp();
  const int total = base_of[RI];
  for (int p0 = 0; p0 < total; p0 += 64) {
    int pa[2], pe[2], pj[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int p = p0 + 32 * t + lane;
      pa[t] = -1; pe[t] = 0; pj[t] = 0;
      if (p < total) {
#pragma unroll
        for (int a = 0; a < RI; ++a)
          if (p >= base_of[a] && p < base_of[a + 1]) { pa[t] = a; pe[t] = p - base_of[a]; }
        pj[t] = sm.surv[warp * RI + pa[t]][pe[t]];
      }
    }
    // both chains in one instruction stream (inlined twice; the loads of the second overlap the first's arithmetic)
    unsigned long long k0 = 0ull, k1 = 0ull;
    if (pa[0] >= 0) k0 = exact_key(sm.qs[warp * RI + pa[0]], pk_u, pj[0]);
    if (pa[1] >= 0) k1 = exact_key(sm.qs[warp * RI + pa[1]], pk_u, pj[1]);
    if (pa[0] >= 0) sm.ekey[warp * RI + pa[0]][pe[0]] = k0;
    if (pa[1] >= 0) sm.ekey[warp * RI + pa[1]][pe[1]] = k1;
  }
  __syncwarp();
#pragma unroll
  for (int a = 0; a < RI; ++a) {
    const int row = warp * RI + a, i = i0 + row;
    if (i >= g.m) break;  // warp-uniform
    int32_t* out = block_idx + ((long long)u * g.m + i) * g.topk;
    if (!((slow >> a) & 1u)) {
      const int n = cnt[a];
      for (int e = lane; e < n; e += 32) {  // rank by counting the survivors that come first
        const unsigned long long key = sm.ekey[row][e];
        const int id = sm.surv[row][e];
        int rank = 0;
        for (int f = 0; f < n; ++f) rank += ranks_before(sm.ekey[row][f], sm.surv[row][f], key, id) ? 1 : 0;
        if (rank < g.topk) out[rank] = id;
      }
      if (lane >= n && lane < g.topk) out[lane] = -1;
    } else {
      unsigned long long lkey = 0ull;
      int lid = -1;
      // too many survivors to hold: score every key of the unit
      for (int jb = 0; jb < g.m; jb += 32) {
        const int j = jb + lane;
        bool cand = j < g.m;
        if (cand) {
          const int jy = j / g.nbw, jx = j - jy * g.nbw;
          int dx = jx - ix[a];
          dx += dx < 0 ? g.nbw : 0;
          cand = g.local_groups ? !(jy / g.rlat == iy[a] / g.rlat && jx / g.rlon == ix[a] / g.rlon)
                                : !(abs(jy - iy[a]) <= g.rlat && (dx <= g.rlon || g.nbw - dx <= g.rlon));
        }
        insert_batch(cand ? exact_key(sm.qs[row], pk_u, j) : 0ull, j, lkey, lid, g.topk, lane);
      }
      if (lane < g.topk) out[lane] = lkey != 0ull ? lid : -1;
    }
  }
}

template <int NW, int RI, int CAP, int JT, int MB>
int launch_topk(const HostCtx& c, const float* pooled_q, const float* pooled_k, const float* norm_q,
                const float* norm_k, int32_t* block_idx) {
  const Geo& g = c.g;
  const size_t smem = sizeof(TopkSmem<NW, RI, CAP, JT>);
  static unsigned long long configured = 0;  // devices on which the kernel's shared-memory opt-in is set
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 0 || dev >= 64) return MOSAIC_E_UNSUPPORTED;
  if (!((configured >> dev) & 1ull)) {
    if (cudaFuncSetAttribute(topk_kernel<NW, RI, CAP, JT, MB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return MOSAIC_E_CUDA;
    configured |= 1ull << dev;
  }
  const int tiles = (g.m + NW * RI - 1) / (NW * RI);
  topk_kernel<NW, RI, CAP, JT, MB><<<(unsigned)(g.U * tiles), NW * 32, smem, c.stream>>>(g, pooled_q, pooled_k, norm_q,
                                                                                norm_k, block_idx);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

// block sums (and norm bounds) of one tensor of `units` units
int launch_pool_one(const HostCtx& c, const void* x, float* pooled, float* norm, int units) {
  const Geo& g = c.g;
  const long long threads = 1ll * units * g.m * 8;
  const unsigned blocks = (unsigned)((threads + 255) / 256);
  if (g.bw == 8)
    pool_kernel<8><<<blocks, 256, 0, c.stream>>>(g, (const uint4*)x, (const uint4*)x, pooled, pooled, norm, norm, 1, units);
  else
    pool_kernel<16><<<blocks, 256, 0, c.stream>>>(g, (const uint4*)x, (const uint4*)x, pooled, pooled, norm, norm, 1, units);
  return cudaGetLastError() == cudaSuccess ? MOSAIC_OK : MOSAIC_E_CUDA;
}

int launch_select(const HostCtx& c, const void* q, const void* k, int32_t* block_idx, float* pooled_q,
                  float* pooled_k, float* norm_q, float* norm_k) {
  const Geo& g = c.g;
  if (g.Ukv != g.U) {  // grouped-query attention: Q and K have different head counts, one launch each
    int rc = launch_pool_one(c, q, pooled_q, norm_q, g.U);
    if (!rc) rc = launch_pool_one(c, k, pooled_k, norm_k, g.Ukv);
    if (rc) return rc;
  } else {
    const long long threads = 2ll * g.U * g.m * 8;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    if (g.bw == 8)
      pool_kernel<8><<<blocks, 256, 0, c.stream>>>(g, (const uint4*)q, (const uint4*)k, pooled_q, pooled_k, norm_q,
                                                   norm_k, 2, g.U);
    else
      pool_kernel<16><<<blocks, 256, 0, c.stream>>>(g, (const uint4*)q, (const uint4*)k, pooled_q, pooled_k, norm_q,
                                                    norm_k, 2, g.U);
    if (cudaGetLastError() != cudaSuccess) return MOSAIC_E_CUDA;
  }
  if (g.topk > 0) {
    // the most query blocks per CTA (64, 32, 16) that still gives every SM about two CTAs; small problems are
    // latency-bound and take 8 rows per CTA and 64-key chunks, so that more warps are resident.  The survivors of a
    // row grow with top-k (the threshold is the k-th best of 64 tracked bounds), and a row whose survivors overflow
    // scores every key exactly: beyond top-k 16 only the configurations with room for 192 survivors are used.
    auto ctas = [&](int ti) { return (long long)g.U * ((g.m + ti - 1) / ti); };
    int rc;
    if (g.topk > 16)
      rc = ctas(16) >= 296 ? launch_topk<4, 4, 192, 128, 2>(c, pooled_q, pooled_k, norm_q, norm_k, block_idx)
                           : launch_topk<4, 2, 192, 64, 4>(c, pooled_q, pooled_k, norm_q, norm_k, block_idx);
    else
      rc = ctas(64) >= 296   ? launch_topk<8, 4, 96, 64, 3>(c, pooled_q, pooled_k, norm_q, norm_k, block_idx)
           : ctas(32) >= 296 ? launch_topk<4, 8, 128, 128, 1>(c, pooled_q, pooled_k, norm_q, norm_k, block_idx)
           : ctas(16) >= 296 ? launch_topk<4, 4, 192, 128, 2>(c, pooled_q, pooled_k, norm_q, norm_k, block_idx)
                             : launch_topk<4, 2, 192, 64, 4>(c, pooled_q, pooled_k, norm_q, norm_k, block_idx);
    if (rc) return rc;
  }
  return MOSAIC_OK;
}

}  // namespace mosaic
