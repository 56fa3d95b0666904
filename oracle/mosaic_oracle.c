/*
 * mosaic_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the MOSAIC block-sparse attention
 * path computes, written from the paper's equations.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it; the CUDA library never
 * does, and the two share no code.
 *
 * Conventions (one "unit" = one (batch, head) pair; units are independent because
 * every equation of the method is per head and per sample):
 *   grid nlat x nlon, token t = lat*nlon + lon, head dim d;
 *   block (by,bx) holds tokens (by*bh + r, bx*bw + c), r < bh, c < bw; id j = by*nbw + bx;
 *   inputs are bf16 bit patterns (uint16), or IEEE binary16 when the geometry says so, widened exactly to double.
 *
 * Steps and where the paper defines them:
 *   pooling      -- "Compression" paragraph of the Block-Sparse Attention section
 *                   (block representations via phi = mean pooling); the mean's 1/b is
 *                   dropped because a positive constant cannot change a ranking.
 *   block score  -- block-level attention equation of the same paragraph; the exp and
 *                   the normalisation are strictly increasing per row, so the raw dot
 *                   product of pooled vectors ranks identically.
 *   top-n        -- "Selection" paragraph: the n best key blocks per query block,
 *                   shared by every token of that block.  Here the candidates are the
 *                   non-local blocks and ties go to the lower block id.
 *   attention    -- the fine-grained attention equation of the "Selection" paragraph,
 *                   taken over the union of the local neighbourhood and the selected
 *                   blocks with ONE softmax (scale 1/sqrt(d_k) unless overridden).
 *   backward     -- analytic gradient of that softmax attention with the selection
 *                   held constant; dK/dV visit only the query blocks connected to a
 *                   key/value block ("Kernel Design" paragraph of the appendix).
 *
 *   three-branch -- mo_fwd3_unit / mo_bwd3_unit at the end of this file: the paper's own gated sum of the
 *                   compression, selection and local branches (Eq. of the aggregated output), each
 *                   branch with its own softmax, gradient into the routing scores through the
 *                   compression branch.
 *
 * Pins (tests/test_oracle_*.py): dense attention when top-k covers every block,
 * brute-force selection on tiny grids, hand-built winners and ties, row-stochastic
 * weights, convex-hull bound, finite differences, longitude-roll equivariance,
 * zero gradient for unconnected blocks, the cost-model pair count; NaN ordering; for the three-branch
 * form each branch against a textbook routine, its link to the union form, finite differences.
 * Parity unpinned: agreement with the authors' own kernels (not available).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct mo_geom {
  int32_t nlat, nlon, d;
  int32_t bh, bw;
  int32_t rlat, rlon;
  int32_t topk;
  double scale; /* softmax scale; <= 0 means 1/sqrt(d) */
  int32_t local_groups; /* 0: local set = sliding neighbourhood of radius (rlat, rlon);
                           1: local set = the aligned group of rlat x rlon blocks that holds the block
                              (the paper's "Local Attention": dense attention inside large blocks) */
  int32_t f16;          /* 0: the 16-bit inputs are bf16 bit patterns; 1: IEEE binary16 (the paper trains in fp16,
                           appendix, "Distributed training" paragraph) */
} mo_geom;

#define MO_MAX_LOCAL 256

static int g_ok(const mo_geom *g) {
  if (!g || g->nlat <= 0 || g->nlon <= 0 || g->d <= 0 || g->bh <= 0 || g->bw <= 0) return 0;
  if (g->nlat % g->bh || g->nlon % g->bw) return 0;
  if (g->rlat < 0 || g->rlon < 0 || g->topk < 0) return 0;
  if (g->local_groups) {
    if (g->rlat < 1 || g->rlon < 1 || g->rlat * g->rlon > MO_MAX_LOCAL) return 0;
  } else if ((2 * g->rlat + 1) * (2 * g->rlon + 1) > MO_MAX_LOCAL) return 0;
  return 1;
}
static int g_nbh(const mo_geom *g) { return g->nlat / g->bh; }
static int g_nbw(const mo_geom *g) { return g->nlon / g->bw; }
static int g_m(const mo_geom *g) { return g_nbh(g) * g_nbw(g); }
static int g_b(const mo_geom *g) { return g->bh * g->bw; }
static double g_scale(const mo_geom *g) { return g->scale > 0.0 ? g->scale : 1.0 / sqrt((double)g->d); }

static double bf16_widen(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}
/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits; exact in double */
static double f16_widen(uint16_t h) {
  int sign = h >> 15, ex = (h >> 10) & 31, fr = h & 1023;
  double v;
  if (ex == 0) v = ldexp((double)fr, -24);                 /* zero and subnormals */
  else if (ex == 31) v = fr ? NAN : INFINITY;
  else v = ldexp((double)(1024 + fr), ex - 25);
  return sign ? -v : v;
}
/* a 16-bit input element in the problem's storage type */
static double w16(const mo_geom *g, uint16_t h) { return g->f16 ? f16_widen(h) : bf16_widen(h); }

/* token index of element e (row-major inside the block) of block j */
static int64_t block_token(const mo_geom *g, int j, int e) {
  int nbw = g_nbw(g);
  int by = j / nbw, bx = j % nbw;
  int r = e / g->bw, c = e % g->bw;
  return (int64_t)(by * g->bh + r) * g->nlon + (bx * g->bw + c);
}

int mo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Local set of query block i: rows clamp(by+dy), columns (bx+dx) mod nbw, as a SET
 * (each block once), listed in first-occurrence order over dy, then dx ascending.
 * With local_groups: the aligned group of rlat x rlon blocks that holds block i.
 */
int mo_local_set(const mo_geom *g, int32_t i, int32_t *out) {
  if (!g_ok(g)) return -1;
  int nbh = g_nbh(g), nbw = g_nbw(g);
  int by = i / nbw, bx = i % nbw, n = 0;
  if (g->local_groups) { /* the blocks of the aligned rlat x rlon group, row-major, those inside the grid */
    int y0 = (by / g->rlat) * g->rlat, x0 = (bx / g->rlon) * g->rlon;
    for (int y = y0; y < y0 + g->rlat && y < nbh; ++y)
      for (int x = x0; x < x0 + g->rlon && x < nbw; ++x) out[n++] = y * nbw + x;
    return n;
  }
  for (int dy = -g->rlat; dy <= g->rlat; ++dy) {
    int y = by + dy;
    if (y < 0) y = 0;
    if (y > nbh - 1) y = nbh - 1;
    for (int dx = -g->rlon; dx <= g->rlon; ++dx) {
      int x = ((bx + dx) % nbw + nbw) % nbw;
      int id = y * nbw + x, seen = 0;
      for (int a = 0; a < n; ++a) seen |= (out[a] == id);
      if (!seen) out[n++] = id;
    }
  }
  return n;
}

/* Block sums of one [N,d] bf16 tensor: sequential fp64 accumulation in row-major
 * block order, rounded once to fp32. */
int mo_pool_unit(const mo_geom *g, const uint16_t *x, float *pooled /* [m,d] */) {
  if (!g_ok(g)) return -1;
  int m = g_m(g), b = g_b(g), d = g->d;
#pragma omp parallel for schedule(static)
  for (int j = 0; j < m; ++j) {
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (int e = 0; e < b; ++e) acc += w16(g, x[block_token(g, j, e) * d + c]);
      pooled[(size_t)j * d + c] = (float)acc;
    }
  }
  return 0;
}

typedef struct { double s; int32_t j; } mo_cand;

/* rank order: higher score first; a NaN ranks below every number; equal scores
 * (+0 and -0 compare equal) go to the lower block id. */
static int cand_cmp(const void *pa, const void *pb) {
  const mo_cand *a = (const mo_cand *)pa, *b = (const mo_cand *)pb;
  int an = isnan(a->s), bn = isnan(b->s);
  if (an != bn) return an ? 1 : -1;
  if (!an) {
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
  }
  return (a->j > b->j) - (a->j < b->j);
}

/*
 * Selection for one unit.  idx is [m, topk]; row i lists the chosen non-local block
 * ids best first, padded with -1.  pq/pk (optional, [m,d] fp32) receive the pooled sums.
 */
int mo_select_unit(const mo_geom *g, const uint16_t *q, const uint16_t *k, int32_t *idx,
                   float *pq_out, float *pk_out) {
  if (!g_ok(g)) return -1;
  int m = g_m(g), d = g->d, topk = g->topk;
  float *pq = (float *)malloc(sizeof(float) * (size_t)m * d);
  float *pk = (float *)malloc(sizeof(float) * (size_t)m * d);
  if (!pq || !pk) { free(pq); free(pk); return -2; }
  mo_pool_unit(g, q, pq);
  mo_pool_unit(g, k, pk);
#pragma omp parallel
  {
    mo_cand *cand = (mo_cand *)malloc(sizeof(mo_cand) * (size_t)m);
    int32_t loc[MO_MAX_LOCAL];
#pragma omp for schedule(dynamic, 4)
    for (int i = 0; i < m; ++i) {
      int nl = mo_local_set(g, i, loc), nc = 0;
      for (int j = 0; j < m; ++j) {
        int is_local = 0;
        for (int a = 0; a < nl; ++a) is_local |= (loc[a] == j);
        if (is_local) continue;
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += (double)pq[(size_t)i * d + c] * (double)pk[(size_t)j * d + c];
        cand[nc].s = s;
        cand[nc].j = j;
        ++nc;
      }
      qsort(cand, (size_t)nc, sizeof(mo_cand), cand_cmp);
      for (int r = 0; r < topk; ++r) idx[(size_t)i * topk + r] = r < nc ? cand[r].j : -1;
    }
    free(cand);
  }
  if (pq_out) memcpy(pq_out, pq, sizeof(float) * (size_t)m * d);
  if (pk_out) memcpy(pk_out, pk, sizeof(float) * (size_t)m * d);
  free(pq);
  free(pk);
  return 0;
}

/* attended block list of query block i: local set, then the selected ids >= 0 */
static int attended(const mo_geom *g, const int32_t *idx, int i, int32_t *out) {
  int n = mo_local_set(g, i, out);
  for (int r = 0; r < g->topk; ++r) {
    int32_t j = idx[(size_t)i * g->topk + r];
    if (j >= 0) out[n++] = j;
  }
  return n;
}

/* logits x_t = scale * q_l . k_t over the attended tokens of one query row */
static void row_logits(const mo_geom *g, const uint16_t *q, const uint16_t *k, int64_t l,
                       const int32_t *att, int na, double *x) {
  int b = g_b(g), d = g->d;
  double sc = g_scale(g);
  for (int a = 0; a < na; ++a)
    for (int e = 0; e < b; ++e) {
      int64_t t = block_token(g, att[a], e);
      double s = 0.0;
      for (int c = 0; c < d; ++c) s += w16(g, q[l * d + c]) * w16(g, k[t * d + c]);
      x[(size_t)a * b + e] = sc * s;
    }
}

/*
 * Softmax weights of one query row (row e_row of block i) over its attended tokens.
 * tokens/w must hold (|L_i|+topk)*b entries; returns the count.
 */
int mo_weights_row(const mo_geom *g, const uint16_t *q, const uint16_t *k, const int32_t *idx,
                   int32_t i, int32_t e_row, int64_t *tokens, double *w) {
  if (!g_ok(g)) return -1;
  int b = g_b(g);
  int32_t *att = (int32_t *)malloc(sizeof(int32_t) * (MO_MAX_LOCAL + (size_t)g->topk));
  int na = attended(g, idx, i, att), n = na * b;
  row_logits(g, q, k, block_token(g, i, e_row), att, na, w);
  double M = -INFINITY, Z = 0.0;
  for (int t = 0; t < n; ++t) M = w[t] > M ? w[t] : M;
  for (int t = 0; t < n; ++t) Z += exp(w[t] - M);
  for (int t = 0; t < n; ++t) w[t] = exp(w[t] - M) / Z;
  for (int a = 0; a < na; ++a)
    for (int e = 0; e < b; ++e) tokens[(size_t)a * b + e] = block_token(g, att[a], e);
  free(att);
  return n;
}

/*
 * Forward for a list of query blocks of one unit (blocks == NULL: all m, in order).
 * O is [n_blocks, b, d], LSE is [n_blocks, b], rows in row-major order inside the block.
 */
int mo_fwd_unit(const mo_geom *g, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                const int32_t *idx, int32_t n_blocks, const int32_t *blocks, double *O, double *LSE) {
  if (!g_ok(g)) return -1;
  int b = g_b(g), d = g->d;
  int max_att = MO_MAX_LOCAL + g->topk;
#pragma omp parallel
  {
    int32_t *att = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
    double *x = (double *)malloc(sizeof(double) * (size_t)max_att * b);
#pragma omp for schedule(dynamic, 1)
    for (int n = 0; n < n_blocks; ++n) {
      int i = blocks ? blocks[n] : n;
      int na = attended(g, idx, i, att), nt = na * b;
      for (int e = 0; e < b; ++e) {
        int64_t l = block_token(g, i, e);
        row_logits(g, q, k, l, att, na, x);
        double M = -INFINITY, Z = 0.0;
        for (int t = 0; t < nt; ++t) M = x[t] > M ? x[t] : M;
        for (int t = 0; t < nt; ++t) Z += exp(x[t] - M);
        double *o = O + ((size_t)n * b + e) * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int a = 0; a < na; ++a)
          for (int e2 = 0; e2 < b; ++e2) {
            double w = exp(x[(size_t)a * b + e2] - M) / Z;
            int64_t t = block_token(g, att[a], e2);
            for (int c = 0; c < d; ++c) o[c] += w * w16(g, v[t * d + c]);
          }
        LSE[(size_t)n * b + e] = M + log(Z);
      }
    }
    free(att);
    free(x);
  }
  return 0;
}

/*
 * Backward for one whole unit, selection held constant.  dQ, dK, dV are [N,d] in
 * token order.  O_out [N,d] and LSE_out [N] (optional) receive the forward results.
 */
int mo_bwd_unit(const mo_geom *g, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                const uint16_t *d_o, const int32_t *idx, double *dQ, double *dK, double *dV,
                double *O_out, double *LSE_out) {
  if (!g_ok(g)) return -1;
  int m = g_m(g), b = g_b(g), d = g->d;
  int64_t N = (int64_t)g->nlat * g->nlon;
  int max_att = MO_MAX_LOCAL + g->topk;
  double sc = g_scale(g);
  double *Ob = (double *)malloc(sizeof(double) * (size_t)m * b * d);
  double *Lb = (double *)malloc(sizeof(double) * (size_t)m * b);
  double *LSE = (double *)malloc(sizeof(double) * (size_t)N);
  double *D = (double *)malloc(sizeof(double) * (size_t)N);
  if (!Ob || !Lb || !LSE || !D) { free(Ob); free(Lb); free(LSE); free(D); return -2; }
  mo_fwd_unit(g, q, k, v, idx, m, NULL, Ob, Lb);
  /* D_l = dO_l . O_l */
#pragma omp parallel for schedule(static)
  for (int i = 0; i < m; ++i)
    for (int e = 0; e < b; ++e) {
      int64_t l = block_token(g, i, e);
      double acc = 0.0;
      for (int c = 0; c < d; ++c) {
        double o = Ob[((size_t)i * b + e) * d + c];
        acc += w16(g, d_o[l * d + c]) * o;
        if (O_out) O_out[l * d + c] = o;
      }
      D[l] = acc;
      LSE[l] = Lb[(size_t)i * b + e];
      if (LSE_out) LSE_out[l] = LSE[l];
    }
  /* dQ: every query row over its attended tokens */
#pragma omp parallel
  {
    int32_t *att = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
    double *x = (double *)malloc(sizeof(double) * (size_t)max_att * b);
#pragma omp for schedule(dynamic, 1)
    for (int i = 0; i < m; ++i) {
      int na = attended(g, idx, i, att);
      for (int e = 0; e < b; ++e) {
        int64_t l = block_token(g, i, e);
        row_logits(g, q, k, l, att, na, x);
        double *dq = dQ + l * d;
        for (int c = 0; c < d; ++c) dq[c] = 0.0;
        for (int a = 0; a < na; ++a)
          for (int e2 = 0; e2 < b; ++e2) {
            int64_t t = block_token(g, att[a], e2);
            double w = exp(x[(size_t)a * b + e2] - LSE[l]);
            double dP = 0.0;
            for (int c = 0; c < d; ++c) dP += w16(g, d_o[l * d + c]) * w16(g, v[t * d + c]);
            double dS = w * (dP - D[l]);
            for (int c = 0; c < d; ++c) dq[c] += sc * dS * w16(g, k[t * d + c]);
          }
      }
    }
    free(att);
    free(x);
  }
  /* dK, dV: every key/value block over the query blocks connected to it */
#pragma omp parallel
  {
    int32_t *att = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
#pragma omp for schedule(dynamic, 1)
    for (int j = 0; j < m; ++j) {
      for (int e2 = 0; e2 < b; ++e2) {
        int64_t t = block_token(g, j, e2);
        for (int c = 0; c < d; ++c) { dK[t * d + c] = 0.0; dV[t * d + c] = 0.0; }
      }
      for (int i = 0; i < m; ++i) {
        int na = attended(g, idx, i, att), connected = 0;
        for (int a = 0; a < na; ++a) connected |= (att[a] == j);
        if (!connected) continue;
        for (int e = 0; e < b; ++e) {
          int64_t l = block_token(g, i, e);
          for (int e2 = 0; e2 < b; ++e2) {
            int64_t t = block_token(g, j, e2);
            double s = 0.0, dP = 0.0;
            for (int c = 0; c < d; ++c) {
              s += w16(g, q[l * d + c]) * w16(g, k[t * d + c]);
              dP += w16(g, d_o[l * d + c]) * w16(g, v[t * d + c]);
            }
            double w = exp(sc * s - LSE[l]);
            double dS = w * (dP - D[l]);
            for (int c = 0; c < d; ++c) {
              dV[t * d + c] += w * w16(g, d_o[l * d + c]);
              dK[t * d + c] += sc * dS * w16(g, q[l * d + c]);
            }
          }
        }
      }
    }
    free(att);
  }
  free(Ob); free(Lb); free(LSE); free(D);
  return 0;
}

/*
 * Backward restricted to lists of blocks of one unit (same arithmetic as mo_bwd_unit, for sizes at
 * which the whole unit takes too long): dQ for the query blocks in qblocks, dK and dV for the
 * key/value blocks in kblocks.  dQ is [nq, b, d], dK and dV are [nk, b, d], rows in row-major order
 * inside each block.  The forward quantities a gradient needs (LSE_l and D_l = dO_l . O_l) are
 * computed for exactly the query blocks involved: the listed ones and every query block connected
 * to a listed key/value block.
 */
int mo_bwd_blocks(const mo_geom *g, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                  const uint16_t *d_o, const int32_t *idx, int32_t nq, const int32_t *qblocks, double *dQ,
                  int32_t nk, const int32_t *kblocks, double *dK, double *dV) {
  if (!g_ok(g)) return -1;
  int m = g_m(g), b = g_b(g), d = g->d;
  int64_t N = (int64_t)g->nlat * g->nlon;
  int max_att = MO_MAX_LOCAL + g->topk;
  double sc = g_scale(g);
  for (int n = 0; n < nq; ++n) if (qblocks[n] < 0 || qblocks[n] >= m) return -1;
  for (int n = 0; n < nk; ++n) if (kblocks[n] < 0 || kblocks[n] >= m) return -1;
  /* which query blocks are involved */
  unsigned char *need = (unsigned char *)calloc((size_t)m, 1);
  int32_t *att0 = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
  if (!need || !att0) { free(need); free(att0); return -2; }
  for (int n = 0; n < nq; ++n) need[qblocks[n]] = 1;
  for (int i = 0; i < m; ++i) {
    int na = attended(g, idx, i, att0);
    for (int a = 0; a < na; ++a)
      for (int n = 0; n < nk; ++n) if (att0[a] == kblocks[n]) need[i] = 1;
  }
  free(att0);
  int nn = 0;
  for (int i = 0; i < m; ++i) nn += need[i];
  int32_t *list = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nn > 0 ? nn : 1));
  double *Ob = (double *)malloc(sizeof(double) * (size_t)(nn > 0 ? nn : 1) * b * d);
  double *Lb = (double *)malloc(sizeof(double) * (size_t)(nn > 0 ? nn : 1) * b);
  double *LSE = (double *)malloc(sizeof(double) * (size_t)N);
  double *D = (double *)malloc(sizeof(double) * (size_t)N);
  if (!list || !Ob || !Lb || !LSE || !D) { free(need); free(list); free(Ob); free(Lb); free(LSE); free(D); return -2; }
  nn = 0;
  for (int i = 0; i < m; ++i) if (need[i]) list[nn++] = i;
  mo_fwd_unit(g, q, k, v, idx, nn, list, Ob, Lb);
  /* D_l = dO_l . O_l and LSE_l of the involved rows */
#pragma omp parallel for schedule(static)
  for (int n = 0; n < nn; ++n)
    for (int e = 0; e < b; ++e) {
      int64_t l = block_token(g, list[n], e);
      double acc = 0.0;
      for (int c = 0; c < d; ++c) acc += w16(g, d_o[l * d + c]) * Ob[((size_t)n * b + e) * d + c];
      D[l] = acc;
      LSE[l] = Lb[(size_t)n * b + e];
    }
  /* dQ of the listed query blocks: every row over its attended tokens */
#pragma omp parallel
  {
    int32_t *att = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
    double *x = (double *)malloc(sizeof(double) * (size_t)max_att * b);
#pragma omp for schedule(dynamic, 1)
    for (int n = 0; n < nq; ++n) {
      int i = qblocks[n];
      int na = attended(g, idx, i, att);
      for (int e = 0; e < b; ++e) {
        int64_t l = block_token(g, i, e);
        row_logits(g, q, k, l, att, na, x);
        double *dq = dQ + ((size_t)n * b + e) * d;
        for (int c = 0; c < d; ++c) dq[c] = 0.0;
        for (int a = 0; a < na; ++a)
          for (int e2 = 0; e2 < b; ++e2) {
            int64_t t = block_token(g, att[a], e2);
            double w = exp(x[(size_t)a * b + e2] - LSE[l]);
            double dP = 0.0;
            for (int c = 0; c < d; ++c) dP += w16(g, d_o[l * d + c]) * w16(g, v[t * d + c]);
            double dS = w * (dP - D[l]);
            for (int c = 0; c < d; ++c) dq[c] += sc * dS * w16(g, k[t * d + c]);
          }
      }
    }
    free(att);
    free(x);
  }
  /* dK, dV of the listed key/value blocks: every row over the query blocks connected to its block,
   * query blocks in ascending order (rows of a key block are independent: parallel over them) */
  for (int n = 0; n < nk; ++n) {
    int j = kblocks[n];
    int32_t *conn = (int32_t *)malloc(sizeof(int32_t) * (size_t)m);
    int32_t *att = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
    int nc = 0;
    for (int i = 0; i < m; ++i) {
      int na = attended(g, idx, i, att), connected = 0;
      for (int a = 0; a < na; ++a) connected |= (att[a] == j);
      if (connected) conn[nc++] = i;
    }
    free(att);
#pragma omp parallel for schedule(dynamic, 1)
    for (int e2 = 0; e2 < b; ++e2) {
      int64_t t = block_token(g, j, e2);
      double *dk = dK + ((size_t)n * b + e2) * d, *dv = dV + ((size_t)n * b + e2) * d;
      for (int c = 0; c < d; ++c) { dk[c] = 0.0; dv[c] = 0.0; }
      for (int ci = 0; ci < nc; ++ci)
        for (int e = 0; e < b; ++e) {
          int64_t l = block_token(g, conn[ci], e);
          double s = 0.0, dP = 0.0;
          for (int c = 0; c < d; ++c) {
            s += w16(g, q[l * d + c]) * w16(g, k[t * d + c]);
            dP += w16(g, d_o[l * d + c]) * w16(g, v[t * d + c]);
          }
          double w = exp(sc * s - LSE[l]);
          double dS = w * (dP - D[l]);
          for (int c = 0; c < d; ++c) {
            dv[c] += w * w16(g, d_o[l * d + c]);
            dk[c] += sc * dS * w16(g, q[l * d + c]);
          }
        }
    }
    free(conn);
  }
  free(need); free(list); free(Ob); free(Lb); free(LSE); free(D);
  return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Three-branch output (the paper's own form of the operator: Eq. of the aggregated output in the
 * section "Native Sparse Attention", and the "Compression", "Selection" and "Local Attention"
 * paragraphs of the section "Block-Sparse Attention").  For token l of query block i:
 *   compression  oCG_l = sum_{j=1..m} abar_ij vbar_j,  abar_i,: = softmax_j(qbar_i . kbar_j * scale) over ALL
 *                m blocks, qbar, kbar, vbar the block MEANS (fp32-rounded block sum / b); the same vector for
 *                every token of the block;
 *   selection    oFG_l = softmax attention of q_l over the tokens of the selected blocks (own normaliser);
 *                an empty selection gives oFG_l = 0 and LSE = -inf;
 *   local        oL_l  = softmax attention of q_l over the tokens of the local neighbourhood (own normaliser);
 *   output       o_l   = gates[l][0] * oCG_l + gates[l][1] * oFG_l + gates[l][2] * oL_l.
 * The gates are functions of the layer input in the paper and therefore inputs here.
 * ------------------------------------------------------------------------------------------------ */

/* softmax attention of one query row over the tokens of a list of blocks; returns LSE (-inf if none) */
static double branch_row(const mo_geom *g, const uint16_t *q, const uint16_t *k, const uint16_t *v, int64_t l,
                         const int32_t *blk, int nb, double *x, double *o) {
  int b = g_b(g), d = g->d, nt = nb * b;
  for (int c = 0; c < d; ++c) o[c] = 0.0;
  if (nb == 0) return -INFINITY;
  row_logits(g, q, k, l, blk, nb, x);
  double M = -INFINITY, Z = 0.0;
  for (int t = 0; t < nt; ++t) M = x[t] > M ? x[t] : M;
  for (int t = 0; t < nt; ++t) Z += exp(x[t] - M);
  for (int a = 0; a < nb; ++a)
    for (int e2 = 0; e2 < b; ++e2) {
      double w = exp(x[(size_t)a * b + e2] - M) / Z;
      int64_t t = block_token(g, blk[a], e2);
      for (int c = 0; c < d; ++c) o[c] += w * w16(g, v[t * d + c]);
    }
  return M + log(Z);
}

/* block means of one tensor: fp32-rounded block sum (as in the selection) divided by b, in double */
static void block_means(const mo_geom *g, const uint16_t *x, double *mean /* [m,d] */) {
  int m = g_m(g), d = g->d;
  float *p = (float *)malloc(sizeof(float) * (size_t)m * d);
  mo_pool_unit(g, x, p);
  for (size_t z = 0; z < (size_t)m * d; ++z) mean[z] = (double)p[z] / (double)g_b(g);
  free(p);
}

/*
 * Forward of the three-branch form for one unit.  gates is [N,3] (CG, FG, L) in token order.
 * Outputs in token order: O [N,d]; optional OCG, OFG, OL [N,d] (branch outputs before gating),
 * LSE_FG, LSE_L [N], ABAR [m,m] (block-level attention).
 */
int mo_fwd3_unit(const mo_geom *g, const uint16_t *q, const uint16_t *k, const uint16_t *v, const int32_t *idx,
                 const double *gates, double *O, double *OCG, double *OFG, double *OL, double *LSE_FG,
                 double *LSE_L, double *ABAR) {
  if (!g_ok(g)) return -1;
  int m = g_m(g), b = g_b(g), d = g->d;
  double sc = g_scale(g);
  double *qm = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *km = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *vm = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *ocg = (double *)malloc(sizeof(double) * (size_t)m * d);
  if (!qm || !km || !vm || !ocg) { free(qm); free(km); free(vm); free(ocg); return -2; }
  block_means(g, q, qm);
  block_means(g, k, km);
  block_means(g, v, vm);
  /* compression branch: block-to-block softmax attention on the means */
#pragma omp parallel
  {
    double *s = (double *)malloc(sizeof(double) * (size_t)m);
#pragma omp for schedule(static)
    for (int i = 0; i < m; ++i) {
      double M = -INFINITY, Z = 0.0;
      for (int j = 0; j < m; ++j) {
        double a = 0.0;
        for (int c = 0; c < d; ++c) a += qm[(size_t)i * d + c] * km[(size_t)j * d + c];
        s[j] = sc * a;
        M = s[j] > M ? s[j] : M;
      }
      for (int j = 0; j < m; ++j) Z += exp(s[j] - M);
      for (int c = 0; c < d; ++c) ocg[(size_t)i * d + c] = 0.0;
      for (int j = 0; j < m; ++j) {
        double a = exp(s[j] - M) / Z;
        if (ABAR) ABAR[(size_t)i * m + j] = a;
        for (int c = 0; c < d; ++c) ocg[(size_t)i * d + c] += a * vm[(size_t)j * d + c];
      }
    }
    free(s);
  }
  /* selection and local branches, then the gated sum */
  int max_att = MO_MAX_LOCAL + g->topk;
#pragma omp parallel
  {
    int32_t *loc = (int32_t *)malloc(sizeof(int32_t) * MO_MAX_LOCAL);
    int32_t *sel = (int32_t *)malloc(sizeof(int32_t) * (size_t)(g->topk > 0 ? g->topk : 1));
    double *x = (double *)malloc(sizeof(double) * (size_t)max_att * b);
    double *ofg = (double *)malloc(sizeof(double) * (size_t)d), *ol = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
    for (int i = 0; i < m; ++i) {
      int nl = mo_local_set(g, i, loc), ns = 0;
      for (int r = 0; r < g->topk; ++r)
        if (idx[(size_t)i * g->topk + r] >= 0) sel[ns++] = idx[(size_t)i * g->topk + r];
      for (int e = 0; e < b; ++e) {
        int64_t l = block_token(g, i, e);
        double lf = branch_row(g, q, k, v, l, sel, ns, x, ofg);
        double ll = branch_row(g, q, k, v, l, loc, nl, x, ol);
        for (int c = 0; c < d; ++c) {
          double cg = ocg[(size_t)i * d + c];
          O[l * d + c] = gates[l * 3 + 0] * cg + gates[l * 3 + 1] * ofg[c] + gates[l * 3 + 2] * ol[c];
          if (OCG) OCG[l * d + c] = cg;
          if (OFG) OFG[l * d + c] = ofg[c];
          if (OL) OL[l * d + c] = ol[c];
        }
        if (LSE_FG) LSE_FG[l] = lf;
        if (LSE_L) LSE_L[l] = ll;
      }
    }
    free(loc); free(sel); free(x); free(ofg); free(ol);
  }
  free(qm); free(km); free(vm); free(ocg);
  return 0;
}

/*
 * Backward of the three-branch form for one unit, selection held constant.  Unlike the union form, gradient
 * reaches the block-level (routing) scores through the compression branch (the paper's ablation appendix notes
 * that the routing scores are trained through that branch only).  The rounding of the pooled sums to fp32 is
 * treated as the identity.  Outputs in token order: dQ, dK, dV [N,d]; dG [N,3] (gradient of the gates).
 */
int mo_bwd3_unit(const mo_geom *g, const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *d_o,
                 const int32_t *idx, const double *gates, double *dQ, double *dK, double *dV, double *dG) {
  if (!g_ok(g)) return -1;
  int m = g_m(g), b = g_b(g), d = g->d;
  int64_t N = (int64_t)g->nlat * g->nlon;
  double sc = g_scale(g);
  int max_att = MO_MAX_LOCAL + g->topk;
  size_t nd = (size_t)N * d;
  double *O = (double *)malloc(sizeof(double) * nd), *OCG = (double *)malloc(sizeof(double) * nd);
  double *OFG = (double *)malloc(sizeof(double) * nd), *OL = (double *)malloc(sizeof(double) * nd);
  double *LF = (double *)malloc(sizeof(double) * (size_t)N), *LL = (double *)malloc(sizeof(double) * (size_t)N);
  double *AB = (double *)malloc(sizeof(double) * (size_t)m * m);
  double *qm = (double *)malloc(sizeof(double) * (size_t)m * d), *km = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *vm = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *dob = (double *)calloc((size_t)m * d, sizeof(double));   /* gradient of the block's compression output */
  double *dqm = (double *)calloc((size_t)m * d, sizeof(double)), *dkm = (double *)calloc((size_t)m * d, sizeof(double));
  double *dvm = (double *)calloc((size_t)m * d, sizeof(double));
  if (!O || !OCG || !OFG || !OL || !LF || !LL || !AB || !qm || !km || !vm || !dob || !dqm || !dkm || !dvm) return -2;
  mo_fwd3_unit(g, q, k, v, idx, gates, O, OCG, OFG, OL, LF, LL, AB);
  block_means(g, q, qm);
  block_means(g, k, km);
  block_means(g, v, vm);
  /* gates, and the gradient that reaches each block's compression output */
  for (int i = 0; i < m; ++i)
    for (int e = 0; e < b; ++e) {
      int64_t l = block_token(g, i, e);
      double gc = 0.0, gf = 0.0, gl = 0.0;
      for (int c = 0; c < d; ++c) {
        double go = w16(g, d_o[l * d + c]);
        gc += go * OCG[l * d + c];
        gf += go * OFG[l * d + c];
        gl += go * OL[l * d + c];
        dob[(size_t)i * d + c] += gates[l * 3 + 0] * go;
      }
      dG[l * 3 + 0] = gc; dG[l * 3 + 1] = gf; dG[l * 3 + 2] = gl;
    }
  /* compression branch: softmax attention backward on the block means */
  for (int i = 0; i < m; ++i) {
    double Dc = 0.0;
    for (int c = 0; c < d; ++c) Dc += dob[(size_t)i * d + c] * OCG[block_token(g, i, 0) * d + c];
    for (int j = 0; j < m; ++j) {
      double a = AB[(size_t)i * m + j], dp = 0.0;
      for (int c = 0; c < d; ++c) dp += dob[(size_t)i * d + c] * vm[(size_t)j * d + c];
      double ds = a * (dp - Dc);
      for (int c = 0; c < d; ++c) {
        dvm[(size_t)j * d + c] += a * dob[(size_t)i * d + c];
        dqm[(size_t)i * d + c] += sc * ds * km[(size_t)j * d + c];
        dkm[(size_t)j * d + c] += sc * ds * qm[(size_t)i * d + c];
      }
    }
  }
  /* the mean spreads its gradient evenly over the block's tokens */
  for (int j = 0; j < m; ++j)
    for (int e = 0; e < b; ++e) {
      int64_t t = block_token(g, j, e);
      for (int c = 0; c < d; ++c) {
        dQ[t * d + c] = dqm[(size_t)j * d + c] / b;
        dK[t * d + c] = dkm[(size_t)j * d + c] / b;
        dV[t * d + c] = dvm[(size_t)j * d + c] / b;
      }
    }
  /* selection (branch 1) and local (branch 2) attention: per query row; dK, dV gathered per key block */
#pragma omp parallel
  {
    int32_t *blk = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
    double *x = (double *)malloc(sizeof(double) * (size_t)max_att * b);
#pragma omp for schedule(dynamic, 1)
    for (int i = 0; i < m; ++i)
      for (int br = 1; br <= 2; ++br) {
        int nb = 0;
        if (br == 1) { for (int r = 0; r < g->topk; ++r) if (idx[(size_t)i * g->topk + r] >= 0) blk[nb++] = idx[(size_t)i * g->topk + r]; }
        else nb = mo_local_set(g, i, blk);
        if (nb == 0) continue;
        const double *OB = br == 1 ? OFG : OL, *LSE = br == 1 ? LF : LL;
        for (int e = 0; e < b; ++e) {
          int64_t l = block_token(g, i, e);
          double gate = gates[l * 3 + br], D = 0.0;
          for (int c = 0; c < d; ++c) D += gate * w16(g, d_o[l * d + c]) * OB[l * d + c];
          row_logits(g, q, k, l, blk, nb, x);
          for (int a = 0; a < nb; ++a)
            for (int e2 = 0; e2 < b; ++e2) {
              int64_t t = block_token(g, blk[a], e2);
              double w = exp(x[(size_t)a * b + e2] - LSE[l]), dP = 0.0;
              for (int c = 0; c < d; ++c) dP += gate * w16(g, d_o[l * d + c]) * w16(g, v[t * d + c]);
              double dS = w * (dP - D);
              for (int c = 0; c < d; ++c) dQ[l * d + c] += sc * dS * w16(g, k[t * d + c]);
            }
        }
      }
    free(blk); free(x);
  }
#pragma omp parallel
  {
    int32_t *blk = (int32_t *)malloc(sizeof(int32_t) * (size_t)max_att);
#pragma omp for schedule(dynamic, 1)
    for (int j = 0; j < m; ++j)
      for (int i = 0; i < m; ++i)
        for (int br = 1; br <= 2; ++br) {
          int nb = 0, connected = 0;
          if (br == 1) { for (int r = 0; r < g->topk; ++r) if (idx[(size_t)i * g->topk + r] >= 0) blk[nb++] = idx[(size_t)i * g->topk + r]; }
          else nb = mo_local_set(g, i, blk);
          for (int a = 0; a < nb; ++a) connected |= (blk[a] == j);
          if (!connected) continue;
          const double *OB = br == 1 ? OFG : OL, *LSE = br == 1 ? LF : LL;
          for (int e = 0; e < b; ++e) {
            int64_t l = block_token(g, i, e);
            double gate = gates[l * 3 + br], D = 0.0;
            for (int c = 0; c < d; ++c) D += gate * w16(g, d_o[l * d + c]) * OB[l * d + c];
            for (int e2 = 0; e2 < b; ++e2) {
              int64_t t = block_token(g, j, e2);
              double s = 0.0, dP = 0.0;
              for (int c = 0; c < d; ++c) {
                s += w16(g, q[l * d + c]) * w16(g, k[t * d + c]);
                dP += gate * w16(g, d_o[l * d + c]) * w16(g, v[t * d + c]);
              }
              double w = exp(sc * s - LSE[l]), dS = w * (dP - D);
              for (int c = 0; c < d; ++c) {
                dV[t * d + c] += w * gate * w16(g, d_o[l * d + c]);
                dK[t * d + c] += sc * dS * w16(g, q[l * d + c]);
              }
            }
          }
        }
    free(blk);
  }
  free(O); free(OCG); free(OFG); free(OL); free(LF); free(LL); free(AB); free(qm); free(km); free(vm);
  free(dob); free(dqm); free(dkm); free(dvm);
  return 0;
}

/*
 * Two-dimensional rotary position embedding of one [N, d] tensor ("Overall architecture" paragraph: RoPE on
 * queries and keys encodes longitude and latitude, the head dimension split equally between the two
 * coordinates, each half a standard RoPE of its angle in radians; architecture table: theta = 10000).
 * Reading: channels [0, d/2) belong to the longitude, [d/2, d) to the latitude; inside a half of width
 * D = d/2 the pair (2i, 2i+1), i < D/2, turns by the angle  pos * theta^(-2i/D):
 *     y_2i = x_2i cos a - x_2i+1 sin a ,   y_2i+1 = x_2i sin a + x_2i+1 cos a .
 * pos: [N, 2] = (longitude, latitude) of every token in radians.  out: fp64, unrounded (may be NULL);
 * out_bits: the same rounded to bf16, nearest even (may be NULL).
 */
static uint16_t bf16_round(double x) {
  float f = (float)x; /* double -> float -> bf16: the float has 24 bits, bf16 keeps 8; ties of the second step are
                         decided on the float, which is what a device that computes in fp32 does too */
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u); /* NaN stays NaN */
  u += 0x7fffu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

/* double -> float -> binary16, both steps to nearest even */
static uint16_t f16_round(double x) {
  float f = (float)x;
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
  uint32_t a = u & 0x7fffffffu;
  if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);                 /* NaN */
  if (a >= 0x47800000u) return (uint16_t)(sign | 0x7c00u);                /* >= 65536 (or inf): inf; [65520, 65536) rounds below */
  if (a < 0x33000000u) return sign;                                       /* below half the smallest subnormal (2^-25): zero */
  int e = (int)(a >> 23) - 127;                                           /* unbiased exponent of the float */
  uint32_t man = (a & 0x7fffffu) | 0x800000u;                             /* 24-bit significand */
  int shift = e >= -14 ? 13 : 13 + (-14 - e);                             /* bits dropped (more for subnormal results) */
  uint32_t kept = man >> shift, rem = man & ((1u << shift) - 1u), half = 1u << (shift - 1);
  if (rem > half || (rem == half && (kept & 1u))) ++kept;
  uint32_t out = e >= -14 ? (((uint32_t)(e + 15) << 10) + (kept - 0x400u)) : kept;   /* a carry moves into the exponent */
  return (uint16_t)(sign | out);
}

int mo_rope_unit(const mo_geom *g, const uint16_t *x, const double *pos, double theta, double *out, uint16_t *out_bits) {
  if (!g_ok(g) || g->d % 4 || theta <= 0.0) return -1;
  int d = g->d, D = d / 2;
  int64_t N = (int64_t)g->nlat * g->nlon;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < N; ++t)
    for (int half = 0; half < 2; ++half)
      for (int i = 0; i < D / 2; ++i) {
        double a = pos[t * 2 + half] * pow(theta, -2.0 * i / D);
        double c = cos(a), s = sin(a);
        int64_t e = t * d + half * D + 2 * i;
        double x0 = w16(g, x[e]), x1 = w16(g, x[e + 1]);
        double y0 = x0 * c - x1 * s, y1 = x0 * s + x1 * c;
        if (out) { out[e] = y0; out[e + 1] = y1; }
        if (out_bits) {
          out_bits[e] = g->f16 ? f16_round(y0) : bf16_round(y0);
          out_bits[e + 1] = g->f16 ? f16_round(y1) : bf16_round(y1);
        }
      }
  return 0;
}

/* The storage type's decoding on its own (for the tests that pin it against a library's conversion). */
int mo_widen16(const mo_geom *g, const uint16_t *x, int64_t n, double *out) {
  if (!g) return -1;
  for (int64_t i = 0; i < n; ++i) out[i] = w16(g, x[i]);
  return 0;
}
