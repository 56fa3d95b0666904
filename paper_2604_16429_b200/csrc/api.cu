// C ABI of the library: argument validation, workspace carving, kernel launches.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace mosaic {

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

int validate(const mosaic_bsa_params* p, Geo* g) {
  if (!p) return MOSAIC_E_INVALID_ARG;
  if (p->B <= 0 || p->H <= 0 || p->nlat <= 0 || p->nlon <= 0 || p->bh <= 0 || p->bw <= 0 || p->topk < 0 ||
      p->rlat < 0 || p->rlon < 0 || (p->flags & ~(MOSAIC_FLAG_LOCAL_GROUPS | MOSAIC_FLAG_FP16)) != 0)
    return MOSAIC_E_INVALID_ARG;
  if (p->nlat % p->bh || p->nlon % p->bw) return MOSAIC_E_INVALID_ARG;
  if (!(p->scale == p->scale) || isinf(p->scale)) return MOSAIC_E_INVALID_ARG;
  if (p->d != kD) return MOSAIC_E_UNSUPPORTED;
  if (!(p->bw == 8 || p->bw == 16)) return MOSAIC_E_UNSUPPORTED;
  const int crows = kChunk / p->bw;
  if (p->bh % crows) return MOSAIC_E_UNSUPPORTED;
  const int cpb = p->bh * p->bw / kChunk;
  if (!(cpb == 1 || cpb % 2 == 0)) return MOSAIC_E_UNSUPPORTED;
  const bool groups = (p->flags & MOSAIC_FLAG_LOCAL_GROUPS) != 0;
  if (groups && (p->rlat < 1 || p->rlon < 1)) return MOSAIC_E_INVALID_ARG;
  if (p->topk > kMaxTopk) return MOSAIC_E_UNSUPPORTED;
  if (groups ? (long long)p->rlat * p->rlon > 32 : (p->rlat > 2 || p->rlon > 2)) return MOSAIC_E_UNSUPPORTED;
  const int nlocal = groups ? p->rlat * p->rlon : (2 * p->rlat + 1) * (2 * p->rlon + 1);
  if (nlocal + p->topk > kMaxList) return MOSAIC_E_UNSUPPORTED;
  const long long U = (long long)p->B * p->H, N = (long long)p->nlat * p->nlon;
  const long long m = (long long)(p->nlat / p->bh) * (p->nlon / p->bw);
  if (U > (1 << 24) || m > (1 << 24) || U * m * cpb > 0x7fffffffll || U * N > (1ll << 40)) return MOSAIC_E_UNSUPPORTED;
  const int hkv = p->Hkv == 0 ? p->H : p->Hkv;
  if (hkv <= 0 || p->H % hkv) return MOSAIC_E_INVALID_ARG;
  g->U = (int)U;
  g->H = p->H; g->Hkv = hkv; g->Ukv = p->B * hkv;
  g->nlat = p->nlat; g->nlon = p->nlon; g->bh = p->bh; g->bw = p->bw;
  g->nbh = p->nlat / p->bh; g->nbw = p->nlon / p->bw; g->m = (int)m;
  g->b = p->bh * p->bw; g->cpb = cpb; g->crows = crows;
  g->rlat = p->rlat; g->rlon = p->rlon; g->topk = p->topk;
  g->local_off = 0;
  g->local_groups = groups ? 1 : 0;
  g->f16 = (p->flags & MOSAIC_FLAG_FP16) ? 1 : 0;
  g->scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf((float)p->d);
  g->scale_log2 = g->scale * 1.4426950408889634f;
  g->N = N;
  return MOSAIC_OK;
}

SelectWs select_layout(const Geo& g) {
  SelectWs w;
  const size_t pooled = align256(sizeof(float) * (size_t)g.U * g.m * kD), norms = align256(sizeof(float) * (size_t)g.U * g.m);
  w.pq = kStatusBytes;
  w.pk = w.pq + pooled;
  w.nq = w.pk + pooled;
  w.nk = w.nq + norms;
  w.total = w.nk + norms;
  return w;
}

BranchWs branch_layout(const Geo& g) {
  BranchWs w;
  const size_t pooled = align256(sizeof(float) * (size_t)g.U * g.m * kD), norms = align256(sizeof(float) * (size_t)g.U * g.m);
  const size_t full = align256(2 * (size_t)g.U * g.N * kD);
  w.pq = kStatusBytes;
  w.pk = w.pq + pooled;
  w.pv = w.pk + pooled;
  w.nrm = w.pv + pooled;
  w.ocg = w.nrm + 2 * norms;
  w.ofg = w.ocg + pooled;
  w.ol = w.ofg + full;
  w.total = w.ol + full;
  return w;
}

namespace {

struct BwdWs { size_t D, negD, nlse2, off, q, order, total; };
BwdWs bwd_layout(const Geo& g) {
  BwdWs w;
  size_t at = kStatusBytes;
  w.D = at; at = align256(at + sizeof(float) * (size_t)g.U * g.N);
  w.negD = at; at = align256(at + sizeof(float) * (size_t)g.U * g.N);
  w.nlse2 = at; at = align256(at + sizeof(float) * (size_t)g.U * g.N);
  w.off = at; at = align256(at + sizeof(int32_t) * (size_t)g.U * (g.m + 1));
  w.q = at; at = align256(at + sizeof(int32_t) * (size_t)g.U * g.m * (g.topk > 0 ? g.topk : 1));
  // dK/dV items (two 128-row tiles per 256-row item of a key/value unit), longest first, and their cost classes
  w.order = at; at = align256(at + 2 * sizeof(int32_t) * 2 * (size_t)g.Ukv * items_per_unit(g));
  w.total = at;
  return w;
}
// Scratch of the three-branch backward: the forward's (pooled sums, obar, both branch outputs), the branch
// log-sum-exps, the block-level backward's vectors, the gated copies of dO, the branch gradients, and the
// attention backward's own scratch (used by the two passes in turn).
struct BwdBranchWs {
  BranchWs f;
  size_t lse_fg, lse_l, lse_cg, delta, dob, dqm, dkm, dvm, do_fg, do_l, dq_fg, dq_l, dk_fg, dk_l, dv_fg, dv_l, inner, total;
};
BwdBranchWs bwd_branch_layout(const Geo& g) {
  BwdBranchWs w;
  w.f = branch_layout(g);
  const size_t pooled = align256(sizeof(float) * (size_t)g.U * g.m * kD), rows = align256(sizeof(float) * (size_t)g.U * g.N);
  const size_t blocks = align256(sizeof(float) * (size_t)g.U * g.m);
  const size_t full = align256(2 * (size_t)g.U * g.N * kD);
  size_t at = w.f.total;
  w.lse_fg = at; at += rows;
  w.lse_l = at; at += rows;
  w.lse_cg = at; at += blocks;
  w.delta = at; at += blocks;
  w.dob = at; at += pooled;
  w.dqm = at; at += pooled;
  w.dkm = at; at += pooled;
  w.dvm = at; at += pooled;
  size_t* fulls[] = {&w.do_fg, &w.do_l, &w.dq_fg, &w.dq_l, &w.dk_fg, &w.dk_l, &w.dv_fg, &w.dv_l};
  for (size_t* f : fulls) { *f = at; at += full; }
  w.inner = at;  // the attention backward's layout starts with a status block of its own (unused here)
  w.total = at + bwd_layout(g).total;
  return w;
}
size_t select_total(const Geo& g) { return select_layout(g).total; }

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int device_ok() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 64 && cached[dev]) return cached[dev] > 0 ? MOSAIC_OK : MOSAIC_E_UNSUPPORTED;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 64) cached[dev] = major == 10 ? 1 : -1;
  return major == 10 ? MOSAIC_OK : MOSAIC_E_UNSUPPORTED;
}

int begin(const mosaic_bsa_params* p, void* ws, size_t ws_bytes, size_t need, void* stream, HostCtx* c) {
  int rc = validate(p, &c->g);
  if (rc) return rc;
  if (!ws) return MOSAIC_E_INVALID_ARG;
  if (!aligned(ws, 256)) return MOSAIC_E_MISALIGNED;
  if (ws_bytes < need) return MOSAIC_E_WORKSPACE_TOO_SMALL;
  if ((rc = device_ok())) return rc;
  c->stream = (cudaStream_t)stream;
  c->status = (int*)ws;
  if (cudaMemsetAsync(ws, 0, kStatusBytes, c->stream) != cudaSuccess) return MOSAIC_E_CUDA;
  return MOSAIC_OK;
}

}  // namespace
}  // namespace mosaic

using namespace mosaic;

extern "C" {

size_t mosaic_bsa_workspace_bytes(const mosaic_bsa_params* p, int op) {
  Geo g;
  if (validate(p, &g)) return 0;
  switch (op) {
    case MOSAIC_OP_SELECT: return select_total(g);
    case MOSAIC_OP_FWD: return kStatusBytes;
    case MOSAIC_OP_BWD: return bwd_layout(g).total;
    case MOSAIC_OP_FWD_BRANCHES: return branch_layout(g).total;
    case MOSAIC_OP_BWD_BRANCHES: return bwd_branch_layout(g).total;
    default: return 0;
  }
}

int mosaic_bsa_select(const mosaic_bsa_params* p, const void* q, const void* k, int32_t* block_idx, void* ws,
                      size_t ws_bytes, void* cuda_stream) {
  HostCtx c;
  Geo g;
  int rc = validate(p, &g);
  if (rc) return rc;
  if (!q || !k || (!block_idx && g.topk > 0)) return MOSAIC_E_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(block_idx, 4)) return MOSAIC_E_MISALIGNED;
  if ((rc = begin(p, ws, ws_bytes, select_total(g), cuda_stream, &c))) return rc;
  const SelectWs w = select_layout(g);
  char* base = (char*)ws;
  return launch_select(c, q, k, block_idx, (float*)(base + w.pq), (float*)(base + w.pk), (float*)(base + w.nq),
                       (float*)(base + w.nk));
}

int mosaic_bsa_fwd(const mosaic_bsa_params* p, const void* q, const void* k, const void* v,
                   const int32_t* block_idx, void* o, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
  HostCtx c;
  Geo g;
  int rc = validate(p, &g);
  if (rc) return rc;
  if (!q || !k || !v || !o || !lse || (!block_idx && g.topk > 0)) return MOSAIC_E_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16) || !aligned(lse, 4) ||
      !aligned(block_idx, 4))
    return MOSAIC_E_MISALIGNED;
  if ((rc = begin(p, ws, ws_bytes, kStatusBytes, cuda_stream, &c))) return rc;
  return launch_fwd_tc(c, q, k, v, block_idx, o, lse, c.status + 1);
}

int mosaic_bsa_fwd_branches(const mosaic_bsa_params* p, const void* q, const void* k, const void* v,
                            const int32_t* block_idx, const float* gates, void* o, float* lse_fg, float* lse_l, void* ws,
                            size_t ws_bytes, void* cuda_stream) {
  HostCtx c;
  Geo g;
  int rc = validate(p, &g);
  if (rc) return rc;
  if (!q || !k || !v || !gates || !o || !lse_fg || !lse_l || (!block_idx && g.topk > 0)) return MOSAIC_E_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16) || !aligned(gates, 4) ||
      !aligned(lse_fg, 4) || !aligned(lse_l, 4) || !aligned(block_idx, 4))
    return MOSAIC_E_MISALIGNED;
  const BranchWs w = branch_layout(g);
  if ((rc = begin(p, ws, ws_bytes, w.total, cuda_stream, &c))) return rc;
  char* base = (char*)ws;
  float *pq = (float*)(base + w.pq), *pk = (float*)(base + w.pk), *pv = (float*)(base + w.pv);
  float *nrm = (float*)(base + w.nrm), *ocg = (float*)(base + w.ocg);
  void *ofg = base + w.ofg, *ol = base + w.ol;
  // compression branch: pooled sums of Q, K (with their norms, unused here) and V, then block-level attention
  HostCtx cp = c;
  cp.g.topk = 0;  // pooling only
  if ((rc = launch_select(cp, q, k, nullptr, pq, pk, nrm, nrm + (size_t)g.U * g.m))) return rc;
  if ((rc = launch_pool_one(c, v, pv, nrm, g.Ukv))) return rc;
  if ((rc = launch_compress(c, pq, pk, pv, ocg, nullptr))) return rc;
  // local branch: the neighbourhood only (no selected blocks); work queue in the second word of the status block
  HostCtx cl = c;
  cl.g.topk = 0;
  if ((rc = launch_fwd_tc(cl, q, k, v, nullptr, ol, lse_l, c.status + 1))) return rc;
  // selection branch: the selected blocks only; work queue in the third word
  HostCtx cs = c;
  cs.g.local_off = 1;
  if ((rc = launch_fwd_tc(cs, q, k, v, block_idx, ofg, lse_fg, c.status + 2))) return rc;
  return launch_combine(c, ocg, ofg, ol, gates, o);
}

int mosaic_bsa_bwd(const mosaic_bsa_params* p, const void* q, const void* k, const void* v, const void* o,
                   const float* lse, const void* d_o, const int32_t* block_idx, void* dq, void* dk, void* dv,
                   void* ws, size_t ws_bytes, void* cuda_stream) {
  HostCtx c;
  Geo g;
  int rc = validate(p, &g);
  if (rc) return rc;
  if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv || (!block_idx && g.topk > 0))
    return MOSAIC_E_INVALID_ARG;
  const void* ptrs[] = {q, k, v, o, d_o, dq, dk, dv};
  for (const void* x : ptrs)
    if (!aligned(x, 16)) return MOSAIC_E_MISALIGNED;
  if (!aligned(lse, 4) || !aligned(block_idx, 4)) return MOSAIC_E_MISALIGNED;
  if (2 * (size_t)g.m * sizeof(int) + (size_t)g.m * g.topk / 8 + 8 > 200 * 1024) return MOSAIC_E_UNSUPPORTED;  // transposed-pattern kernel
  BwdWs w = bwd_layout(g);
  if ((rc = begin(p, ws, ws_bytes, w.total, cuda_stream, &c))) return rc;
  char* base = (char*)ws;
  return launch_bwd(c, q, k, v, o, lse, d_o, block_idx, dq, dk, dv, (float*)(base + w.D),
                    (float*)(base + w.negD), (float*)(base + w.nlse2), (int32_t*)(base + w.off),
                    (int32_t*)(base + w.q), (int32_t*)(base + w.order), c.status + 1);
}

int mosaic_bsa_bwd_branches(const mosaic_bsa_params* p, const void* q, const void* k, const void* v,
                            const int32_t* block_idx, const float* gates, const void* d_o, void* dq, void* dk,
                            void* dv, float* dgates, void* ws, size_t ws_bytes, void* cuda_stream) {
  HostCtx c;
  Geo g;
  int rc = validate(p, &g);
  if (rc) return rc;
  if (!q || !k || !v || !gates || !d_o || !dq || !dk || !dv || !dgates || (!block_idx && g.topk > 0))
    return MOSAIC_E_INVALID_ARG;
  const void* ptrs[] = {q, k, v, d_o, dq, dk, dv};
  for (const void* x : ptrs)
    if (!aligned(x, 16)) return MOSAIC_E_MISALIGNED;
  if (!aligned(gates, 4) || !aligned(dgates, 4) || !aligned(block_idx, 4)) return MOSAIC_E_MISALIGNED;
  if (2 * (size_t)g.m * sizeof(int) + (size_t)g.m * g.topk / 8 + 8 > 200 * 1024) return MOSAIC_E_UNSUPPORTED;  // transposed-pattern kernel
  const BwdBranchWs w = bwd_branch_layout(g);
  if ((rc = begin(p, ws, ws_bytes, w.total, cuda_stream, &c))) return rc;
  char* base = (char*)ws;
  auto F = [&](size_t off) { return (float*)(base + off); };
  float *pq = F(w.f.pq), *pk = F(w.f.pk), *pv = F(w.f.pv), *nrm = F(w.f.nrm), *ocg = F(w.f.ocg);
  void *ofg = base + w.f.ofg, *ol = base + w.f.ol;
  // the forward again: pooled sums, block-level attention (with its log-sum-exp), both attention branches
  HostCtx cp = c;
  cp.g.topk = 0;  // pooling only
  if ((rc = launch_select(cp, q, k, nullptr, pq, pk, nrm, nrm + (size_t)g.U * g.m))) return rc;
  if ((rc = launch_pool_one(c, v, pv, nrm, g.Ukv))) return rc;
  if ((rc = launch_compress(c, pq, pk, pv, ocg, F(w.lse_cg)))) return rc;
  HostCtx cl = c;
  cl.g.topk = 0;          // local branch: the neighbourhood only
  HostCtx cs = c;
  cs.g.local_off = 1;     // selection branch: the selected blocks only
  const bool sel = g.topk > 0;
  if ((rc = launch_fwd_tc(cl, q, k, v, nullptr, ol, F(w.lse_l), c.status + 1))) return rc;
  if (sel) {
    if ((rc = launch_fwd_tc(cs, q, k, v, block_idx, ofg, F(w.lse_fg), c.status + 2))) return rc;
  } else if (cudaMemsetAsync(ofg, 0, 2 * (size_t)g.U * g.N * kD, c.stream) != cudaSuccess) {
    return MOSAIC_E_CUDA;
  }
  // gate gradients, gated copies of dO, gated block sums of dO
  if ((rc = launch_gate(c, d_o, ofg, ol, ocg, gates, dgates, base + w.do_fg, base + w.do_l, F(w.dob)))) return rc;
  // compression branch on the block level
  if ((rc = launch_compress_bwd(c, pq, pk, pv, F(w.dob), ocg, F(w.lse_cg), F(w.delta), F(w.dqm), F(w.dkm), F(w.dvm))))
    return rc;
  // the two attention branches, one after the other on the same scratch
  const BwdWs bw = bwd_layout(g);
  char* in = base + w.inner;
  auto attention_bwd = [&](const HostCtx& cx, const void* o_x, const float* lse_x, const void* do_x, const int32_t* idx,
                           void* dq_x, void* dk_x, void* dv_x, int* counters) {
    return launch_bwd(cx, q, k, v, o_x, lse_x, do_x, idx, dq_x, dk_x, dv_x, (float*)(in + bw.D), (float*)(in + bw.negD),
                      (float*)(in + bw.nlse2), (int32_t*)(in + bw.off), (int32_t*)(in + bw.q), (int32_t*)(in + bw.order),
                      counters);
  };
  if ((rc = attention_bwd(cl, ol, F(w.lse_l), base + w.do_l, nullptr, base + w.dq_l, base + w.dk_l, base + w.dv_l,
                          c.status + 3)))
    return rc;
  if (sel && (rc = attention_bwd(cs, ofg, F(w.lse_fg), base + w.do_fg, block_idx, base + w.dq_fg, base + w.dk_fg,
                                 base + w.dv_fg, c.status + 5)))
    return rc;
  // sums: both attention branches plus what the compression branch gives every token of a block
  if ((rc = launch_grad_sum(c, g.U, base + w.dq_l, sel ? base + w.dq_fg : nullptr, F(w.dqm), dq))) return rc;
  if ((rc = launch_grad_sum(c, g.Ukv, base + w.dk_l, sel ? base + w.dk_fg : nullptr, F(w.dkm), dk))) return rc;
  return launch_grad_sum(c, g.Ukv, base + w.dv_l, sel ? base + w.dv_fg : nullptr, F(w.dvm), dv);
}

int mosaic_bsa_rope(const mosaic_bsa_params* p, const void* q, const void* k, const float* pos, float theta, void* q_out,
                    void* k_out, void* cuda_stream) {
  HostCtx c;
  int rc = validate(p, &c.g);
  if (rc) return rc;
  if (!q || !k || !pos || !q_out || !k_out || !(theta > 0.f)) return MOSAIC_E_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(q_out, 16) || !aligned(k_out, 16) || !aligned(pos, 4))
    return MOSAIC_E_MISALIGNED;
  if ((rc = device_ok())) return rc;
  c.stream = (cudaStream_t)cuda_stream;
  c.status = nullptr;
  return launch_rope(c, q, k, pos, (double)theta, q_out, k_out);
}

int mosaic_bsa_last_status(const void* ws, void* cuda_stream) {
  if (!ws) return MOSAIC_E_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return MOSAIC_E_CUDA;
  int st = 0;
  if (cudaMemcpy(&st, ws, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return MOSAIC_E_CUDA;
  return st;
}

const char* mosaic_bsa_strerror(int code) {
  switch (code) {
    case MOSAIC_OK: return "ok";
    case MOSAIC_E_INVALID_ARG: return "invalid argument";
    case MOSAIC_E_UNSUPPORTED: return "unsupported shape, option or device";
    case MOSAIC_E_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MOSAIC_E_MISALIGNED: return "misaligned pointer";
    case MOSAIC_E_CUDA: return "CUDA call failed";
    case MOSAIC_E_DEVICE_TIMEOUT: return "device: bounded wait ran out";
    case MOSAIC_E_DEVICE_BAD_INDEX: return "device: block id out of range, inside the local set, or repeated in its row";
    default: return "unknown code";
  }
}

}  // extern "C"
