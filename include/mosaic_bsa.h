/*
 * mosaic_bsa.h -- C ABI of the MOSAIC mesh-aligned block-sparse attention hot path
 * for NVIDIA B200 (sm_100a).
 *
 * Method (paper: section "Block-Sparse Attention", paragraphs "Compression",
 * "Selection", "Local Attention"; appendix "Block-sparse attention implementation",
 * paragraph "Kernel Design"):  the N = nlat*nlon tokens of a lat-lon grid are tiled
 * into bh x bw blocks.  Every query block attends ONE key/value set shared by all of
 * its tokens: its local mesh neighbourhood (own block and the blocks within
 * rlat/rlon block rows/columns; longitude periodic, latitude clamped, every block
 * counted once) plus the top-k non-local blocks ranked by the dot product of the
 * mean-pooled query block with the mean-pooled key block.  Attention over that union
 * is one softmax (scale 1/sqrt(d) unless given).
 *
 * Common rules for every entry point
 *   - All tensor pointers are DEVICE pointers on the current CUDA device.  Q, K, V, O,
 *     dO are contiguous [B, H, N, d] bf16 with token t = lat*nlon + lon, base address
 *     16-byte aligned.  "unit" u = b*H + h; units are independent.  With grouped-query
 *     attention (Hkv < H; paper: "Overall architecture" paragraph, GQA ratio 4) K, V, dK, dV
 *     are [B, Hkv, N, d] and query head h reads key/value head h / (H / Hkv); the selection
 *     stays per query head, dK and dV sum over the query heads of a group.
 *   - block_idx is contiguous [B, H, m, topk] int32, m = (nlat/bh)*(nlon/bw), block id
 *     j = by*(nlon/bw) + bx.  Row i holds the selected non-local block ids of query
 *     block i, best first, padded with -1.  The local set is implicit.
 *   - The caller owns every buffer, including the workspace `ws` (device memory, 256-byte
 *     aligned, at least mosaic_bsa_workspace_bytes() long).  The library allocates no
 *     device memory.  Host-side state: a small cache of TMA descriptors keyed by (device, base
 *     pointer, geometry) and per-device launch attributes; mosaic_bsa_select_static also keeps the
 *     device address of its fixed scratch array.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t, NULL = default stream) and
 *     return without synchronising.  Two calls that share a workspace must be ordered
 *     on one stream.
 *   - Return value: MOSAIC_OK or a negative MOSAIC_E_* code; nothing aborts, traps or
 *     throws across the boundary.  Faults detected on the device (a bounded wait that
 *     ran out, a block id out of range) do not fault the GPU: the kernel records a code
 *     in the first word of the workspace, skips the offending work and returns; read it
 *     with mosaic_bsa_last_status().
 *   - Supported in this version: d = 64; bw = 8 or 16 with bh a multiple of 64/bw
 *     (8x8, 16x16 and 8x16 are the tested shapes); rlat, rlon in 0..2 (group mode: rlat*rlon
 *     <= 32); (local blocks + topk)
 *     <= 64; topk <= 32; any B, H and any grid with nlat % bh == 0, nlon % bw == 0
 *     (grids with fewer than 2*rlon+1 block columns de-duplicate the neighbourhood).
 */
#ifndef MOSAIC_BSA_H_
#define MOSAIC_BSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mosaic_bsa_params {
  int32_t B, H;       /* batch (ensemble members) and heads; Q, K, V share H          */
  int32_t nlat, nlon; /* grid; N = nlat*nlon                                           */
  int32_t d;          /* head dimension (64)                                           */
  int32_t bh, bw;     /* block shape in grid points                                    */
  int32_t rlat, rlon; /* local neighbourhood radius in blocks (1,1 = 3x3); with
                         MOSAIC_FLAG_LOCAL_GROUPS: height and width of the local group    */
  int32_t topk;       /* selected non-local blocks per query block, >= 0               */
  float scale;        /* softmax scale; <= 0 means 1/sqrt(d)                           */
  uint32_t flags;     /* 0 or a sum of MOSAIC_FLAG_LOCAL_GROUPS, MOSAIC_FLAG_FP16      */
  int32_t Hkv;        /* heads of K and V (grouped-query attention, the paper's GQA ratio
                         H / Hkv); 0 means H; H % Hkv == 0                                */
} mosaic_bsa_params;

/* Local attention inside aligned groups of blocks instead of a sliding neighbourhood (the paper's "Local
 * Attention" paragraph: dense attention inside large blocks, computed independently): the local set of a block
 * is the aligned tile of rlat x rlon blocks that contains it (rlat, rlon >= 1, rlat*rlon <= 32; the last group
 * of a row or column may be ragged).  The paper's HEALPix layout -- 128 contiguous tokens per block, local
 * blocks of 1024 tokens -- is nlat = N/16, nlon = 16, bh = 8, bw = 16, rlat = 8, rlon = 1 with this flag. */
#define MOSAIC_FLAG_LOCAL_GROUPS 1u
/* The 16-bit tensors (q, k, v, o, d_o, dq, dk, dv and the rotated q, k) are IEEE binary16 instead of bf16
 * wherever a comment says "bf16" (appendix, "Distributed training" paragraph: the paper trains entirely in
 * float16).  Arithmetic is unchanged: tensor-core products of 16-bit operands with fp32 accumulation, fp32
 * softmax, selection on the exactly widened values. */
#define MOSAIC_FLAG_FP16 2u

enum { MOSAIC_OP_SELECT = 0, MOSAIC_OP_FWD = 1, MOSAIC_OP_BWD = 2, MOSAIC_OP_FWD_BRANCHES = 3,
       MOSAIC_OP_BWD_BRANCHES = 4 };

enum {
  MOSAIC_OK = 0,
  MOSAIC_E_INVALID_ARG = -1,        /* null pointer, non-divisible grid, negative size    */
  MOSAIC_E_UNSUPPORTED = -2,        /* d, block shape, radius or device not supported     */
  MOSAIC_E_WORKSPACE_TOO_SMALL = -3,
  MOSAIC_E_MISALIGNED = -4,         /* a tensor base or the workspace is not aligned      */
  MOSAIC_E_CUDA = -5,               /* a CUDA runtime/driver call failed (launch, query)  */
  /* device-side status codes (mosaic_bsa_last_status) */
  MOSAIC_E_DEVICE_TIMEOUT = -16,    /* a bounded wait on an on-chip barrier ran out       */
  MOSAIC_E_DEVICE_BAD_INDEX = -17   /* a row of block_idx held an id outside [-1, m), an id
                                       inside the row's local set, or the same id twice      */
};

/* Bytes of device workspace the given op needs for these params (0 on invalid params).
 * The first 256 bytes of any workspace are the status block. */
size_t mosaic_bsa_workspace_bytes(const mosaic_bsa_params *p, int op);

/*
 * Selection ("Compression" + "Selection" paragraphs: pooled block representations,
 * block-level scores, top-n per query block).
 *   q, k       in   [B,H,N,d] bf16
 *   block_idx  out  [B,H,m,topk] int32
 * Arithmetic is fixed so that the result is unique: block sums accumulate in fp64 in
 * row-major order inside the block and round once to fp32; a score is the fp64 sum, in
 * channel order, of the exact products of those fp32 values; order = (score descending,
 * block id ascending); +0 and -0 tie; a NaN score ranks after every number, -inf included
 * (inputs are expected to be finite; this only fixes what happens when they are not).
 * The selection kernels detect no device-side faults and never write the status word.
 */
int mosaic_bsa_select(const mosaic_bsa_params *p, const void *q, const void *k, int32_t *block_idx,
                      void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Forward (fine-grained attention equation of the "Selection" paragraph over the union
 * of local and selected blocks; streaming evaluation per the "Kernel Design" paragraph).
 *   q, k, v    in   [B,H,N,d] bf16
 *   block_idx  in   [B,H,m,topk] int32 (from mosaic_bsa_select or the caller: ids in
 *                   [0,m) or -1, no repeats in a row, none inside the row's local set.  An
 *                   entry that breaks these rules is skipped -- a block is never attended
 *                   twice -- and MOSAIC_E_DEVICE_BAD_INDEX is recorded; the backward applies
 *                   the same rule, so it stays the gradient of what the forward computed)
 *   o          out  [B,H,N,d] bf16
 *   lse        out  [B,H,N] fp32, natural-log sum-exp of the scaled logits of each row
 */
int mosaic_bsa_fwd(const mosaic_bsa_params *p, const void *q, const void *k, const void *v,
                   const int32_t *block_idx, void *o, float *lse, void *ws, size_t ws_bytes,
                   void *cuda_stream);

/*
 * Forward in the paper's three-branch form (Eq. of the aggregated output, section "Native Sparse
 * Attention"; "Compression", "Selection" and "Local Attention" paragraphs of the section
 * "Block-Sparse Attention"):  for token l of query block i
 *     o_l = gates[l][0] * oCG_i + gates[l][1] * oFG_l + gates[l][2] * oL_l
 *   oCG_i  block-level softmax attention over ALL m blocks on the mean-pooled queries, keys and
 *          values (the same vector for every token of the block),
 *   oFG_l  softmax attention of q_l over the tokens of the selected blocks of row i of block_idx
 *          (own normaliser; an empty row gives 0 and a log-sum-exp of -inf),
 *   oL_l   softmax attention of q_l over the tokens of the local neighbourhood (own normaliser).
 * The gates are learned functions of the layer input in the paper and therefore inputs here.
 *   q, k, v    in   [B,H,N,d] bf16
 *   block_idx  in   [B,H,m,topk] int32, same rules as mosaic_bsa_fwd
 *   gates      in   [B,H,N,3] fp32, order (compression, selection, local)
 *   o          out  [B,H,N,d] bf16
 *   lse_fg, lse_l  out  [B,H,N] fp32, natural-log sum-exp of the selection and local branches
 * Workspace: mosaic_bsa_workspace_bytes(p, MOSAIC_OP_FWD_BRANCHES) (pooled sums, the block-level output
 * and the two branch outputs in bf16).
 */
int mosaic_bsa_fwd_branches(const mosaic_bsa_params *p, const void *q, const void *k, const void *v,
                            const int32_t *block_idx, const float *gates, void *o, float *lse_fg,
                            float *lse_l, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Backward (gradient of the forward with the selection held constant; dK/dV visit only
 * the query blocks connected to a key/value block, "Kernel Design" paragraph).
 *   q, k, v, o, d_o  in   [B,H,N,d] bf16;  lse in [B,H,N] fp32 (from mosaic_bsa_fwd)
 *   dq, dk, dv       out  [B,H,N,d] bf16
 * Results are deterministic (fixed summation order, no floating-point atomics).
 */
int mosaic_bsa_bwd(const mosaic_bsa_params *p, const void *q, const void *k, const void *v,
                   const void *o, const float *lse, const void *d_o, const int32_t *block_idx,
                   void *dq, void *dk, void *dv, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Backward of the three-branch form (gradient of mosaic_bsa_fwd_branches with the selection held constant).
 * Each attention branch is a softmax attention of its own, so each takes the attention backward with dO
 * scaled by its gate; the compression branch is differentiated on the block level (softmax backward on the
 * mean-pooled vectors; a mean spreads its gradient evenly over the block's tokens), which is the only path by
 * which gradient reaches the block-level (routing) scores (the paper's ablation appendix: the routing scores
 * are trained through the compression branch).  The forward's intermediates are recomputed, so nothing of the
 * forward call has to be kept.
 *   q                in   [B,H,N,d] bf16;  k, v in [B,Hkv,N,d] bf16
 *   block_idx        in   [B,H,m,topk] int32, same rules as mosaic_bsa_fwd
 *   gates            in   [B,H,N,3] fp32, order (compression, selection, local)
 *   d_o              in   [B,H,N,d] bf16, gradient of the forward's o
 *   dq               out  [B,H,N,d] bf16;  dk, dv out [B,Hkv,N,d] bf16
 *   dgates           out  [B,H,N,3] fp32, dgates[l][x] = <d_o_l, branch output x of token l>
 * Workspace: mosaic_bsa_workspace_bytes(p, MOSAIC_OP_BWD_BRANCHES) (about ten tensors of the size of q).
 * Results are deterministic.  Errors as for mosaic_bsa_bwd.
 */
int mosaic_bsa_bwd_branches(const mosaic_bsa_params *p, const void *q, const void *k, const void *v,
                            const int32_t *block_idx, const float *gates, const void *d_o, void *dq,
                            void *dk, void *dv, float *dgates, void *ws, size_t ws_bytes,
                            void *cuda_stream);

/*
 * Two-dimensional rotary position embedding of queries and keys ("Overall architecture" paragraph: RoPE encodes
 * longitude and latitude, the head dimension split equally between the two coordinates, each half a standard
 * RoPE of its angle in radians; architecture table: theta = 10000).  Channels [0, d/2) turn with the longitude,
 * [d/2, d) with the latitude; inside a half of width D = d/2 the pair (2i, 2i+1) turns by pos * theta^(-2i/D).
 * The paper applies it before the attention operator; the other entry points take what this one writes.
 *   q        in   [B,H,N,d] bf16;  k  in  [B,Hkv,N,d] bf16
 *   pos      in   [N,2] fp32, (longitude, latitude) of every token in radians (the same for all units)
 *   theta    in   base of the frequencies (> 0)
 *   q_out, k_out  out  same shapes as q, k (may be q, k themselves: every element is read once, then written)
 * No workspace and no status word; errors are the host-side codes only.  The other fields of `p` than B, H, Hkv and
 * the grid must still describe a valid problem.
 */
int mosaic_bsa_rope(const mosaic_bsa_params *p, const void *q, const void *k, const float *pos, float theta,
                    void *q_out, void *k_out, void *cuda_stream);

/*
 * Selection for callers that cannot allocate device memory.  (The paper has no counterpart of this
 * entry point: it computes exactly what mosaic_bsa_select computes, with the same arguments minus the
 * workspace.)
 *
 * Some callers cannot hand the library a workspace: a process whose framework claimed its whole memory
 * budget at start-up, a plug-in whose host application owns the allocator, a latency-critical loop in
 * which cudaMalloc (it may synchronise the device) is forbidden.  For them the scratch of the selection
 * (the pooled block sums of Q and K and the norms of those sums) lives in a fixed array inside the library image,
 * MOSAIC_BSA_STATIC_SCRATCH_BYTES long; every GPU that loads the library holds that array until the
 * process exits.  The call performs no cudaMalloc, cudaFree or other allocating routine.
 *   q, k       in   [B,H,N,d] bf16 (device)
 *   block_idx  out  [B,H,m,topk] int32 (device)
 * Limits and rules
 *   - The problem must fit: 256 + 2 * round_up_256(B*H*m*d*4) + 2 * round_up_256(B*H*m*4)
 *     <= MOSAIC_BSA_STATIC_SCRATCH_BYTES (= mosaic_bsa_workspace_bytes(p, MOSAIC_OP_SELECT)), i.e. about
 *     B*H*m <= 8060 blocks for d = 64 (the 1.5-degree grid with 8 heads uses 3600).  A larger
 *     problem returns MOSAIC_E_WORKSPACE_TOO_SMALL and launches nothing.
 *   - The first call on each device looks up the device address of the array (with that device current)
 *     and remembers it; make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents (the call
 *     clears what has to start at zero).  Two calls that overlap on the GPU -- different streams without
 *     an ordering between them -- race on it: keep calls of this entry point ordered.
 *   - Other return codes as for mosaic_bsa_select.  There is no status word to read afterwards (the
 *     selection kernels record no device-side faults), so mosaic_bsa_last_status has no counterpart here.
 */
#define MOSAIC_BSA_STATIC_SCRATCH_BYTES (4u << 20)
int mosaic_bsa_select_static(const mosaic_bsa_params *p, const void *q, const void *k, int32_t *block_idx,
                             void *cuda_stream);

/* Synchronises `cuda_stream`, then returns the device status word of `ws`
 * (MOSAIC_OK, MOSAIC_E_DEVICE_*) or MOSAIC_E_CUDA if the stream reports an error.
 * Every op resets the word when it starts. */
int mosaic_bsa_last_status(const void *ws, void *cuda_stream);

/* Diagnostic: how many TMA descriptors the library has encoded so far in this process.  A call that
 * sees the same tensors (device, base pointers, geometry) as an earlier one encodes none. */
long long mosaic_bsa_descriptor_encodes(void);

/* Static, NUL-terminated description of a return code. */
const char *mosaic_bsa_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MOSAIC_BSA_H_ */
