/*
 * tcmoe - token-centric MoE layer for NVIDIA B200 (sm_100a): C ABI.
 *
 * The library computes one expert-parallel MoE layer as the paper states it
 * (Sec. II-A): a gate picks `topk` experts per token, Dispatch moves the token
 * to the expert groups ("GPUs" in the paper, logical partitions of one HBM
 * here) that host them, every chosen expert runs its FFN (GEMM-1, GEMM-2), and
 * Combine aggregates the `topk` outputs.  Symbols: T tokens, d hidden size,
 * f expert FFN width, E experts, k = topk, G expert groups, m = E / G experts
 * per group, P = T * k (token, expert) pairs, N_disp = number of distinct
 * (token, group) pairs.
 *
 * Conventions for every entry point
 *  - All tensor pointers are DEVICE pointers unless the name ends in `_host`.
 *    The caller owns every buffer, including the workspace; the library never
 *    allocates or frees device memory and keeps no pointer after a call.
 *  - bf16 tensors are raw 16-bit patterns, row-major, rows contiguous.  Every
 *    pointer must be 16-byte aligned; x, xg, o, y, w1, w3, w2 and the workspace
 *    128-byte aligned.
 *  - Calls only enqueue work on `stream` (a cudaStream_t passed as void*) and
 *    never synchronise, except moe_status, moe_traffic_stats and
 *    moe_profile_read (which return values to the host).  Data-dependent sizes (N_disp,
 *    counts) stay on the device.
 *  - Return value: 0 on success, a negative MOE_ERR_* when the host rejects the
 *    call (nothing is launched then).  Conditions only the device can see go
 *    to a status block at the start of the workspace, read with moe_status.
 *  - The workspace must be zero-filled once before first use (or
 *    moe_status_reset called on it).  Calls that share a workspace must be
 *    ordered on one stream.
 *  - There is no CPU fallback: without a CUDA device every compute entry point
 *    returns MOE_ERR_CUDA.
 */
#ifndef TCMOE_H_
#define TCMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = -1,        /* null pointer, bad enum, inconsistent sizes          */
  MOE_ERR_UNSUPPORTED_SHAPE = -2,  /* shape outside the limits listed at moe_shape_t      */
  MOE_ERR_WORKSPACE_TOO_SMALL = -3,
  MOE_ERR_MISALIGNED = -4,
  MOE_ERR_CUDA = -5,               /* a CUDA runtime / driver call failed (incl. no GPU)  */
  MOE_ERR_SCRATCH_LIMIT = -6,      /* moe_dispatch_noalloc: shape needs more scratch than
                                      the library's built-in array holds                  */
  /* device-side codes, reported through moe_status()[0] */
  MOE_DEV_TIMEOUT = 1,             /* a bounded wait inside a kernel expired              */
  MOE_DEV_INDEX_OUT_OF_RANGE = 2   /* an expert index outside [0, E) was read             */
};
/* bits of moe_status()[5] */
enum { MOE_WARN_NONFINITE_LOGIT = 1 };

enum { MOE_SCORE_SOFTMAX = 0,      /* weights = softmax over the k selected keys          */
       MOE_SCORE_SIGMOID = 1 };    /* weights = sigmoid(key) renormalised over the k      */
enum { MOE_FLAG_WEIGHT_IN_COMBINE = 1,   /* default (0): gate weight applied in GEMM-2's
                                            epilogue, Combine un-weighted (Sec. III-C)    */
       MOE_FLAG_COMBINE_IN_EPILOGUE = 2, /* moe_layer only: Combine runs inside GEMM-2's
                                            epilogue (Sec. IV, fused pipeline): every weighted
                                            expert row is added into an fp32 accumulator row of
                                            its token with vector reductions, o is never
                                            written, a last pass rounds the accumulators to
                                            bf16.  The k additions of a token then happen in
                                            arrival order, so y may differ from the default
                                            form in the last fp32 bit before rounding (not
                                            run-to-run reproducible).  Excludes
                                            MOE_FLAG_WEIGHT_IN_COMBINE; the stage entry points
                                            moe_expert_ffn / moe_combine reject it.        */
       MOE_FLAG_SPARSE_TOPK = 4,         /* moe_dispatch / moe_expert_ffn / moe_combine: entries
                                            of topk_idx may be -1 (slot unused).  The switch of
                                            Sec. III-D trims a replica to the targets behind its
                                            port, so a row received by an expert group carries
                                            between 1 and min(k, m) experts: this is the form of
                                            its routing table.  expert_offsets[E] is then the
                                            number of slots in use (<= T*k), pair_row is -1 for
                                            unused slots, and the per-pair arrays are filled only
                                            up to expert_offsets[E].                          */
       MOE_FLAG_SM_PARTITION = 16,       /* with MOE_FLAG_FUSED_FFN: the thread blocks are divided between the
                                            stages as in Sec. IV-C - two thirds of the SMs take only GEMM-1 tiles
                                            (their worker warps the Dispatch tasks), one third only GEMM-2 tiles
                                            (their worker warps the Combine tasks), each group paced by the tracker
                                            alone.  Same results.                                                 */
       MOE_FLAG_GEMM1_PAIR = 128,        /* moe_expert_ffn / moe_layer (bf16 experts): Dispatch writes the per-expert
                                            layout tensors of Sec. III-D (one dense row per (token, expert), expert-
                                            sorted, in the workspace) and GEMM-1 reads them as TMA tiles on CTA pairs
                                            (cta_group::2, 256-row tiles) instead of gathering token rows inside
                                            the GEMM.  Same h as the gathering form, bit for bit.  Without this flag
                                            and without MOE_FLAG_GEMM1_GATHER the library takes this form by itself
                                            for wide experts (f >= 8192, at least 512 rows per expert on average),
                                            where the extra pass over the rows costs less than it gains.  Excludes
                                            MOE_FLAG_FUSED_FFN and MOE_FLAG_GEMM1_GATHER.                              */
       MOE_FLAG_GEMM1_GATHER = 512,      /* GEMM-1 always gathers token rows itself (cta_group::1, 128-row tiles)   */
       MOE_FLAG_TRACK_DISPATCH = 256,    /* with MOE_FLAG_FUSED_FFN: Dispatch runs as tasks of the same kernel.  Worker
                                            warps write the per-expert layout tensors (Sec. III-D) 16 rows at a time and
                                            count them in the Tile Status table (DAcc, Sec. IV-B); a GEMM-1 tile starts
                                            when all rows of its 128-row tile have landed and reads them in place.
                                            Without the flag GEMM-1 gathers token rows itself and no copy is written.
                                            Same results.                                                          */
       MOE_FLAG_GEMM2_PAIR = 32,         /* GEMM-2 runs on 256-row CTA-pair tiles (cta_group::2) whatever the shape */
       MOE_FLAG_GEMM2_SINGLE = 64,       /* GEMM-2 runs on 128-row single-CTA tiles whatever the shape.  Without either
                                            flag the library picks from the shape: pair tiles unless experts hold
                                            fewer than 512 rows on average.  The two flags exclude each other; the
                                            results of both forms meet the same tolerances.               */
       MOE_FLAG_FUSED_FFN = 8 };         /* moe_expert_ffn / moe_layer (bf16 experts): the stages after the layout run
                                            as ONE persistent kernel paced by the token tracker of Sec. IV-B (tiles of
                                            128 tokens): a GEMM-2 tile starts as soon as the 128 rows of h it reads are
                                            complete (TBCnt1); in moe_layer the kernel also runs the Combine tasks - a
                                            token is combined when all of its topk rows of o are complete (TBCnt2 and
                                            the Output Readiness counter nReady), so y is produced by the same launch.
                                            Same results as the separate kernels, bit for bit.  Excludes
                                            MOE_FLAG_COMBINE_IN_EPILOGUE.  The kernel needs every thread block of its
                                            grid resident at once (one per SM): a device shared with other work may
                                            make its bounded waits expire (MOE_DEV_TIMEOUT after 2 s), never hang.   */

/* Shape of one layer.  Limits: 1 <= k <= min(E, 32); E <= 1024; E % G == 0;
 * d % 8 == 0; f % 8 == 0; T >= 0; T * max(k, G) < 2^31. */
typedef struct {
  int32_t T, d, f, E, k, G;
  int32_t score_fn;   /* MOE_SCORE_* */
  int32_t flags;      /* MOE_FLAG_*  */
} moe_shape_t;

/* Dispatch layout: the software form of the paper's per-destination AL tables
 * (Sec. III-D: algebraic index = token id -> layout index = row in a dense
 * buffer) and TID table (Sec. IV-B).  All int32 device arrays, caller-allocated.
 * Rows inside an expert / group are in ascending token order. */
typedef struct {
  int32_t* expert_counts;   /* [E]    rows per expert (the paper's nactive[expert])      */
  int32_t* expert_offsets;  /* [E+1]  exclusive prefix sum, [E] = T*k                    */
  int32_t* group_counts;    /* [G]    dispatched rows per group                          */
  int32_t* group_offsets;   /* [G+1]  exclusive prefix sum, [G] = N_disp                 */
  int32_t* pair_row;        /* [T*k]  expert-sorted row of pair p = t*k + j              */
  int32_t* row_pair;        /* [T*k]  inverse of pair_row                                */
  int32_t* al;              /* [G*T]  layout index of token t in group g, or -1          */
  int32_t* disp_token;      /* [T*min(k,G)] token of dispatched row n; first N_disp used */
  int32_t* row_src;         /* [T*k]  dispatched row feeding expert row r                */
} moe_layout_t;

/* Bytes of workspace that any entry point may need for this shape. */
int moe_workspace_bytes(const moe_shape_t* shape, size_t* bytes);

/* Zero the status block of a workspace (enqueued on `stream`). */
int moe_status_reset(void* ws, void* stream);

/* Copy the status block to the host: out[0] code (0 = ok, MOE_DEV_*), out[1]
 * where (kernel id), out[2] detail, out[3] aux, out[4] abort flag, out[5]
 * warning bits, out[6..7] reserved.  Synchronises `stream`. */
int moe_status(const void* ws, int32_t out[8], void* stream);

const char* moe_strerror(int code);

/* Gate (Sec. II-A "selected by the gate network"): logits = x * w_gate in fp32;
 * key = logit + bias (one fp32 add); the k largest keys per token, ordered by
 * (key descending, expert index ascending), the lowest index winning ties;
 * gate weights over the selected keys per shape->score_fn.
 *   x          [T, d]  bf16
 *   w_gate     [d, E]  fp32, or NULL: `logits` is then an INPUT
 *   logit_bias NULL, or fp32 [E] (bias_row_stride = 0) or [T, E] (stride = E)
 *   logits     [T, E]  fp32 out (raw, before the bias)
 *   topk_idx   [T, k]  int32 out;  topk_w [T, k] fp32 out (sums to 1 per token) */
int moe_route(const moe_shape_t* shape, const void* x, const float* w_gate,
              const float* logit_bias, int64_t bias_row_stride,
              float* logits, int32_t* topk_idx, float* topk_w,
              void* ws, size_t ws_bytes, void* stream);

/* Dispatch (Sec. II-A; Sec. III-D switch routing: group = expert / m, one
 * replica per group trimmed to that group's targets; AL management).  Builds
 * the layout from topk_idx (experts of a token must be distinct) and writes
 * one copy of x[t] per DISTINCT group the token's experts live in:
 *   xg[group_offsets[g] + al[g][t], :] = x[t, :].
 *   xg  [T*min(k,G), d] bf16 capacity; may be NULL to build the layout only. */
int moe_dispatch(const moe_shape_t* shape, const void* x, const int32_t* topk_idx,
                 const moe_layout_t* layout, void* xg,
                 void* ws, size_t ws_bytes, void* stream);

/* Expert FFN (Sec. II-A GEMM-1 / GEMM-2; Sec. III-C: gate weight in GEMM-2's
 * epilogue).  For expert e and each of its rows r (expert-sorted order):
 *   a = xg[row_src[r]];  h = silu(a W1[e]) * (a W3[e]);  o[r] = w_r * (h W2[e])
 * with w_r = topk_w[row_pair[r]] (or 1 with MOE_FLAG_WEIGHT_IN_COMBINE).
 * bf16 operands, fp32 accumulation, h and o rounded to bf16.
 *   w1, w3 [E, d, f] bf16;  w2 [E, f, d] bf16;  o [T*k, d] bf16 out. */
int moe_expert_ffn(const moe_shape_t* shape, const void* xg, const moe_layout_t* layout,
                   const float* topk_w, const void* w1, const void* w3, const void* w2,
                   void* o, void* ws, size_t ws_bytes, void* stream);

/* Combine (Sec. II-A aggregation; Sec. III-D reduction logic): for dispatched
 * row n = (t, g), pg[n] = sum of token t's expert rows that live in group g
 * (pre-reduction inside the group, ascending slot j); y[t] = sum over groups
 * (ascending g) of the partial sums; fp32 accumulation, un-permuted to token
 * order.  With MOE_FLAG_WEIGHT_IN_COMBINE rows are scaled by topk_w here.
 *   o [T*k, d] bf16;  pg NULL or [N_disp, d] bf16 out;  y [T, d] bf16 out. */
int moe_combine(const moe_shape_t* shape, const void* o, const moe_layout_t* layout,
                const int32_t* topk_idx, const float* topk_w, void* pg, void* y,
                void* ws, size_t ws_bytes, void* stream);

/* Fused layer (Sec. IV token-centric kernel fusion): gate, layout, expert FFN
 * fed straight from x (the dispatched copy is never written: the gather is
 * GEMM-1's prologue) and combine, in one call.  logits, topk_idx, topk_w and
 * layout are optional outputs (NULL: kept in the workspace). */
int moe_layer(const moe_shape_t* shape, const void* x, const float* w_gate,
              const float* logit_bias, int64_t bias_row_stride,
              const void* w1, const void* w3, const void* w2, void* y,
              float* logits, int32_t* topk_idx, float* topk_w, const moe_layout_t* layout,
              void* ws, size_t ws_bytes, void* stream);

/* moe_layer on HOST activations: copies x_host -> x_dev, runs moe_layer, copies
 * y_dev -> y_host, all enqueued on `stream` (pinned host memory makes the copies
 * asynchronous).  x_dev / y_dev are caller-owned device staging buffers
 * [T, d] bf16; weights and workspace stay on the device. */
int moe_layer_host(const moe_shape_t* shape, const void* x_host, void* x_dev, const float* w_gate,
                   const float* logit_bias, int64_t bias_row_stride,
                   const void* w1, const void* w3, const void* w2, void* y_dev, void* y_host,
                   void* ws, size_t ws_bytes, void* stream);

/* ---- backward pass ----------------------------------------------------------------------------------
 * Sec. VI-A evaluates training, forward + backward, of the layer of Sec. II-A.  For FIXED routing (expert indices
 * and gate weights as the forward produced them, held constant: the gate network's own gradient is the separate
 * call moe_gate_backward below), with dy = dL/dy:
 *     dx[t]  = sum_j w[t,j] * dFFN_e/da (x[t]) applied to dy[t]          [T, d] bf16
 *     dw1[e] = Xs_e^T dA1_e,  dw3[e] = Xs_e^T dA3_e,  dw2[e] = H_e^T dO_e   [E, d, f], [E, d, f], [E, f, d] bf16
 * where Xs_e / H_e / dO_e / dA*_e are the rows of expert e (dO = w * dy, dH = dO W2^T, dA1 = dH * a3 * silu'(a1),
 * dA3 = dH * silu(a1), a1 = x W1, a3 = x W3 recomputed).  bf16 operands, fp32 accumulation, intermediates rounded
 * to bf16.  Weight gradients are written in full (zeros for experts no token selected).
 *   x, dy       [T, d] bf16
 *   topk_idx, topk_w, layout   as written by moe_layer / moe_route + moe_dispatch for the same x
 *   w1, w3, w2  the forward weights, read in place (transposed operands are read K-major, nothing is repacked)
 *   ws          moe_backward_workspace_bytes(shape) bytes, 128-byte aligned, status block at its start (zero it
 *               once or call moe_status_reset; read with moe_status); the size includes the scratch of
 *               moe_gate_backward, which reads what this call leaves there
 * shape->flags: 0 or MOE_FLAG_SPARSE_TOPK. */
int moe_backward_workspace_bytes(const moe_shape_t* shape, size_t* bytes);
int moe_layer_backward(const moe_shape_t* shape, const void* x, const void* dy, const int32_t* topk_idx,
                       const float* topk_w, const moe_layout_t* layout, const void* w1, const void* w3, const void* w2,
                       void* dx, void* dw1, void* dw3, void* dw2, void* ws, size_t ws_bytes, void* stream);

/* Gradient of the gate network (Sec. II-A: the gate picks the topk experts of a token and weighs their outputs;
 * Sec. VI-A: training).  The SELECTION (topk_idx) is held fixed; the gate weights are differentiated as functions of
 * the router keys key[t, e] = x[t] . w_gate[:, e] + logit_bias[t, e] (softmax over the k selected keys, or sigmoid
 * renormalised over them, as shape->score_fn says).  With g[t, j] = topk_w[t, j] * dy[t] . FFN_{e_j}(x[t]):
 *     dkey[t, j] = (g[t, j] - topk_w[t, j] * sum_i g[t, i]) * c,   c = 1 (softmax) or 1 - sigmoid(key[t, j]),
 *     dw_gate[:, e] = sum over the pairs (t, j) with e_j = e of dkey[t, j] * x[t, :]        fp32 [d, E], written whole,
 *     dx[t, :]     += sum_j dkey[t, j] * w_gate[:, e_j]                                     bf16 [T, d], in / out.
 * MUST follow moe_layer_backward for the same shape, routing and backward workspace on the same stream: it reads
 * what that call leaves in `ws` (the recomputed h, dH, the per-expert rows of x and the padded row numbers) and the
 * dx it wrote.  `logits` are the forward's fp32 router logits [T, E] (moe_layer's optional output); required for
 * sigmoid scores, ignored (may be NULL) for softmax.  logit_bias / bias_row_stride as in moe_route.  `layout` is the
 * forward's layout (only expert_counts is read).  shape->flags: 0 or MOE_FLAG_SPARSE_TOPK.
 * Alignment: dx and ws 128 bytes, the other pointers 16.  Errors as moe_layer_backward; sigmoid scores without
 * logits: MOE_ERR_INVALID_ARG.  Five small launches; deterministic (each expert's rows are summed in ascending
 * order, no atomics). */
int moe_gate_backward(const moe_shape_t* shape, const float* logits, const float* logit_bias, int64_t bias_row_stride,
                      const int32_t* topk_idx, const float* topk_w, const moe_layout_t* layout, const float* w_gate,
                      void* dx, float* dw_gate, void* ws, size_t ws_bytes, void* stream);

/* ---- FP8 form of the expert FFN --------------------------------------------------------------
 * Sec. V-A evaluates the DeepSeek-V3 experts with FP8 GEMM kernels and gives no recipe; this
 * library's reading: E4M3 elements (largest finite value 448, round to nearest even, saturating),
 * one fp32 scale per activation row and one per (expert, output column) of a weight matrix,
 * scale = fl32(max|v| / 448) (1 for an all-zero vector), code = e4m3(fl32(v / scale)); fp32
 * accumulation; the scales multiply the accumulator in the epilogue; h is written as bf16 and
 * quantised per row before GEMM-2. */

/* src bf16 [rows, cols] -> dst E4M3 codes [rows, cols] (one byte each), scale fp32 [rows].
 * cols % 8 == 0; src 16-byte, dst 8-byte aligned.  Device pointers; enqueues on `stream`. */
int moe_quantize_rows(const void* src, int64_t rows, int64_t cols, void* dst, float* scale, void* stream);

/* w bf16 [E, K, N] (N contiguous, the layout moe_expert_ffn takes) -> wq E4M3 codes [E, N, K]
 * (K contiguous: the K-major operand of the FP8 GEMMs), scale fp32 [E, N].  A one-time
 * preparation of static weights. */
int moe_quantize_weights(const void* w, int32_t E, int32_t K, int32_t N, void* wq, float* scale, void* stream);

/* moe_expert_ffn on quantised operands: xq E4M3 [rows of the dispatched buffer, d] with row
 * scales sx (row r of expert e reads dispatched row layout->row_src[r]); w1q, w3q [E, f, d] with
 * s1, s3 [E, f]; w2q [E, d, f] with s2 [E, d] (all from moe_quantize_weights).  o bf16 [T*k, d] as
 * in moe_expert_ffn (gate weight in the epilogue unless MOE_FLAG_WEIGHT_IN_COMBINE).  Needs
 * d % 16 == 0 and f % 16 == 0 (MOE_ERR_UNSUPPORTED_SHAPE otherwise); the workspace holds h (bf16),
 * its E4M3 copy and its row scales. */
int moe_expert_ffn_fp8(const moe_shape_t* shape, const void* xq, const float* sx, const moe_layout_t* layout,
                       const float* topk_w, const void* w1q, const float* s1, const void* w3q, const float* s3,
                       const void* w2q, const float* s2, void* o, void* ws, size_t ws_bytes, void* stream);

/* moe_layer with FP8 experts: gate, top-k and layout on the bf16 activations as in moe_layer; x is
 * quantised per token into the workspace, GEMM-1 gathers the E4M3 rows, h is quantised per row,
 * GEMM-2 and Combine as in moe_layer.  Weights and scales as for moe_expert_ffn_fp8.  Same flags,
 * optional outputs and limits as moe_layer, plus d % 16 == 0 and f % 16 == 0. */
int moe_layer_fp8(const moe_shape_t* shape, const void* x, const float* w_gate, const float* logit_bias,
                  int64_t bias_row_stride, const void* w1q, const float* s1, const void* w3q, const float* s3,
                  const void* w2q, const float* s2, void* y, float* logits, int32_t* topk_idx, float* topk_w,
                  const moe_layout_t* layout, void* ws, size_t ws_bytes, void* stream);

/* moe_layer_fp8 on HOST activations (bf16 x_host / y_host, pinned for asynchronous copies): the
 * counterpart of moe_layer_host. */
int moe_layer_fp8_host(const moe_shape_t* shape, const void* x_host, void* x_dev, const float* w_gate,
                       const float* logit_bias, int64_t bias_row_stride, const void* w1q, const float* s1,
                       const void* w3q, const float* s3, const void* w2q, const float* s2, void* y_dev, void* y_host,
                       void* ws, size_t ws_bytes, void* stream);

/* Dispatch without a workspace (the paper has no counterpart; this entry point exists for
 * callers that cannot supply scratch memory).  Some users of this library run where device
 * memory cannot be obtained around the call: plugins that execute inside a host framework's
 * pre-planned arena, serving loops whose policy bans allocator calls (and the synchronisation
 * they imply) on the hot path, callers bound to a fixed C interface with no slot for a scratch
 * pointer.  For them this variant of moe_dispatch keeps the layout builder's scratch tables
 * (membership bitmasks, popcount prefixes, tile prefixes, status block) in one fixed device
 * array of MOE_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU that loads the
 * library holds it until the process exits.  Inputs and outputs are still the caller's.
 *  - Same arguments and results as moe_dispatch (layout arrays and, unless xg is NULL, the
 *    dispatched copy), bit for bit.  The call allocates nothing and frees nothing.
 *  - Limit: 256 + 8*(E+G)*ceil(T/32) + 8*(E+1) bytes (each table rounded up to 256) must fit in
 *    MOE_NOALLOC_SCRATCH_BYTES; larger shapes return MOE_ERR_SCRATCH_LIMIT and launch nothing.
 *  - The array used is the CURRENT device's copy (cudaGetDevice at the time of the call): `stream`
 *    and every pointer must belong to that device.
 *  - The first call on a device looks up the array's device address, which also makes the CUDA
 *    runtime load the library's device code there (an implicit allocation and synchronisation by
 *    the runtime, once); make that first call outside any stream capture.  "Allocates nothing"
 *    holds for every later call, which only enqueues work on `stream`.
 *  - All calls on a device share the array and it keeps the previous call's contents; the
 *    entry point clears what must start at zero.  Two calls that overlap on the GPU (different
 *    streams, no ordering between them) race on it: serialise them.
 *  - status_out: NULL, or 8 int32 on the device that receive the status block of this call
 *    (same slots as moe_status) once the work has run. */
#define MOE_NOALLOC_SCRATCH_BYTES (2u << 20)
int moe_dispatch_noalloc(const moe_shape_t* shape, const void* x, const int32_t* topk_idx,
                         const moe_layout_t* layout, void* xg, int32_t* status_out, void* stream);

/* Byte offsets of named regions inside the workspace, for tests and profilers:
 * out[0] status, out[1] h (GEMM-1 output [T*k, f] bf16), out[2] o scratch used
 * by moe_layer, out[3] expert m-tile prefix [E+1] int32. */
int moe_workspace_layout(const moe_shape_t* shape, size_t out[4]);

/* Kernel ids for moe_profile_enable (also the `where` slot of moe_status). */
enum { MOE_KERNEL_TOPK = 1, MOE_KERNEL_MASKS = 2, MOE_KERNEL_FILL = 3, MOE_KERNEL_DISPATCH = 4,
       MOE_KERNEL_GEMM1 = 5, MOE_KERNEL_GEMM2 = 6, MOE_KERNEL_COMBINE = 7, MOE_KERNEL_GATE = 8,
       MOE_KERNEL_WGRAD = 10, MOE_KERNEL_BWD_GATHER = 11, MOE_KERNEL_GATE_BWD = 12 };

/* Per-kernel timing hook for benchmarks (host-side state, one record per process, guarded by a
 * mutex so that launches from several host threads are safe; not part of the method).  After moe_profile_enable(id) every launch of that kernel by any entry point is
 * bracketed by a pair of CUDA events on the launching stream (up to 4096 launches; later ones
 * are not recorded).  moe_profile_read waits for the recorded events, returns the summed
 * device time in milliseconds and the number of launches, and clears the record.
 * moe_profile_enable(0) switches the hook off. */
int moe_profile_enable(int kernel_id);
int moe_profile_read(float* total_ms, int32_t* launches);

/* ---- expert parallelism across GPUs (group g = GPU g) -------------------------------------------
 * The dispatched buffer xg of moe_dispatch is what travels out (segment g to GPU g: one row per
 * distinct (token, group), Sec. III-D) and one pre-reduced row per (token, group) travels back.
 * The exchange itself (an all-to-all with the segment sizes group_counts) is the caller's; these
 * two entry points are the steps expert parallelism adds on either side of it.
 *
 * moe_ep_pack: the trimmed target list of every dispatched row (Sec. III-D: a replica is trimmed
 * to the targets behind its port).  For row n = (t, g), in ascending slot order:
 *   send_idx[n, 0..kk)  the experts of token t that live in group g, as indices LOCAL to the group
 *                       (e - g*m), -1 for unused entries;   kk = min(k, m)
 *   send_w  [n, 0..kk)  their gate weights, 0 for unused entries
 * Both [T*min(k,G), kk]; segment g of them travels with segment g of xg.  On the receiving GPU the
 * rows, send_idx and send_w of all senders, concatenated, are x, topk_idx and topk_w of a layer with
 * shape {T = rows received, E = m, k = kk, G = 1, MOE_FLAG_SPARSE_TOPK}: moe_dispatch (xg = NULL)
 * builds its layout, moe_expert_ffn runs the local experts on the received rows (row_src is the
 * identity there), moe_combine sums each received row's outputs - the pre-reduced row that goes back. */
int moe_ep_pack(const moe_shape_t* shape, const int32_t* topk_idx, const float* topk_w,
                const moe_layout_t* layout, int32_t* send_idx, float* send_w, void* stream);

/* moe_ep_finish: back [N_disp, d] bf16 holds, in the order of xg, the pre-reduced rows returned by the
 * GPUs;  y[t] = sum over the groups g that token t touched of back[group_offsets[g] + al[g][t]]
 * (fp32, ascending g), bf16 out [T, d]. */
int moe_ep_finish(const moe_shape_t* shape, const void* back, const moe_layout_t* layout, void* y, void* stream);

/* Traffic figures of Sec. II-B / II-C for the routing held in `layout` (a filled dispatch layout
 * of `shape`), with the G expert groups read as the G GPUs of an expert-parallel node:
 *   out[0] T   out[1] P = T*k   out[2] N_disp (distinct (token, group) pairs)
 *   out[3] D = N_disp / T, the mean number of distinct destinations of a token
 *   out[4] 1 - N_disp / P: share of the point-to-point Dispatch copies that one-copy-per-group
 *          (in-switch multicast) removes; the same share of Combine rows is removed by the in-group
 *          pre-reduction
 *   out[5] (G - D) / D: useless traffic when Dispatch / Combine are emulated by AllGather /
 *          Reduce-Scatter (the paper's "340 %" for DeepSeek-V3 on 32 GPUs)
 *   out[6] (D - 1) / (2 D): redundant share of the source <-> switch traffic ("nearly 50 %")
 *   out[7] 2 D / (1 + D): ideal communication speed-up ("near 2x")
 * Reads one int32 from the device and synchronises `stream`.  T = 0 gives zeros. */
int moe_traffic_stats(const moe_shape_t* shape, const moe_layout_t* layout, double out[8], void* stream);

/* Payload efficiency of one multi-destination transfer under the packet formats of Sec. III-A / III-B
 * (efficiency = data flits / all transmitted flits, Sec. VI-B).  Host arithmetic only: no device is touched.
 * What the paper fixes: 16-byte flits; flit0 holds the single multimem address, a stage bit and the target
 * count; target-extension flits hold eight 16-bit expert ids each; explicit addressing needs one destination
 * flit per target in the request and as many in the response, which for eight targets lowers an ideal 80 % to
 * 69 %.  What it leaves open and this library reads as: packets carry at most 256 bytes (16 data flits) and
 * cost 4 further flits over request and response (the share that makes plain transfers 80 % efficient), and
 * the destination / target flits are paid once per transfer.  The printed pair 80 % / 69 % is reproduced at
 * transfer_bytes = 1280, n_targets = 8.
 *   out[0] data flits = ceil(transfer_bytes / 16)
 *   out[1] ideal efficiency (headers of plain packets only)
 *   out[2] explicit addressing: + 2 * n_targets flits
 *   out[3] dynamic multimem addressing: + ceil(n_targets / 8) flits
 * transfer_bytes >= 1, 0 <= n_targets < 2^15 (the 15-bit target count), else MOE_ERR_INVALID_ARG. */
int moe_payload_efficiency(int64_t transfer_bytes, int32_t n_targets, double out[4]);

/* Self-test of the bounded waits every kernel of the library relies on (the paper's runtime polls
 * without a bound, Sec. IV-C; here a wait that outlives its budget ends the kernel with a status
 * instead of hanging the GPU).  Launches one small kernel that waits, with a budget of `limit_ns`
 * nanoseconds (1 us .. 100 ms), on a shared-memory barrier that nothing ever signals, with the
 * same wait routine the GEMM kernels use.  The wait gives up, the kernel records
 * {MOE_DEV_TIMEOUT, where = MOE_KERNEL_SELFTEST, detail = waited microseconds} in the status block
 * at `ws` (as every kernel does), sets the abort word and returns normally: the context stays
 * usable.  moe_status_reset() clears the status afterwards.  Returns MOE_OK once the kernel is
 * enqueued; read the outcome with moe_status(). */
enum { MOE_KERNEL_SELFTEST = 9 };
int moe_selftest_wait_timeout(void* ws, uint64_t limit_ns, void* stream);

/* TMA descriptors.  The tcgen05 kernels read their operands through TMA tensor maps, which are a function of an
 * operand's address, extents and strides only (not of its contents).  The library keeps the 64 most recent maps,
 * keyed by every argument of the encode, so that a layer called again on the same weights and workspace does not
 * encode them again; a buffer freed and reallocated at the same address with the same shape gets the same (still
 * correct) map.  moe_clear_cache forgets them all (host memory only; nothing on the device).  Thread-safe.
 * Returns MOE_OK. */
int moe_clear_cache(void);

#ifdef __cplusplus
}
#endif
#endif /* TCMOE_H_ */
