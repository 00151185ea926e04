// Internal declarations shared by the tcmoe translation units (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <utility>

namespace tcmoe {

// ---- status block at the start of the workspace (16 x int32) --------------------------------
enum StatusSlot { ST_CODE = 0, ST_WHERE = 1, ST_DETAIL = 2, ST_AUX = 3, ST_ABORT = 4, ST_WARN = 5 };
enum KernelId { KID_TOPK = 1, KID_MASKS = 2, KID_FILL = 3, KID_DISPATCH = 4, KID_GEMM1 = 5, KID_GEMM2 = 6,
                KID_COMBINE = 7, KID_GATE = 8, KID_SELFTEST = 9, KID_WGRAD = 10, KID_BWD = 11, KID_GATE_BWD = 12 };
constexpr int DEV_TIMEOUT = 1;
constexpr int DEV_INDEX_OUT_OF_RANGE = 2;
constexpr int WARN_NONFINITE_LOGIT = 1;

__device__ __forceinline__ void report_error(int32_t* status, int code, int where, int detail, int aux) {
  if (atomicCAS(&status[ST_CODE], 0, code) == 0) {
    status[ST_WHERE] = where;
    status[ST_DETAIL] = detail;
    status[ST_AUX] = aux;
  }
}

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialisation and starts with
// grid_dependency_sync(): set-up that touches no global data (barrier init, TMEM allocation,
// tensor-map prefetch) may run while the previous kernel of the stream drains; nothing is read
// from or written to global memory before the previous kernel has completed and flushed, so
// results are those of plain stream order.  The call also lets the next kernel of the stream
// begin its own set-up.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// ---- problem description passed to the launchers ---------------------------------------------
struct Shape {
  int T, d, f, E, k, G, score_fn, flags;
};

struct Layout {
  int32_t *expert_counts, *expert_offsets, *group_counts, *group_offsets, *pair_row, *row_pair, *al,
      *disp_token, *row_src;
};

// Arguments of the Combine stage (the combine kernel and the Combine tasks of the tracker-paced kernel).
struct CombineArgs {
  const uint4* o;                 // [P, d] bf16 expert-sorted rows
  uint4* y;                       // [T, d] bf16 out
  uint4* pg;                      // NULL or [N_disp, d] bf16 out (group partial sums)
  const int32_t* topk_idx;        // [T, k]
  const float* topk_w;            // [T, k] (read only when weighted)
  const int32_t* pair_row;        // [T, k]
  const int32_t* al;              // [G, T]
  const int32_t* group_offsets;   // [G + 1]
  int T, E, k, m, vec_per_row, weighted, n_rows;
  int32_t* status;
};

// Scratch tables of the layout builder (inside the workspace).
struct LayoutScratch {
  uint32_t* emask;    // [E, W] bit t%32 of word t/32: token t selected expert e
  uint32_t* gmask;    // [G, W] token t touches group g
  int32_t* eprefix;   // [E, W] exclusive popcount prefix along the row
  int32_t* gprefix;   // [G, W]
  int32_t* mt_prefix; // [E+1]  exclusive prefix of 128-row tiles per expert (GEMM-1 tasks)
  int32_t* mp_prefix; // [E+1]  exclusive prefix of 256-row CTA-pair tiles per expert (GEMM-2 tasks)
  int W;
};

// gate_gemm.cu: wsplit is scratch of gate_split_bytes(d, E) bytes for the bf16 hi/mid/lo terms of w_gate
size_t gate_split_bytes(int d, int E);
cudaError_t launch_gate_logits(const Shape& s, const void* x, const float* w_gate, float* logits, void* wsplit,
                               int32_t* status, cudaStream_t st);
// route.cu
cudaError_t launch_topk(const Shape& s, const float* logits, const float* bias, int64_t bias_stride,
                        int32_t* topk_idx, float* topk_w, int32_t* status, cudaStream_t st,
                        uint32_t* clear = nullptr, size_t clear_words = 0);   // clear: words zeroed on the side
// layout.cu
cudaError_t launch_layout(const Shape& s, const int32_t* topk_idx, const Layout& L, const LayoutScratch& sc,
                          int32_t* status, cudaStream_t st, bool masks_cleared = false);
cudaError_t launch_tile_prefix(const Shape& s, const int32_t* expert_counts, int32_t* mt_prefix, int32_t* mp_prefix,
                               cudaStream_t st);
cudaError_t launch_dispatch(const Shape& s, const void* x, const Layout& L, void* xg, cudaStream_t st);
cudaError_t launch_permute_rows(const Shape& s, const void* src, int src_rows, const int32_t* gather_idx,
                                int gather_div, const int32_t* expert_offsets, void* xs, int32_t* status,
                                cudaStream_t st);
cudaError_t launch_round_rows(const Shape& s, const float* acc, void* y, cudaStream_t st);
cudaError_t launch_combine(const Shape& s, const void* o, const Layout& L, const int32_t* topk_idx,
                           const float* topk_w, void* pg, void* y, int32_t* status, cudaStream_t st);
cudaError_t launch_combine_rows(const Shape& s, const void* o, const Layout& L, const int32_t* topk_idx,
                                const float* topk_w, void* pg, void* y, int n_rows, int32_t* status, cudaStream_t st);
// bwd.cu: backward pass of the layer for fixed routing
struct BwdArgs {
  const void *x, *dy;               // [T, d] bf16
  const int32_t* topk_idx;          // [T, k]
  const float* topk_w;              // [T, k]
  Layout L;                         // the forward layout
  const void *w1, *w3, *w2;         // forward weights
  void *dx, *dw1, *dw3, *dw2;       // outputs
  // scratch (padded row space: bwd_row_capacity() rows each)
  int32_t *poff, *mt_prefix, *mp_prefix, *pair_prow;
  void *xs, *dos, *dh, *h, *da1, *da3, *dxs;
  int32_t* status;
};
size_t bwd_row_capacity(const Shape& s);
cudaError_t launch_layer_backward(const Shape& s, const BwdArgs& a, cudaStream_t st);
// gate_bwd.cu: gradient of the gate network, after launch_layer_backward on the same scratch
struct GateBwdArgs {
  const int32_t* topk_idx;          // [T, k]
  const float* topk_w;              // [T, k]
  const int32_t* expert_counts;     // [E] (the forward layout)
  const float* logits;              // [T, E] fp32 router logits of the forward (sigmoid scores only, else may be NULL)
  const float* bias;                // NULL, [E] (stride 0) or [T, E] (stride E)
  int64_t bias_stride;
  const float* w_gate;              // [d, E] fp32
  void* dx;                         // [T, d] bf16, in / out: the gate path is added
  float* dw_gate;                   // [d, E] fp32 out
  // left behind by launch_layer_backward
  const int32_t *poff, *pair_prow;
  const void *xs, *h, *dh;
  // scratch
  float *g_row, *dkey, *wgt;        // [bwd_row_capacity], [T * k], [E, d]
};
cudaError_t launch_gate_backward(const Shape& s, const GateBwdArgs& a, cudaStream_t st);
// ffn.cu
struct FfnArgs {
  const void* a_src;          // GEMM-1 activations: xg (gather_div = 1) or x (gather_div = k)
  int a_rows;                 // rows of a_src (gather indices are checked against it)
  const int32_t* gather_idx;  // row_src, or row_pair (token = row_pair / k)
  int gather_div;
  const void *w1, *w3, *w2;
  void* xs;                   // [P, d] bf16 scratch: expert-sorted activation rows (CTA-pair GEMM-1), or NULL
  bool pair_gemm1;            // GEMM-1 on CTA pairs from xs (the caller's flag or the shape rule)
  void* h;                    // [P, f] bf16 scratch
  void* o;                    // [P, d] bf16 out (unused when y_acc is set)
  float* y_acc;               // Combine in GEMM-2's epilogue: zeroed fp32 [T, d] accumulator, else NULL
  const float* topk_w;        // NULL: un-weighted epilogue
  const int32_t* row_pair;
  const int32_t* expert_offsets;
  const int32_t* mt_prefix;   // 128-row tiles per expert, exclusive prefix
  const int32_t* mp_prefix;   // 256-row pair tiles per expert, exclusive prefix
  // single-kernel FFN (MOE_FLAG_FUSED_FFN): task tables and the tile tracker, scratch in the workspace
  const int32_t* expert_counts;
  int32_t* blk_start;
  void* blk_info;
  int32_t* n_blocks;
  int32_t* tracker;           // fused_tracker_words() int32 words
  CombineArgs comb;           // comb.y != NULL: the kernel also runs the Combine tasks (moe_layer)
  bool track_dispatch;        // Dispatch tasks write xs inside the kernel, GEMM-1 waits for them (needs xs)
  int32_t* status;
};
size_t fused_table_blocks(const Shape& s);   // task-block capacity for a shape (ffn_fused.cu)
size_t fused_tracker_bytes(const Shape& s);  // bytes of the tracker tables for a shape
namespace ffn {
void clear_map_cache();                      // forget the cached TMA tensor maps (ffn.cu)
}
cudaError_t launch_expert_ffn(const Shape& s, const FfnArgs& a, cudaStream_t st);
// FP8 form of the expert FFN: a.a_src / a.w1 / a.w3 / a.w2 hold E4M3 codes (weights [E, N, K]).
struct Fp8Args {
  const float* sx;            // per source row of a.a_src
  const float *s1, *s3, *s2;  // per (expert, output column)
  void* hq;                   // [P, f] E4M3 scratch
  float* sh;                  // [P] scratch: row scales of h
};
cudaError_t launch_expert_ffn_fp8(const Shape& s, const FfnArgs& a, const Fp8Args& q, cudaStream_t st);
// ep.cu: the two steps that expert parallelism across GPUs adds to the single-GPU path
cudaError_t launch_ep_pack(const Shape& s, const int32_t* topk_idx, const float* topk_w, const Layout& L,
                           int32_t* send_idx, float* send_w, cudaStream_t st);
cudaError_t launch_ep_finish(const Shape& s, const void* back, const Layout& L, void* y, cudaStream_t st);
// quant.cu: bf16 -> E4M3 with one scale per row / per (expert, output column)
cudaError_t launch_quantize_rows(const void* src, long long rows, int cols, void* dst, float* scale, cudaStream_t st);
cudaError_t launch_quantize_weights(const void* w, int E, int K, int N, void* wq, float* scale, cudaStream_t st);
int sm_count();
int current_device();   // index of the current CUDA device, clamped to [0, MAX_DEVICES)
constexpr int MAX_DEVICES = 64;   // per-device caches (kernel attributes, SM counts) are arrays of this size

// Optional event bracket around launches of one kernel id (see moe_profile_enable).
struct ProfileScope {
  ProfileScope(int kernel_id, cudaStream_t st);
  ~ProfileScope();
  int slot;
  cudaStream_t st;
};

}  // namespace tcmoe
