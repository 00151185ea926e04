// C ABI of the library: argument checks, workspace carving, stage sequencing.
#include "../../include/tcmoe.h"

#include "common.cuh"
#include "ptx.cuh"

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

namespace tcmoe {
namespace {

constexpr size_t ALIGN = 1024;
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Regions of the workspace, in order.  Every region starts on a 1 KiB boundary.
struct WsPlan {
  size_t status, emask, gmask, eprefix, gprefix, mt_prefix, mp_prefix, blk_start, blk_info, n_blocks, tracker, wsplit, xs, h, hq, sh, xq, sx, o, logits, topk_idx, topk_w;
  size_t expert_counts, expert_offsets, group_counts, group_offsets, pair_row, row_pair, al, disp_token, row_src;
  size_t total;
  int W;
};

// GEMM-1 form.  The CTA-pair form needs the per-expert layout tensors (one more pass over P rows of d) and runs
// GEMM-1 about 8 % faster; the pass costs about 240 / f of GEMM-1's time, so it pays for wide experts.  Taken when asked
// for (MOE_FLAG_GEMM1_PAIR), or by itself for f >= 8192 with experts of at least 512 rows on average (measured: the
// Mixtral-shaped layer gains 3 %, f = 1536 and f = 2048 layers lose 1-6 %); MOE_FLAG_GEMM1_GATHER keeps the gathering
// form.  bf16 experts outside the tracker-paced kernel only.
bool pair_gemm1(const moe_shape_t& s) {
  if (s.flags & (MOE_FLAG_FUSED_FFN | MOE_FLAG_GEMM1_GATHER)) return false;
  if (s.flags & MOE_FLAG_GEMM1_PAIR) return true;
  return s.f >= 8192 && (long long)s.T * s.k >= 512ll * s.E;
}

WsPlan plan(const moe_shape_t& s) {
  WsPlan p{};
  const size_t T = (size_t)s.T, E = (size_t)s.E, G = (size_t)s.G, k = (size_t)s.k;
  const size_t P = T * k;
  const size_t W = (T + 31) / 32;
  const size_t kg = k < G ? k : G;
  p.W = (int)W;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = round_up(off + bytes, ALIGN);
    return at;
  };
  p.status = take(64);
  p.emask = off;  // emask and gmask must be adjacent (one memset clears both)
  off += E * W * 4;
  p.gmask = off;
  off = round_up(off + G * W * 4, ALIGN);
  p.eprefix = take(E * W * 4);
  p.gprefix = take(G * W * 4);
  p.mt_prefix = take((E + 1) * 4);
  p.mp_prefix = take((E + 1) * 4);
  {   // single-kernel FFN: task tables and tile tracker
    const size_t nbmax = fused_table_blocks(Shape{s.T, s.d, s.f, s.E, s.k, s.G, s.score_fn, s.flags});
    p.blk_start = take(3 * (nbmax + 1) * 4);   // interleaved | GEMM-1 only | GEMM-2 only
    p.blk_info = take(3 * (nbmax + 1) * 16);
    p.n_blocks = take(3 * 4);
    p.tracker = take(fused_tracker_bytes(Shape{s.T, s.d, s.f, s.E, s.k, s.G, s.score_fn, s.flags}));
  }
  p.wsplit = take(gate_split_bytes(s.d, s.E));
  // expert-sorted activation rows of the CTA-pair GEMM-1 (only reserved when that form is asked for)
  p.xs = take((pair_gemm1(s) || (s.flags & MOE_FLAG_TRACK_DISPATCH)) ? P * (size_t)s.d * 2 : 0);
  p.h = take(P * (size_t)s.f * 2);
  p.hq = take(P * (size_t)s.f);   // FP8 form: E4M3 copy of h and its row scales
  p.sh = take(P * 4);
  p.xq = take(T * (size_t)s.d);   // FP8 layer: E4M3 copy of x and its row scales
  p.sx = take(T * 4);
  // o [P, d] bf16, or the fp32 token accumulators [T, d] of the Combine-in-epilogue form
  p.o = take((P * 2 > T * 4 ? P * 2 : T * 4) * (size_t)s.d);
  p.logits = take(T * E * 4);
  p.topk_idx = take(P * 4);
  p.topk_w = take(P * 4);
  p.expert_counts = take(E * 4);
  p.expert_offsets = take((E + 1) * 4);
  p.group_counts = take(G * 4);
  p.group_offsets = take((G + 1) * 4);
  p.pair_row = take(P * 4);
  p.row_pair = take(P * 4);
  p.al = take(G * T * 4);
  p.disp_token = take(T * kg * 4);
  p.row_src = take(P * 4);
  p.total = off;
  return p;
}

int check_shape(const moe_shape_t* s) {
  if (s == nullptr) return MOE_ERR_INVALID_ARG;
  if (s->T < 0 || s->d <= 0 || s->f <= 0 || s->E <= 0 || s->k <= 0 || s->G <= 0) return MOE_ERR_INVALID_ARG;
  if (s->score_fn != MOE_SCORE_SOFTMAX && s->score_fn != MOE_SCORE_SIGMOID) return MOE_ERR_INVALID_ARG;
  if (s->flags & ~(MOE_FLAG_WEIGHT_IN_COMBINE | MOE_FLAG_COMBINE_IN_EPILOGUE | MOE_FLAG_SPARSE_TOPK | MOE_FLAG_FUSED_FFN |
                   MOE_FLAG_SM_PARTITION | MOE_FLAG_GEMM2_PAIR | MOE_FLAG_GEMM2_SINGLE | MOE_FLAG_GEMM1_PAIR | MOE_FLAG_TRACK_DISPATCH |
                   MOE_FLAG_GEMM1_GATHER))
    return MOE_ERR_INVALID_ARG;
  if ((s->flags & MOE_FLAG_GEMM2_PAIR) && (s->flags & MOE_FLAG_GEMM2_SINGLE)) return MOE_ERR_INVALID_ARG;
  if ((s->flags & MOE_FLAG_GEMM1_PAIR) && (s->flags & (MOE_FLAG_FUSED_FFN | MOE_FLAG_GEMM1_GATHER))) return MOE_ERR_INVALID_ARG;
  if ((s->flags & MOE_FLAG_SM_PARTITION) && !(s->flags & MOE_FLAG_FUSED_FFN)) return MOE_ERR_INVALID_ARG;
  if ((s->flags & MOE_FLAG_TRACK_DISPATCH) && !(s->flags & MOE_FLAG_FUSED_FFN)) return MOE_ERR_INVALID_ARG;
  if ((s->flags & MOE_FLAG_FUSED_FFN) && (s->flags & MOE_FLAG_COMBINE_IN_EPILOGUE)) return MOE_ERR_INVALID_ARG;
  if ((s->flags & MOE_FLAG_WEIGHT_IN_COMBINE) && (s->flags & MOE_FLAG_COMBINE_IN_EPILOGUE)) return MOE_ERR_INVALID_ARG;
  if (s->k > s->E || s->G > s->E || s->E % s->G != 0) return MOE_ERR_INVALID_ARG;
  if (s->k > 32 || s->E > 1024 || s->d % 8 != 0 || s->f % 8 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;
  const long long kg = s->k > s->G ? s->k : s->G;
  if ((long long)s->T * kg >= (1ll << 31)) return MOE_ERR_UNSUPPORTED_SHAPE;
  return MOE_OK;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_ws(const moe_shape_t* s, const void* ws, size_t ws_bytes, WsPlan* out) {
  if (ws == nullptr) return MOE_ERR_INVALID_ARG;
  if (!aligned(ws, 128)) return MOE_ERR_MISALIGNED;
  *out = plan(*s);
  if (ws_bytes < out->total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  return MOE_OK;
}

int check_layout(const moe_layout_t* L) {
  if (L == nullptr) return MOE_ERR_INVALID_ARG;
  const void* ptrs[9] = {L->expert_counts, L->expert_offsets, L->group_counts, L->group_offsets, L->pair_row,
                         L->row_pair,      L->al,             L->disp_token,   L->row_src};
  for (const void* p : ptrs) {
    if (p == nullptr) return MOE_ERR_INVALID_ARG;
    if (!aligned(p, 16)) return MOE_ERR_MISALIGNED;
  }
  return MOE_OK;
}

Shape to_shape(const moe_shape_t& s) { return Shape{s.T, s.d, s.f, s.E, s.k, s.G, s.score_fn, s.flags}; }
Layout to_layout(const moe_layout_t& L) {
  return Layout{L.expert_counts, L.expert_offsets, L.group_counts, L.group_offsets, L.pair_row,
                L.row_pair,      L.al,             L.disp_token,   L.row_src};
}
template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<uint8_t*>(ws) + off); }

LayoutScratch scratch(void* ws, const WsPlan& p) {
  LayoutScratch sc;
  sc.emask = at<uint32_t>(ws, p.emask);
  sc.gmask = at<uint32_t>(ws, p.gmask);
  sc.eprefix = at<int32_t>(ws, p.eprefix);
  sc.gprefix = at<int32_t>(ws, p.gprefix);
  sc.mt_prefix = at<int32_t>(ws, p.mt_prefix);
  sc.mp_prefix = at<int32_t>(ws, p.mp_prefix);
  sc.W = p.W;
  return sc;
}

bool have_device() {
  int n = 0;
  return cudaGetDeviceCount(&n) == cudaSuccess && n > 0;
}

#define TCMOE_CUDA(expr)                     \
  do {                                       \
    if ((expr) != cudaSuccess) {             \
      (void)cudaGetLastError();              \
      return MOE_ERR_CUDA;                   \
    }                                        \
  } while (0)

}  // namespace
}  // namespace tcmoe

namespace tcmoe {
namespace {
// State of the timing hook.  One record per process, guarded by a mutex: launches from several host threads
// may be bracketed while another thread enables, disables or reads the hook.
constexpr int PROFILE_CAP = 4096;
std::mutex g_profile_mutex;
std::atomic<int> g_profile_id{0};   // read without the lock on the launch path when the hook is off
int g_profile_n = 0;
cudaEvent_t g_ev0[PROFILE_CAP], g_ev1[PROFILE_CAP];
int g_events_made = 0;
}  // namespace

ProfileScope::ProfileScope(int kernel_id, cudaStream_t s) : slot(-1), st(s) {
  if (g_profile_id.load(std::memory_order_relaxed) != kernel_id || kernel_id == 0) return;
  std::lock_guard<std::mutex> lock(g_profile_mutex);
  if (g_profile_id.load(std::memory_order_relaxed) != kernel_id || g_profile_n >= PROFILE_CAP) return;
  while (g_events_made <= g_profile_n) {
    if (cudaEventCreate(&g_ev0[g_events_made]) != cudaSuccess || cudaEventCreate(&g_ev1[g_events_made]) != cudaSuccess)
      return;
    ++g_events_made;
  }
  slot = g_profile_n++;
  cudaEventRecord(g_ev0[slot], st);
}
ProfileScope::~ProfileScope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lock(g_profile_mutex);
  cudaEventRecord(g_ev1[slot], st);
}
}  // namespace tcmoe

namespace tcmoe {
namespace {
// One thread waits on a barrier nobody signals; the bounded wait gives up after `limit_ns`.
__global__ void selftest_wait_kernel(int32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_s;
  grid_dependency_sync();
  if (threadIdx.x == 0) {
    abort_s = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_mbar_init();
    const uint64_t t0 = ptx::globaltimer_ns();
    volatile int* abort_flag = &abort_s;
    const bool ok = ptx::mbar_wait<false, 0>(ptx::smem_u32(&bar), 0, abort_flag, abort_flag, limit_ns);
    if (!ok) {
      report_error(status, DEV_TIMEOUT, 9, (int)((ptx::globaltimer_ns() - t0) / 1000), blockIdx.x);
      status[ST_ABORT] = 1;
    }
  }
}
}  // namespace
}  // namespace tcmoe

using namespace tcmoe;

extern "C" {

int moe_ep_pack(const moe_shape_t* shape, const int32_t* topk_idx, const float* topk_w, const moe_layout_t* layout,
                int32_t* send_idx, float* send_w, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (topk_idx == nullptr || topk_w == nullptr || send_idx == nullptr || send_w == nullptr) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(topk_idx, 16) || !aligned(topk_w, 16) || !aligned(send_idx, 16) || !aligned(send_w, 16))
    return MOE_ERR_MISALIGNED;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(launch_ep_pack(to_shape(*shape), topk_idx, topk_w, to_layout(*layout), send_idx, send_w,
                            static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_ep_finish(const moe_shape_t* shape, const void* back, const moe_layout_t* layout, void* y, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (back == nullptr || y == nullptr) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(back, 128) || !aligned(y, 128)) return MOE_ERR_MISALIGNED;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(launch_ep_finish(to_shape(*shape), back, to_layout(*layout), y, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_traffic_stats(const moe_shape_t* shape, const moe_layout_t* layout, double out[8], void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (out == nullptr) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  for (int i = 0; i < 8; ++i) out[i] = 0.0;
  if (shape->T == 0) return MOE_OK;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t n_disp = 0;
  TCMOE_CUDA(cudaMemcpyAsync(&n_disp, layout->group_offsets + shape->G, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  TCMOE_CUDA(cudaStreamSynchronize(st));
  const double T = shape->T, P = (double)shape->T * shape->k, G = shape->G, N = n_disp;
  const double D = N / T;
  out[0] = T;
  out[1] = P;
  out[2] = N;
  out[3] = D;
  out[4] = 1.0 - N / P;
  if (D > 0.0) {
    out[5] = (G - D) / D;
    out[6] = (D - 1.0) / (2.0 * D);
    out[7] = 2.0 * D / (1.0 + D);
  }
  return MOE_OK;
}

int moe_payload_efficiency(int64_t transfer_bytes, int32_t n_targets, double out[4]) {
  if (out == nullptr || transfer_bytes < 1 || n_targets < 0 || n_targets >= (1 << 15)) return MOE_ERR_INVALID_ARG;
  constexpr int64_t kFlit = 16, kPacketData = 16, kPacketOverhead = 4, kIdsPerFlit = 8;
  const int64_t data = (transfer_bytes + kFlit - 1) / kFlit;
  const int64_t packets = (data + kPacketData - 1) / kPacketData;
  const int64_t base = data + packets * kPacketOverhead;
  out[0] = (double)data;
  out[1] = (double)data / (double)base;
  out[2] = (double)data / (double)(base + 2 * (int64_t)n_targets);
  out[3] = (double)data / (double)(base + ((int64_t)n_targets + kIdsPerFlit - 1) / kIdsPerFlit);
  return MOE_OK;
}

int moe_selftest_wait_timeout(void* ws, uint64_t limit_ns, void* stream) {
  if (ws == nullptr) return MOE_ERR_INVALID_ARG;
  if (limit_ns < 1000ull || limit_ns > 100000000ull) return MOE_ERR_INVALID_ARG;
  if (!aligned(ws, 128)) return MOE_ERR_MISALIGNED;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(launch_pdl(selftest_wait_kernel, 1, 32, 0, static_cast<cudaStream_t>(stream), static_cast<int32_t*>(ws),
                        (unsigned long long)limit_ns));
  return MOE_OK;
}

int moe_profile_enable(int kernel_id) {
  if (kernel_id < 0 || kernel_id > 12) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_profile_mutex);
  g_profile_id.store(kernel_id, std::memory_order_relaxed);
  g_profile_n = 0;
  return MOE_OK;
}

int moe_clear_cache(void) {
  tcmoe::ffn::clear_map_cache();
  return MOE_OK;
}

int moe_profile_read(float* total_ms, int32_t* launches) {
  if (total_ms == nullptr || launches == nullptr) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_profile_mutex);
  float sum = 0.f;
  for (int i = 0; i < g_profile_n; ++i) {
    float ms = 0.f;
    TCMOE_CUDA(cudaEventSynchronize(g_ev1[i]));
    TCMOE_CUDA(cudaEventElapsedTime(&ms, g_ev0[i], g_ev1[i]));
    sum += ms;
  }
  *total_ms = sum;
  *launches = g_profile_n;
  g_profile_n = 0;
  return MOE_OK;
}


int moe_workspace_bytes(const moe_shape_t* shape, size_t* bytes) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (bytes == nullptr) return MOE_ERR_INVALID_ARG;
  *bytes = plan(*shape).total;
  return MOE_OK;
}

int moe_workspace_layout(const moe_shape_t* shape, size_t out[4]) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (out == nullptr) return MOE_ERR_INVALID_ARG;
  const WsPlan p = plan(*shape);
  out[0] = p.status;
  out[1] = p.h;
  out[2] = p.o;
  out[3] = p.mt_prefix;
  return MOE_OK;
}

int moe_status_reset(void* ws, void* stream) {
  if (ws == nullptr) return MOE_ERR_INVALID_ARG;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(cudaMemsetAsync(ws, 0, 64, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_status(const void* ws, int32_t out[8], void* stream) {
  if (ws == nullptr || out == nullptr) return MOE_ERR_INVALID_ARG;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  TCMOE_CUDA(cudaMemcpyAsync(out, ws, 8 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  TCMOE_CUDA(cudaStreamSynchronize(st));
  return MOE_OK;
}

const char* moe_strerror(int code) {
  switch (code) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case MOE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MOE_ERR_MISALIGNED: return "misaligned pointer";
    case MOE_ERR_CUDA: return "CUDA error (or no CUDA device)";
    case MOE_ERR_SCRATCH_LIMIT: return "shape needs more scratch than the built-in no-allocation array holds";
    case MOE_DEV_TIMEOUT: return "device: bounded wait expired";
    case MOE_DEV_INDEX_OUT_OF_RANGE: return "device: expert index out of range";
    default: return "unknown code";
  }
}

int moe_route(const moe_shape_t* shape, const void* x, const float* w_gate, const float* logit_bias,
              int64_t bias_row_stride, float* logits, int32_t* topk_idx, float* topk_w, void* ws, size_t ws_bytes,
              void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (logits == nullptr || topk_idx == nullptr || topk_w == nullptr) return MOE_ERR_INVALID_ARG;
  if (w_gate != nullptr && x == nullptr) return MOE_ERR_INVALID_ARG;
  if (bias_row_stride != 0 && bias_row_stride != shape->E) return MOE_ERR_INVALID_ARG;
  if (!aligned(x, 128) || !aligned(w_gate, 16) || !aligned(logits, 16) || !aligned(topk_idx, 16) ||
      !aligned(topk_w, 16) || !aligned(logit_bias, 4))
    return MOE_ERR_MISALIGNED;
  WsPlan p;
  if ((rc = check_ws(shape, ws, ws_bytes, &p)) != MOE_OK) return rc;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Shape s = to_shape(*shape);
  if (w_gate != nullptr)
    TCMOE_CUDA(launch_gate_logits(s, x, w_gate, logits, at<void>(ws, p.wsplit), at<int32_t>(ws, p.status), st));
  TCMOE_CUDA(launch_topk(s, logits, logit_bias, bias_row_stride, topk_idx, topk_w, at<int32_t>(ws, p.status), st));
  return MOE_OK;
}

int moe_dispatch(const moe_shape_t* shape, const void* x, const int32_t* topk_idx, const moe_layout_t* layout,
                 void* xg, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (topk_idx == nullptr || (xg != nullptr && x == nullptr)) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(x, 128) || !aligned(xg, 128) || !aligned(topk_idx, 16)) return MOE_ERR_MISALIGNED;
  WsPlan p;
  if ((rc = check_ws(shape, ws, ws_bytes, &p)) != MOE_OK) return rc;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Shape s = to_shape(*shape);
  const Layout L = to_layout(*layout);
  TCMOE_CUDA(launch_layout(s, topk_idx, L, scratch(ws, p), at<int32_t>(ws, p.status), st));
  if (xg != nullptr) TCMOE_CUDA(launch_dispatch(s, x, L, xg, st));
  return MOE_OK;
}

int moe_expert_ffn(const moe_shape_t* shape, const void* xg, const moe_layout_t* layout, const float* topk_w,
                   const void* w1, const void* w3, const void* w2, void* o, void* ws, size_t ws_bytes,
                   void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (xg == nullptr || w1 == nullptr || w3 == nullptr || w2 == nullptr || o == nullptr) return MOE_ERR_INVALID_ARG;
  if (shape->flags & MOE_FLAG_COMBINE_IN_EPILOGUE) return MOE_ERR_INVALID_ARG;   // a moe_layer option: o is the result here
  const bool in_combine = (shape->flags & MOE_FLAG_WEIGHT_IN_COMBINE) != 0;
  if (!in_combine && topk_w == nullptr) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(xg, 128) || !aligned(w1, 128) || !aligned(w3, 128) || !aligned(w2, 128) || !aligned(o, 128) ||
      !aligned(topk_w, 16))
    return MOE_ERR_MISALIGNED;
  WsPlan p;
  if ((rc = check_ws(shape, ws, ws_bytes, &p)) != MOE_OK) return rc;
  if (!have_device()) return MOE_ERR_CUDA;
  FfnArgs a{};
  a.a_src = xg;
  a.a_rows = shape->T * (shape->k < shape->G ? shape->k : shape->G);   // capacity of the dispatched buffer
  a.gather_idx = layout->row_src;
  a.gather_div = 1;
  a.w1 = w1;
  a.w3 = w3;
  a.w2 = w2;
  a.xs = (pair_gemm1(*shape) || (shape->flags & MOE_FLAG_TRACK_DISPATCH)) ? at<void>(ws, p.xs) : nullptr;
  a.pair_gemm1 = pair_gemm1(*shape);
  a.track_dispatch = (shape->flags & MOE_FLAG_TRACK_DISPATCH) != 0;
  a.h = at<void>(ws, p.h);
  a.o = o;
  a.topk_w = in_combine ? nullptr : topk_w;
  a.row_pair = layout->row_pair;
  a.expert_offsets = layout->expert_offsets;
  a.expert_counts = layout->expert_counts;
  a.mt_prefix = at<int32_t>(ws, p.mt_prefix);
  a.mp_prefix = at<int32_t>(ws, p.mp_prefix);
  a.blk_start = at<int32_t>(ws, p.blk_start);
  a.blk_info = at<void>(ws, p.blk_info);
  a.n_blocks = at<int32_t>(ws, p.n_blocks);
  a.tracker = at<int32_t>(ws, p.tracker);
  a.status = at<int32_t>(ws, p.status);
  // rebuilt from the counts so that this call does not depend on what moe_dispatch left in ws
  TCMOE_CUDA(launch_tile_prefix(to_shape(*shape), layout->expert_counts, at<int32_t>(ws, p.mt_prefix),
                                at<int32_t>(ws, p.mp_prefix), static_cast<cudaStream_t>(stream)));
  TCMOE_CUDA(launch_expert_ffn(to_shape(*shape), a, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

namespace tcmoe {
namespace {
// Regions of the backward workspace, in order, each on a 1 KiB boundary.
struct BwdPlan {
  size_t status, poff, mt_prefix, mp_prefix, pair_prow, xs, dos, dh, h, da1, da3, dxs, g_row, dkey, wgt, total;
};
BwdPlan bwd_plan(const moe_shape_t& s) {
  BwdPlan p{};
  const size_t E = (size_t)s.E, P = (size_t)s.T * s.k;
  const size_t R = bwd_row_capacity(to_shape(s));
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = round_up(off + bytes, ALIGN);
    return at;
  };
  p.status = take(64);
  p.poff = take((E + 1) * 4);
  p.mt_prefix = take((E + 1) * 4);
  p.mp_prefix = take((E + 1) * 4);
  p.pair_prow = take(P * 4);
  p.xs = take(R * (size_t)s.d * 2);
  p.dos = take(R * (size_t)s.d * 2);
  p.dh = take(R * (size_t)s.f * 2);
  p.h = take(R * (size_t)s.f * 2);
  p.da1 = take(R * (size_t)s.f * 2);
  p.da3 = take(R * (size_t)s.f * 2);
  p.dxs = take(R * (size_t)s.d * 2);
  p.g_row = take(R * 4);                       // moe_gate_backward: row dots, then key gradients per padded row
  p.dkey = take(P * 4);                        //   key gradients per pair
  p.wgt = take(E * (size_t)s.d * 4);           //   the gate weight transposed
  p.total = off;
  return p;
}
}  // namespace
}  // namespace tcmoe

int moe_backward_workspace_bytes(const moe_shape_t* shape, size_t* bytes) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (bytes == nullptr) return MOE_ERR_INVALID_ARG;
  *bytes = bwd_plan(*shape).total;
  return MOE_OK;
}

int moe_layer_backward(const moe_shape_t* shape, const void* x, const void* dy, const int32_t* topk_idx,
                       const float* topk_w, const moe_layout_t* layout, const void* w1, const void* w3, const void* w2,
                       void* dx, void* dw1, void* dw3, void* dw2, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (shape->flags & ~MOE_FLAG_SPARSE_TOPK) return MOE_ERR_INVALID_ARG;   // the forward's kernel-form flags do not apply
  if (x == nullptr || dy == nullptr || topk_idx == nullptr || topk_w == nullptr || w1 == nullptr || w3 == nullptr ||
      w2 == nullptr || dx == nullptr || dw1 == nullptr || dw3 == nullptr || dw2 == nullptr || ws == nullptr)
    return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(x, 128) || !aligned(dy, 128) || !aligned(w1, 128) || !aligned(w3, 128) || !aligned(w2, 128) ||
      !aligned(dx, 128) || !aligned(dw1, 128) || !aligned(dw3, 128) || !aligned(dw2, 128) || !aligned(ws, 128) ||
      !aligned(topk_idx, 16) || !aligned(topk_w, 16))
    return MOE_ERR_MISALIGNED;
  const BwdPlan p = bwd_plan(*shape);
  if (ws_bytes < p.total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  if (!have_device()) return MOE_ERR_CUDA;
  BwdArgs a{};
  a.x = x;
  a.dy = dy;
  a.topk_idx = topk_idx;
  a.topk_w = topk_w;
  a.L = to_layout(*layout);
  a.w1 = w1;
  a.w3 = w3;
  a.w2 = w2;
  a.dx = dx;
  a.dw1 = dw1;
  a.dw3 = dw3;
  a.dw2 = dw2;
  a.poff = at<int32_t>(ws, p.poff);
  a.mt_prefix = at<int32_t>(ws, p.mt_prefix);
  a.mp_prefix = at<int32_t>(ws, p.mp_prefix);
  a.pair_prow = at<int32_t>(ws, p.pair_prow);
  a.xs = at<void>(ws, p.xs);
  a.dos = at<void>(ws, p.dos);
  a.dh = at<void>(ws, p.dh);
  a.h = at<void>(ws, p.h);
  a.da1 = at<void>(ws, p.da1);
  a.da3 = at<void>(ws, p.da3);
  a.dxs = at<void>(ws, p.dxs);
  a.status = at<int32_t>(ws, p.status);
  TCMOE_CUDA(launch_layer_backward(to_shape(*shape), a, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_gate_backward(const moe_shape_t* shape, const float* logits, const float* logit_bias, int64_t bias_row_stride,
                      const int32_t* topk_idx, const float* topk_w, const moe_layout_t* layout, const float* w_gate,
                      void* dx, float* dw_gate, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (shape->flags & ~MOE_FLAG_SPARSE_TOPK) return MOE_ERR_INVALID_ARG;
  if (topk_idx == nullptr || topk_w == nullptr || w_gate == nullptr || dx == nullptr || dw_gate == nullptr ||
      ws == nullptr)
    return MOE_ERR_INVALID_ARG;
  if (shape->score_fn == MOE_SCORE_SIGMOID && logits == nullptr) return MOE_ERR_INVALID_ARG;
  if (logit_bias != nullptr && bias_row_stride != 0 && bias_row_stride != shape->E) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(dx, 128) || !aligned(ws, 128) || !aligned(w_gate, 16) || !aligned(dw_gate, 16) ||
      !aligned(topk_idx, 16) || !aligned(topk_w, 16) || !aligned(logits, 16) || !aligned(logit_bias, 4))
    return MOE_ERR_MISALIGNED;
  const BwdPlan p = bwd_plan(*shape);
  if (ws_bytes < p.total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  if (!have_device()) return MOE_ERR_CUDA;
  GateBwdArgs a{};
  a.topk_idx = topk_idx;
  a.topk_w = topk_w;
  a.expert_counts = layout->expert_counts;
  a.logits = logits;
  a.bias = logit_bias;
  a.bias_stride = bias_row_stride;
  a.w_gate = w_gate;
  a.dx = dx;
  a.dw_gate = dw_gate;
  a.poff = at<int32_t>(ws, p.poff);
  a.pair_prow = at<int32_t>(ws, p.pair_prow);
  a.xs = at<void>(ws, p.xs);
  a.h = at<void>(ws, p.h);
  a.dh = at<void>(ws, p.dh);
  a.g_row = at<float>(ws, p.g_row);
  a.dkey = at<float>(ws, p.dkey);
  a.wgt = at<float>(ws, p.wgt);
  TCMOE_CUDA(launch_gate_backward(to_shape(*shape), a, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_quantize_rows(const void* src, int64_t rows, int64_t cols, void* dst, float* scale, void* stream) {
  if (rows < 0 || cols <= 0 || cols > (1ll << 30)) return MOE_ERR_INVALID_ARG;
  if (cols % 8 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (rows > 0 && (src == nullptr || dst == nullptr || scale == nullptr)) return MOE_ERR_INVALID_ARG;
  if (!aligned(src, 16) || !aligned(dst, 8) || !aligned(scale, 4)) return MOE_ERR_MISALIGNED;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(launch_quantize_rows(src, rows, (int)cols, dst, scale, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_quantize_weights(const void* w, int32_t E, int32_t K, int32_t N, void* wq, float* scale, void* stream) {
  if (E <= 0 || K <= 0 || N <= 0 || E > 65535) return MOE_ERR_INVALID_ARG;
  if (w == nullptr || wq == nullptr || scale == nullptr) return MOE_ERR_INVALID_ARG;
  if (!aligned(w, 16) || !aligned(wq, 16) || !aligned(scale, 4)) return MOE_ERR_MISALIGNED;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(launch_quantize_weights(w, E, K, N, wq, scale, static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

int moe_expert_ffn_fp8(const moe_shape_t* shape, const void* xq, const float* sx, const moe_layout_t* layout,
                       const float* topk_w, const void* w1q, const float* s1, const void* w3q, const float* s3,
                       const void* w2q, const float* s2, void* o, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (shape->d % 16 != 0 || shape->f % 16 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;   // 16-byte rows of 8-bit elements
  if (shape->flags & MOE_FLAG_FUSED_FFN) return MOE_ERR_INVALID_ARG;                  // bf16 experts only
  if (xq == nullptr || sx == nullptr || w1q == nullptr || w3q == nullptr || w2q == nullptr || s1 == nullptr ||
      s3 == nullptr || s2 == nullptr || o == nullptr)
    return MOE_ERR_INVALID_ARG;
  if (shape->flags & MOE_FLAG_COMBINE_IN_EPILOGUE) return MOE_ERR_INVALID_ARG;
  const bool in_combine = (shape->flags & MOE_FLAG_WEIGHT_IN_COMBINE) != 0;
  if (!in_combine && topk_w == nullptr) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(xq, 128) || !aligned(w1q, 128) || !aligned(w3q, 128) || !aligned(w2q, 128) || !aligned(o, 128) ||
      !aligned(topk_w, 16) || !aligned(sx, 4) || !aligned(s1, 4) || !aligned(s3, 4) || !aligned(s2, 4))
    return MOE_ERR_MISALIGNED;
  WsPlan p;
  if ((rc = check_ws(shape, ws, ws_bytes, &p)) != MOE_OK) return rc;
  if (!have_device()) return MOE_ERR_CUDA;
  FfnArgs a{};
  a.a_src = xq;
  a.a_rows = shape->T * (shape->k < shape->G ? shape->k : shape->G);   // capacity of the dispatched buffer
  a.gather_idx = layout->row_src;
  a.gather_div = 1;
  a.w1 = w1q;
  a.w3 = w3q;
  a.w2 = w2q;
  a.xs = (pair_gemm1(*shape) || (shape->flags & MOE_FLAG_TRACK_DISPATCH)) ? at<void>(ws, p.xs) : nullptr;
  a.pair_gemm1 = pair_gemm1(*shape);
  a.track_dispatch = (shape->flags & MOE_FLAG_TRACK_DISPATCH) != 0;
  a.h = at<void>(ws, p.h);
  a.o = o;
  a.topk_w = in_combine ? nullptr : topk_w;
  a.row_pair = layout->row_pair;
  a.expert_offsets = layout->expert_offsets;
  a.expert_counts = layout->expert_counts;
  a.mt_prefix = at<int32_t>(ws, p.mt_prefix);
  a.mp_prefix = at<int32_t>(ws, p.mp_prefix);
  a.blk_start = at<int32_t>(ws, p.blk_start);
  a.blk_info = at<void>(ws, p.blk_info);
  a.n_blocks = at<int32_t>(ws, p.n_blocks);
  a.tracker = at<int32_t>(ws, p.tracker);
  a.status = at<int32_t>(ws, p.status);
  Fp8Args q{sx, s1, s3, s2, at<void>(ws, p.hq), at<float>(ws, p.sh)};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  TCMOE_CUDA(launch_tile_prefix(to_shape(*shape), layout->expert_counts, at<int32_t>(ws, p.mt_prefix),
                                at<int32_t>(ws, p.mp_prefix), st));
  TCMOE_CUDA(launch_expert_ffn_fp8(to_shape(*shape), a, q, st));
  return MOE_OK;
}

int moe_combine(const moe_shape_t* shape, const void* o, const moe_layout_t* layout, const int32_t* topk_idx,
                const float* topk_w, void* pg, void* y, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (o == nullptr || y == nullptr || topk_idx == nullptr) return MOE_ERR_INVALID_ARG;
  if (shape->flags & MOE_FLAG_COMBINE_IN_EPILOGUE) return MOE_ERR_INVALID_ARG;
  if ((shape->flags & MOE_FLAG_WEIGHT_IN_COMBINE) && topk_w == nullptr) return MOE_ERR_INVALID_ARG;
  if ((rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(o, 128) || !aligned(y, 128) || !aligned(pg, 128) || !aligned(topk_idx, 16) || !aligned(topk_w, 16))
    return MOE_ERR_MISALIGNED;
  WsPlan p;
  if ((rc = check_ws(shape, ws, ws_bytes, &p)) != MOE_OK) return rc;
  if (!have_device()) return MOE_ERR_CUDA;
  TCMOE_CUDA(launch_combine(to_shape(*shape), o, to_layout(*layout), topk_idx, topk_w, pg, y,
                            at<int32_t>(ws, p.status), static_cast<cudaStream_t>(stream)));
  return MOE_OK;
}

// Shared body of moe_layer and moe_layer_fp8.  fp8 == nullptr: bf16 experts, w1 / w3 / w2 are
// [E, K, N] bf16.  Otherwise they are E4M3 codes [E, N, K] with the scales in *fp8 (sx, hq, sh are
// filled here from the workspace).
static int layer_impl(const moe_shape_t* shape, const void* x, const float* w_gate, const float* logit_bias,
                      int64_t bias_row_stride, const void* w1, const void* w3, const void* w2, const Fp8Args* fp8,
                      void* y, float* logits, int32_t* topk_idx, float* topk_w, const moe_layout_t* layout, void* ws,
                      size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (shape->flags & MOE_FLAG_SPARSE_TOPK) return MOE_ERR_INVALID_ARG;   // the layer's own top-k fills every slot
  if (fp8 != nullptr) {
    if (shape->flags & MOE_FLAG_FUSED_FFN) return MOE_ERR_INVALID_ARG;   // bf16 experts only
    if (shape->d % 16 != 0 || shape->f % 16 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;
    if (fp8->s1 == nullptr || fp8->s3 == nullptr || fp8->s2 == nullptr) return MOE_ERR_INVALID_ARG;
    if (!aligned(fp8->s1, 4) || !aligned(fp8->s3, 4) || !aligned(fp8->s2, 4)) return MOE_ERR_MISALIGNED;
  }
  if (x == nullptr || w_gate == nullptr || w1 == nullptr || w3 == nullptr || w2 == nullptr || y == nullptr)
    return MOE_ERR_INVALID_ARG;
  if (bias_row_stride != 0 && bias_row_stride != shape->E) return MOE_ERR_INVALID_ARG;
  if (layout != nullptr && (rc = check_layout(layout)) != MOE_OK) return rc;
  if (!aligned(x, 128) || !aligned(w1, 128) || !aligned(w3, 128) || !aligned(w2, 128) || !aligned(y, 128) ||
      !aligned(w_gate, 16) || !aligned(logits, 16) || !aligned(topk_idx, 16) || !aligned(topk_w, 16) ||
      !aligned(logit_bias, 4))
    return MOE_ERR_MISALIGNED;
  WsPlan p;
  if ((rc = check_ws(shape, ws, ws_bytes, &p)) != MOE_OK) return rc;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Shape s = to_shape(*shape);
  int32_t* status = at<int32_t>(ws, p.status);
  float* lg = logits != nullptr ? logits : at<float>(ws, p.logits);
  int32_t* idx = topk_idx != nullptr ? topk_idx : at<int32_t>(ws, p.topk_idx);
  float* tw = topk_w != nullptr ? topk_w : at<float>(ws, p.topk_w);
  Layout L;
  if (layout != nullptr) {
    L = to_layout(*layout);
  } else {
    L = Layout{at<int32_t>(ws, p.expert_counts), at<int32_t>(ws, p.expert_offsets), at<int32_t>(ws, p.group_counts),
               at<int32_t>(ws, p.group_offsets), at<int32_t>(ws, p.pair_row),       at<int32_t>(ws, p.row_pair),
               at<int32_t>(ws, p.al),            at<int32_t>(ws, p.disp_token),     at<int32_t>(ws, p.row_src)};
  }
  // gate
  TCMOE_CUDA(launch_gate_logits(s, x, w_gate, lg, at<void>(ws, p.wsplit), status, st));
  // the top-k kernel also zeroes the bitmasks of the layout builder (emask and gmask are adjacent)
  const LayoutScratch sc = scratch(ws, p);
  TCMOE_CUDA(launch_topk(s, lg, logit_bias, bias_row_stride, idx, tw, status, st, sc.emask,
                         (size_t)(s.E + s.G) * sc.W));
  // layout only: the dispatched copy xg is never written, GEMM-1 gathers token rows from x
  TCMOE_CUDA(launch_layout(s, idx, L, sc, status, st, /*masks_cleared=*/s.T > 0));
  FfnArgs a{};
  a.a_src = x;
  Fp8Args q{};
  if (fp8 != nullptr) {   // experts read the E4M3 copy of x
    q = *fp8;
    q.sx = at<float>(ws, p.sx);
    q.hq = at<void>(ws, p.hq);
    q.sh = at<float>(ws, p.sh);
    a.a_src = at<void>(ws, p.xq);
    TCMOE_CUDA(launch_quantize_rows(x, s.T, s.d, at<void>(ws, p.xq), at<float>(ws, p.sx), st));
  }
  a.a_rows = s.T;
  a.gather_idx = L.row_pair;   // token of expert row r = row_pair[r] / k
  a.gather_div = s.k;
  a.w1 = w1;
  a.w3 = w3;
  a.w2 = w2;
  a.xs = (pair_gemm1(*shape) || (shape->flags & MOE_FLAG_TRACK_DISPATCH)) ? at<void>(ws, p.xs) : nullptr;
  a.pair_gemm1 = pair_gemm1(*shape);
  a.track_dispatch = (shape->flags & MOE_FLAG_TRACK_DISPATCH) != 0;
  a.h = at<void>(ws, p.h);
  a.o = at<void>(ws, p.o);
  a.topk_w = (s.flags & MOE_FLAG_WEIGHT_IN_COMBINE) ? nullptr : tw;
  a.row_pair = L.row_pair;
  a.expert_offsets = L.expert_offsets;
  a.expert_counts = L.expert_counts;
  a.mt_prefix = at<int32_t>(ws, p.mt_prefix);
  a.mp_prefix = at<int32_t>(ws, p.mp_prefix);
  a.blk_start = at<int32_t>(ws, p.blk_start);
  a.blk_info = at<void>(ws, p.blk_info);
  a.n_blocks = at<int32_t>(ws, p.n_blocks);
  a.tracker = at<int32_t>(ws, p.tracker);
  a.status = status;
  if (s.flags & MOE_FLAG_COMBINE_IN_EPILOGUE) {
    // o never materialises: GEMM-2 adds each weighted row into its token's fp32 accumulator
    a.y_acc = at<float>(ws, p.o);
    if (s.T > 0) TCMOE_CUDA(cudaMemsetAsync(a.y_acc, 0, (size_t)s.T * s.d * 4, st));
    TCMOE_CUDA(fp8 != nullptr ? launch_expert_ffn_fp8(s, a, q, st) : launch_expert_ffn(s, a, st));
    TCMOE_CUDA(launch_round_rows(s, a.y_acc, y, st));
    return MOE_OK;
  }
  if (s.flags & MOE_FLAG_FUSED_FFN) {
    // one kernel after the layout: GEMM-1, GEMM-2 and Combine tasks (and Dispatch tasks when asked for) paced by
    // the token tracker; the Combine tasks produce y
    a.comb = CombineArgs{static_cast<const uint4*>(a.o), static_cast<uint4*>(y), nullptr, idx, tw, L.pair_row, L.al,
                         L.group_offsets, s.T, s.E, s.k, s.E / s.G, s.d / 8,
                         (s.flags & MOE_FLAG_WEIGHT_IN_COMBINE) ? 1 : 0, s.T * s.k, status};
    TCMOE_CUDA(launch_expert_ffn(s, a, st));
    return MOE_OK;
  }
  TCMOE_CUDA(fp8 != nullptr ? launch_expert_ffn_fp8(s, a, q, st) : launch_expert_ffn(s, a, st));
  TCMOE_CUDA(launch_combine(s, a.o, L, idx, tw, nullptr, y, status, st));
  return MOE_OK;
}

int moe_layer(const moe_shape_t* shape, const void* x, const float* w_gate, const float* logit_bias,
              int64_t bias_row_stride, const void* w1, const void* w3, const void* w2, void* y, float* logits,
              int32_t* topk_idx, float* topk_w, const moe_layout_t* layout, void* ws, size_t ws_bytes, void* stream) {
  return layer_impl(shape, x, w_gate, logit_bias, bias_row_stride, w1, w3, w2, nullptr, y, logits, topk_idx, topk_w,
                    layout, ws, ws_bytes, stream);
}

int moe_layer_fp8(const moe_shape_t* shape, const void* x, const float* w_gate, const float* logit_bias,
                  int64_t bias_row_stride, const void* w1q, const float* s1, const void* w3q, const float* s3,
                  const void* w2q, const float* s2, void* y, float* logits, int32_t* topk_idx, float* topk_w,
                  const moe_layout_t* layout, void* ws, size_t ws_bytes, void* stream) {
  Fp8Args q{};
  q.s1 = s1;
  q.s3 = s3;
  q.s2 = s2;
  return layer_impl(shape, x, w_gate, logit_bias, bias_row_stride, w1q, w3q, w2q, &q, y, logits, topk_idx, topk_w,
                    layout, ws, ws_bytes, stream);
}

int moe_layer_host(const moe_shape_t* shape, const void* x_host, void* x_dev, const float* w_gate,
                   const float* logit_bias, int64_t bias_row_stride, const void* w1, const void* w3, const void* w2,
                   void* y_dev, void* y_host, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (x_host == nullptr || x_dev == nullptr || y_dev == nullptr || y_host == nullptr) return MOE_ERR_INVALID_ARG;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)shape->T * shape->d * 2;
  if (bytes) TCMOE_CUDA(cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, st));
  rc = moe_layer(shape, x_dev, w_gate, logit_bias, bias_row_stride, w1, w3, w2, y_dev, nullptr, nullptr, nullptr,
                 nullptr, ws, ws_bytes, stream);
  if (rc != MOE_OK) return rc;
  if (bytes) TCMOE_CUDA(cudaMemcpyAsync(y_host, y_dev, bytes, cudaMemcpyDeviceToHost, st));
  return MOE_OK;
}

int moe_layer_fp8_host(const moe_shape_t* shape, const void* x_host, void* x_dev, const float* w_gate,
                       const float* logit_bias, int64_t bias_row_stride, const void* w1q, const float* s1,
                       const void* w3q, const float* s3, const void* w2q, const float* s2, void* y_dev, void* y_host,
                       void* ws, size_t ws_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (x_host == nullptr || x_dev == nullptr || y_dev == nullptr || y_host == nullptr) return MOE_ERR_INVALID_ARG;
  if (!have_device()) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)shape->T * shape->d * 2;
  if (bytes) TCMOE_CUDA(cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, st));
  rc = moe_layer_fp8(shape, x_dev, w_gate, logit_bias, bias_row_stride, w1q, s1, w3q, s3, w2q, s2, y_dev, nullptr,
                     nullptr, nullptr, nullptr, ws, ws_bytes, stream);
  if (rc != MOE_OK) return rc;
  if (bytes) TCMOE_CUDA(cudaMemcpyAsync(y_host, y_dev, bytes, cudaMemcpyDeviceToHost, st));
  return MOE_OK;
}

}  // extern "C"
