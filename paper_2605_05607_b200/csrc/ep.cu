// Expert-parallel execution of the layer across GPUs (paper Sec. II-A: Dispatch sends each token to the
// GPUs hosting its experts, Combine brings the outputs back; Sec. III-D: one replica per destination, trimmed
// to that destination's targets; reduction of the outputs of one destination before they travel back).
// With the G expert groups placed on G GPUs, the data that crosses the links is exactly what the single-GPU
// path already builds: the dispatched buffer xg (one row per distinct (token, group)) on the way out, one
// pre-reduced row per (token, group) on the way back.  Two small kernels complete the picture:
//   ep_pack    for every dispatched row the trimmed target list: the token's experts that live in the row's
//              group (as indices local to the group) and their gate weights - the routing table the
//              receiving GPU runs its experts from (MOE_FLAG_SPARSE_TOPK form)
//   ep_finish  y[t] = sum over the groups t touched of the pre-reduced row that came back
// Everything between them (layout, expert FFN, in-group reduction) is the ordinary entry points applied to
// the received rows.
#include "common.cuh"

#include <cuda_bf16.h>

namespace tcmoe {
namespace {

// thread per token: walk the k slots, append each to the list of its (token, group) row
__global__ void __launch_bounds__(256) ep_pack_kernel(const int32_t* __restrict__ topk_idx,
                                                      const float* __restrict__ topk_w,
                                                      const int32_t* __restrict__ al,
                                                      const int32_t* __restrict__ group_offsets,
                                                      int32_t* __restrict__ send_idx, float* __restrict__ send_w, int T,
                                                      int E, int k, int m, int kk) {
  grid_dependency_sync();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  for (int j = 0; j < k; ++j) {
    const int e = __ldg(topk_idx + (size_t)t * k + j);
    if (e < 0 || e >= E) continue;
    const int g = e / m;
    int pos = 0;   // slots of this token before j that live in the same group
    for (int i = 0; i < j; ++i) {
      const int ei = __ldg(topk_idx + (size_t)t * k + i);
      if (ei >= 0 && ei < E && ei / m == g) ++pos;
    }
    const size_t n = (size_t)__ldg(group_offsets + g) + __ldg(al + (size_t)g * T + t);
    send_idx[n * kk + pos] = e - g * m;
    send_w[n * kk + pos] = __ldg(topk_w + (size_t)t * k + j);
  }
}

// warp per token: fp32 sum over the groups, ascending g, 8 bf16 per lane per step
__global__ void __launch_bounds__(256) ep_finish_kernel(const uint4* __restrict__ back, uint4* __restrict__ y,
                                                        const int32_t* __restrict__ al,
                                                        const int32_t* __restrict__ group_offsets, int T, int G,
                                                        int vec_per_row) {
  grid_dependency_sync();
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  for (int t = blockIdx.x * wpb + (threadIdx.x >> 5); t < T; t += gridDim.x * wpb) {
    for (int v = lane; v < vec_per_row; v += 32) {
      float acc[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) acc[q] = 0.f;
      for (int g = 0; g < G; ++g) {
        const int a = __ldg(al + (size_t)g * T + t);
        if (a < 0) continue;
        const uint4 raw = __ldcs(back + ((size_t)__ldg(group_offsets + g) + a) * vec_per_row + v);
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 f = __bfloat1622float2(p[q]);
          acc[2 * q] += f.x;
          acc[2 * q + 1] += f.y;
        }
      }
      uint4 out;
      __nv_bfloat162* o = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
      for (int q = 0; q < 4; ++q) o[q] = __floats2bfloat162_rn(acc[2 * q], acc[2 * q + 1]);
      y[(size_t)t * vec_per_row + v] = out;
    }
  }
}

}  // namespace

cudaError_t launch_ep_pack(const Shape& s, const int32_t* topk_idx, const float* topk_w, const Layout& L,
                           int32_t* send_idx, float* send_w, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  const int m = s.E / s.G, kk = s.k < m ? s.k : m;
  const size_t cap = (size_t)s.T * (s.k < s.G ? s.k : s.G) * kk;   // dispatched-row capacity x list length
  cudaError_t err;
  if ((err = cudaMemsetAsync(send_idx, 0xFF, cap * sizeof(int32_t), st)) != cudaSuccess) return err;   // -1: unused slot
  if ((err = cudaMemsetAsync(send_w, 0, cap * sizeof(float), st)) != cudaSuccess) return err;
  return launch_pdl(ep_pack_kernel, (s.T + 255) / 256, 256, 0, st, topk_idx, topk_w, L.al, L.group_offsets, send_idx,
                    send_w, s.T, s.E, s.k, m, kk);
}

cudaError_t launch_ep_finish(const Shape& s, const void* back, const Layout& L, void* y, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  int blocks = (s.T + 7) / 8;
  const int cap = sm_count() * 8;
  if (blocks > cap) blocks = cap;
  return launch_pdl(ep_finish_kernel, blocks, 256, 0, st, static_cast<const uint4*>(back), static_cast<uint4*>(y), L.al,
                    L.group_offsets, s.T, s.G, s.d / 8);
}

}  // namespace tcmoe
