// Gradient that reaches the gate network (paper Sec. II-A: the gate picks the topk experts of a token and weighs
// their outputs; Sec. VI-A evaluates training).  The SELECTION is held fixed; the gate weights are functions of the
// router keys  key[t, e] = x[t] . w_gate[:, e] + bias[t, e]:
//     y[t] = sum_j w[t, j] * FFN_{e_j}(x[t]),   w[t, :] = softmax (or renormalised sigmoid) of key[t, e_0 .. e_{k-1}]
// With L = sum(dy * y):
//     g[t, j]    = w[t, j] * dL/dw[t, j] = w[t, j] * dy[t] . FFN_{e_j}(x[t])
//     dkey[t, j] = (g[t, j] - w[t, j] * sum_i g[t, i]) * c[t, j],     c = 1 (softmax),  1 - sigmoid(key[t, j]) (sigmoid)
//     dw_gate    = x^T . dlogits,    dx[t] += sum_j dkey[t, j] * w_gate[:, e_j]
// (dkey follows from the quotient rule with w_j = s_j / sum_i s_i; no division is left in either form.)
//
// The expert part of the backward pass (bwd.cu) has just produced, in the padded row space of its workspace,
// h (the recomputed SwiGLU output of every pair) and dH = (w * dy) . W2^T.  Their row-wise dot product is
//     h[r] . dH[r] = w_r * (h[r] . W2) . dy[t_r] = g  of the pair in row r,
// so dL/dw costs one pass over two [rows, f] buffers and no GEMM.  dw_gate is a weighted sum of each expert's rows of
// xs (also still in the workspace), dx gets k rows of the transposed gate weight per token.
//
// Sequence (one stream): row dots -> per-token key gradients -> dw_gate (one block per expert and column slab, rows in
// ascending order: deterministic) -> transpose of w_gate -> dx update.
#include "common.cuh"

#include <cuda_bf16.h>

namespace tcmoe {
namespace {

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b) {
  const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
  float s = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float2 fa = __bfloat1622float2(pa[q]), fb = __bfloat1622float2(pb[q]);
    s = fmaf(fa.x, fb.x, s);
    s = fmaf(fa.y, fb.y, s);
  }
  return s;
}

// g_row[r] = h[r] . dH[r] for the rows in use (r < poff[E]); a warp per row
__global__ void __launch_bounds__(256) gate_rowdot_kernel(const uint4* __restrict__ h, const uint4* __restrict__ dh,
                                                          const int32_t* __restrict__ poff, float* __restrict__ g_row,
                                                          int E, int vec_per_row) {
  grid_dependency_sync();
  const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
  const int rows = __ldg(poff + E);
  for (int r = blockIdx.x * wpb + (threadIdx.x >> 5); r < rows; r += gridDim.x * wpb) {
    const uint4* hr = h + (size_t)r * vec_per_row;
    const uint4* dr = dh + (size_t)r * vec_per_row;
    float s = 0.f;
    for (int v = lane; v < vec_per_row; v += 32) s += dot8(__ldcs(hr + v), __ldcs(dr + v));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
    if (lane == 0) g_row[r] = s;
  }
}

// One thread per token: key gradients of its k pairs; written per pair (dkey) and in place per padded row (g_row)
__global__ void __launch_bounds__(256) gate_route_bwd_kernel(const int32_t* __restrict__ topk_idx,
                                                             const float* __restrict__ topk_w,
                                                             const int32_t* __restrict__ pair_prow,
                                                             const float* __restrict__ logits,
                                                             const float* __restrict__ bias, long long bias_stride,
                                                             float* g_row, float* __restrict__ dkey, int T, int E, int k,
                                                             int sigmoid, int n_rows) {
  grid_dependency_sync();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  const size_t base = (size_t)t * k;
  float dot = 0.f;
  for (int j = 0; j < k; ++j) {
    const int r = __ldg(pair_prow + base + j);
    if (r >= 0 && r < n_rows) dot += g_row[r];
  }
  for (int j = 0; j < k; ++j) {
    const int r = __ldg(pair_prow + base + j);
    float v = 0.f;
    if (r >= 0 && r < n_rows) {
      const float w = __ldg(topk_w + base + j);
      v = g_row[r] - w * dot;
      if (sigmoid) {
        const int e = __ldg(topk_idx + base + j);
        float key = __ldg(logits + (size_t)t * E + e);
        if (bias != nullptr) key += __ldg(bias + (size_t)t * bias_stride + e);
        v *= 1.f - 1.f / (1.f + __expf(-key));
      }
      g_row[r] = v;   // from here on g_row holds the key gradient of the pair in row r
    }
    dkey[base + j] = v;
  }
}

// dw_gate[c, e] = sum over the rows r of expert e (ascending) of dkey_row[r] * xs[r, c].  Block: 256 threads x 8
// columns; grid (column slabs, experts).
__global__ void __launch_bounds__(256) gate_dw_kernel(const uint4* __restrict__ xs, const float* __restrict__ dkey_row,
                                                      const int32_t* __restrict__ poff,
                                                      const int32_t* __restrict__ expert_counts,
                                                      float* __restrict__ dw_gate, int E, int d) {
  grid_dependency_sync();
  const int e = blockIdx.y;
  const int v = blockIdx.x * blockDim.x + threadIdx.x;   // uint4 index inside the row
  const int vec_per_row = d >> 3;
  if (v >= vec_per_row) return;
  const int r0 = __ldg(poff + e), n = __ldg(expert_counts + e);
  float acc[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) acc[q] = 0.f;
  const uint4* col = xs + (size_t)r0 * vec_per_row + v;
#pragma unroll 4
  for (int i = 0; i < n; ++i) {
    const float g = __ldg(dkey_row + r0 + i);
    const uint4 xv = __ldcs(col + (size_t)i * vec_per_row);
    const __nv_bfloat162* px = reinterpret_cast<const __nv_bfloat162*>(&xv);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 f = __bfloat1622float2(px[q]);
      acc[2 * q] = fmaf(g, f.x, acc[2 * q]);
      acc[2 * q + 1] = fmaf(g, f.y, acc[2 * q + 1]);
    }
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) dw_gate[(size_t)(v * 8 + q) * E + e] = acc[q];
}

// wgt[e, c] = w_gate[c, e]: 32 x 32 tiles through shared memory
__global__ void __launch_bounds__(256) gate_transpose_kernel(const float* __restrict__ w_gate, float* __restrict__ wgt,
                                                             int d, int E) {
  grid_dependency_sync();
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, e0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 8 rows per pass
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i, e = e0 + tx;
    tile[i][tx] = (c < d && e < E) ? __ldg(w_gate + (size_t)c * E + e) : 0.f;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int e = e0 + i, c = c0 + tx;
    if (e < E && c < d) wgt[(size_t)e * d + c] = tile[tx][i];
  }
}

// dx[t, :] += sum_j dkey[t, j] * wgt[e_j, :]; a warp per token, four columns per lane and step
__global__ void __launch_bounds__(256) gate_dx_kernel(const int32_t* __restrict__ topk_idx, const float* __restrict__ dkey,
                                                      const float* __restrict__ wgt, __nv_bfloat16* dx, int T, int E,
                                                      int k, int d) {
  grid_dependency_sync();
  __shared__ int s_e[8][32];
  __shared__ float s_g[8][32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, wpb = blockDim.x >> 5;
  for (int t = blockIdx.x * wpb + wid; t < T; t += gridDim.x * wpb) {
    __syncwarp();
    if (lane < k) {
      const int e = __ldg(topk_idx + (size_t)t * k + lane);
      const bool in = e >= 0 && e < E;
      s_e[wid][lane] = in ? e : 0;
      s_g[wid][lane] = in ? __ldg(dkey + (size_t)t * k + lane) : 0.f;
    }
    __syncwarp();
    __nv_bfloat16* row = dx + (size_t)t * d;
    for (int c = lane * 4; c < d; c += 128) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int j = 0; j < k; ++j) {
        const float g = s_g[wid][j];
        const float4 wv = __ldg(reinterpret_cast<const float4*>(wgt + (size_t)s_e[wid][j] * d + c));
        acc.x = fmaf(g, wv.x, acc.x);
        acc.y = fmaf(g, wv.y, acc.y);
        acc.z = fmaf(g, wv.z, acc.z);
        acc.w = fmaf(g, wv.w, acc.w);
      }
      uint2 raw = *reinterpret_cast<const uint2*>(row + c);
      __nv_bfloat162* p2 = reinterpret_cast<__nv_bfloat162*>(&raw);
      const float2 lo = __bfloat1622float2(p2[0]), hi = __bfloat1622float2(p2[1]);
      p2[0] = __floats2bfloat162_rn(lo.x + acc.x, lo.y + acc.y);
      p2[1] = __floats2bfloat162_rn(hi.x + acc.z, hi.y + acc.w);
      *reinterpret_cast<uint2*>(row + c) = raw;
    }
  }
}

}  // namespace

cudaError_t launch_gate_backward(const Shape& s, const GateBwdArgs& a, cudaStream_t st) {
  cudaError_t err;
  if (s.T == 0) return cudaMemsetAsync(a.dw_gate, 0, (size_t)s.d * s.E * sizeof(float), st);
  const int n_rows = (int)bwd_row_capacity(s);
  ProfileScope prof(KID_GATE_BWD, st);
  const int cap = sm_count() * 8;
  int blocks = (n_rows + 7) / 8;
  if (blocks > cap) blocks = cap;
  if ((err = launch_pdl(gate_rowdot_kernel, blocks, 256, 0, st, static_cast<const uint4*>(a.h),
                        static_cast<const uint4*>(a.dh), a.poff, a.g_row, s.E, s.f / 8)) != cudaSuccess)
    return err;
  if ((err = launch_pdl(gate_route_bwd_kernel, (s.T + 255) / 256, 256, 0, st, a.topk_idx, a.topk_w, a.pair_prow,
                        a.logits, a.bias, (long long)a.bias_stride, a.g_row, a.dkey, s.T, s.E, s.k,
                        s.score_fn == 1 ? 1 : 0, n_rows)) != cudaSuccess)
    return err;
  if ((err = launch_pdl(gate_dw_kernel, dim3((s.d / 8 + 255) / 256, s.E), 256, 0, st, static_cast<const uint4*>(a.xs),
                        static_cast<const float*>(a.g_row), a.poff, a.expert_counts, a.dw_gate, s.E, s.d)) != cudaSuccess)
    return err;
  if ((err = launch_pdl(gate_transpose_kernel, dim3((s.d + 31) / 32, (s.E + 31) / 32), 256, 0, st, a.w_gate, a.wgt, s.d,
                        s.E)) != cudaSuccess)
    return err;
  blocks = (s.T + 7) / 8;
  if (blocks > cap) blocks = cap;
  return launch_pdl(gate_dx_kernel, blocks, 256, 0, st, a.topk_idx, static_cast<const float*>(a.dkey),
                    static_cast<const float*>(a.wgt), static_cast<__nv_bfloat16*>(a.dx), s.T, s.E, s.k, s.d);
}

}  // namespace tcmoe
