// bf16 -> E4M3 quantisation for the FP8 form of the expert FFN (paper Sec. V-A: the evaluated
// DeepSeek-V3 experts run FP8 GEMMs; format and scaling are this library's reading):
//   scale = fl32(max|v| / 448) over a row (activations) or over K for one (expert, output column)
//           (weights); 1 for an all-zero vector
//   code  = e4m3(fl32(v / scale)), round to nearest even, saturating at +-448
// Every step is a single fp32 operation, so a CPU restatement takes the same decisions.
#include "common.cuh"

#include <cuda_bf16.h>
#include <cuda_fp8.h>

namespace tcmoe {
namespace {

__device__ __forceinline__ uint8_t to_e4m3(float v, float scale) {
  return (uint8_t)__nv_cvt_float_to_fp8(__fdiv_rn(v, scale), __NV_SATFINITE, __NV_E4M3);
}
__device__ __forceinline__ float scale_of(float amax) { return amax == 0.f ? 1.f : __fdiv_rn(amax, 448.f); }

// One warp per row: pass 1 takes max|v| (16-byte loads), pass 2 re-reads the row (L1 / L2) and
// writes 8 codes per lane per step.  cols % 8 == 0.
__global__ void __launch_bounds__(256) quantize_rows_kernel(const uint4* __restrict__ src, uint2* __restrict__ dst,
                                                            float* __restrict__ scale, long long rows, int vec_per_row) {
  grid_dependency_sync();
  const int lane = threadIdx.x & 31;
  const long long wpb = blockDim.x >> 5;
  for (long long r = blockIdx.x * wpb + (threadIdx.x >> 5); r < rows; r += (long long)gridDim.x * wpb) {
    const uint4* row = src + r * vec_per_row;
    float amax = 0.f;
    for (int v = lane; v < vec_per_row; v += 32) {
      const uint4 raw = __ldg(row + v);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __bfloat1622float2(p[q]);
        amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, off));
    const float sc = scale_of(amax);
    if (lane == 0) scale[r] = sc;
    uint2* out = dst + r * vec_per_row;
    for (int v = lane; v < vec_per_row; v += 32) {
      const uint4 raw = __ldg(row + v);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
      uint32_t w[2] = {0u, 0u};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __bfloat1622float2(p[q]);
        w[q >> 1] |= ((uint32_t)to_e4m3(f.x, sc) | ((uint32_t)to_e4m3(f.y, sc) << 8)) << (16 * (q & 1));
      }
      out[v] = make_uint2(w[0], w[1]);
    }
  }
}

// Weights [E, K, N] (N contiguous) -> codes [E, N, K] (K contiguous) + scale [E, N].  One block
// per (expert, 32 output columns): pass 1 reduces max|w| over K per column, pass 2 quantises and
// transposes 32 x 32 tiles through shared memory.  A one-time preparation step.
__global__ void __launch_bounds__(256) quantize_weights_kernel(const __nv_bfloat16* __restrict__ w,
                                                               uint8_t* __restrict__ wq, float* __restrict__ scale,
                                                               int K, int N) {
  __shared__ float red[8][32];
  __shared__ float sc_s[32];
  __shared__ uint8_t tile[32][33];
  grid_dependency_sync();
  const int e = blockIdx.y, n0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // tx: column (pass 1 / tile load), ty: 0..7
  const __nv_bfloat16* we = w + (size_t)e * K * N;
  const int n = n0 + tx;
  float amax = 0.f;
  if (n < N)
    for (int k = ty; k < K; k += 8) amax = fmaxf(amax, fabsf(__bfloat162float(we[(size_t)k * N + n])));
  red[ty][tx] = amax;
  __syncthreads();
  if (ty == 0) {
    for (int i = 1; i < 8; ++i) amax = fmaxf(amax, red[i][tx]);
    const float sc = scale_of(amax);
    sc_s[tx] = sc;
    if (n < N) scale[(size_t)e * N + n] = sc;
  }
  __syncthreads();
  uint8_t* qe = wq + (size_t)e * N * K;
  for (int k0 = 0; k0 < K; k0 += 32) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {   // tile[k][n]
      const int k = k0 + ty + 8 * i;
      tile[ty + 8 * i][tx] = (k < K && n < N) ? to_e4m3(__bfloat162float(we[(size_t)k * N + n]), sc_s[tx]) : 0;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {   // write rows of [n][k0 .. k0+31]
      const int nn = n0 + ty + 8 * i, k = k0 + tx;
      if (nn < N && k < K) qe[(size_t)nn * K + k] = tile[tx][ty + 8 * i];
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_quantize_rows(const void* src, long long rows, int cols, void* dst, float* scale, cudaStream_t st) {
  if (rows <= 0 || cols <= 0) return cudaSuccess;
  long long blocks = (rows + 7) / 8;
  const long long cap = (long long)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  return launch_pdl(quantize_rows_kernel, (unsigned)blocks, 256, 0, st, static_cast<const uint4*>(src),
                    static_cast<uint2*>(dst), scale, rows, cols / 8);
}

cudaError_t launch_quantize_weights(const void* w, int E, int K, int N, void* wq, float* scale, cudaStream_t st) {
  if (E <= 0 || K <= 0 || N <= 0) return cudaSuccess;
  return launch_pdl(quantize_weights_kernel, dim3((N + 31) / 32, E), 256, 0, st,
                    static_cast<const __nv_bfloat16*>(w), static_cast<uint8_t*>(wq), scale, K, N);
}

}  // namespace tcmoe
