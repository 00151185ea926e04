// Routing of the MoE layer (paper Sec. II-A: the gate network selects topk experts per token); the
// gate logits themselves are computed in gate_gemm.cu.
//   topk_kernel : key = logit + bias; k largest keys per token ordered by
//                 (key descending, expert index ascending); gate weights over the k keys
#include "common.cuh"

#include <cuda_bf16.h>

namespace tcmoe {

// ------------------------------------------------------------------------------------------------
// Top-k: one warp per token.  Lane l holds experts l, l+32, ... (KPL of them) as order-preserving
// unsigned keys.  k rounds of: lane-local best -> warp max of the key -> warp min of the expert
// index among the lanes holding that key.  -0.0 is folded onto +0.0 and NaN onto -inf before
// ordering, so comparisons agree with IEEE "==" ties and never hang on NaN.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t order_key(float v, bool& nonfinite) {
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) == 0x7F800000u) {
    nonfinite = true;
    if (u & 0x007FFFFFu) u = 0xFF800000u;  // NaN -> -inf
  }
  if ((u << 1) == 0) u = 0;                // -0.0 -> +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t o) {
  return __uint_as_float((o & 0x80000000u) ? (o ^ 0x80000000u) : ~o);
}

template <int KPL>
__global__ void __launch_bounds__(256) topk_kernel(const float* __restrict__ logits, const float* __restrict__ bias,
                                                   long long bias_stride, int32_t* __restrict__ topk_idx,
                                                   float* __restrict__ topk_w, int T, int E, int k, int score_fn,
                                                   int32_t* status, uint32_t* clear, size_t clear_words) {
  grid_dependency_sync();
  // optional side job for the fused layer: zero the membership bitmasks of the layout builder that
  // runs next, so that no memset sits between this kernel and it
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < clear_words; i += (size_t)gridDim.x * blockDim.x)
    clear[i] = 0u;
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  bool nonfinite = false;
  for (int t = blockIdx.x * warps_per_block + (threadIdx.x >> 5); t < T; t += gridDim.x * warps_per_block) {
    uint32_t key[KPL];
#pragma unroll
    for (int i = 0; i < KPL; ++i) {
      const int e = lane + 32 * i;
      if (e < E) {
        float v = __ldg(logits + (size_t)t * E + e);
        if (bias != nullptr) v = __fadd_rn(v, __ldg(bias + (size_t)t * bias_stride + e));
        key[i] = order_key(v, nonfinite);
      } else {
        key[i] = 0;  // below every real key (-inf maps to 0x007FFFFF)
      }
    }
    uint32_t my_e = 0;     // lane j keeps the j-th selected expert and its key
    float my_key = 0.f;
    for (int j = 0; j < k; ++j) {
      uint32_t best = 0;
      int best_i = 0;
#pragma unroll
      for (int i = 0; i < KPL; ++i)
        if (key[i] > best) { best = key[i]; best_i = i; }  // strict: lowest i (lowest expert) wins ties
      const uint32_t top = __reduce_max_sync(0xFFFFFFFFu, best);
      const uint32_t cand = (best == top) ? (uint32_t)(lane + 32 * best_i) : 0xFFFFFFFFu;
      const uint32_t win = __reduce_min_sync(0xFFFFFFFFu, cand);
      if ((int)(win & 31u) == lane) {
#pragma unroll
        for (int i = 0; i < KPL; ++i)
          if (i == (int)(win >> 5)) key[i] = 0;
      }
      if (lane == j) { my_e = win; my_key = key_value(top); }
    }
    // gate weights over the k selected keys (lanes 0..k-1)
    const float key0 = __shfl_sync(0xFFFFFFFFu, my_key, 0);
    float z = 0.f;
    if (lane < k) z = (score_fn == 0) ? expf(my_key - key0) : 1.f / (1.f + expf(-my_key));
    float sum = z;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
    if (lane < k) {
      topk_idx[(size_t)t * k + lane] = (int32_t)my_e;
      topk_w[(size_t)t * k + lane] = z / sum;
    }
  }
  if (__any_sync(0xFFFFFFFFu, nonfinite) && lane == 0) atomicOr(&status[ST_WARN], WARN_NONFINITE_LOGIT);
}

cudaError_t launch_topk(const Shape& s, const float* logits, const float* bias, int64_t bias_stride,
                        int32_t* topk_idx, float* topk_w, int32_t* status, cudaStream_t st, uint32_t* clear,
                        size_t clear_words) {
  if (s.T == 0) return cudaSuccess;
  const int warps = 8;
  int blocks = (s.T + warps - 1) / warps;
  const int cap = sm_count() * 8;
  if (blocks > cap) blocks = cap;
  const int kpl = (s.E + 31) / 32;
  ProfileScope prof(KID_TOPK, st);
#define TCMOE_TOPK(KPL)                                                                                      \
  launch_pdl(topk_kernel<KPL>, blocks, warps * 32, 0, st, logits, bias, (long long)bias_stride, topk_idx, topk_w, \
             s.T, s.E, s.k, s.score_fn, status, clear, clear_words)
  if (kpl <= 1) return TCMOE_TOPK(1);
  if (kpl <= 2) return TCMOE_TOPK(2);
  if (kpl <= 4) return TCMOE_TOPK(4);
  if (kpl <= 8) return TCMOE_TOPK(8);
  if (kpl <= 16) return TCMOE_TOPK(16);
  return TCMOE_TOPK(32);
#undef TCMOE_TOPK
}

}  // namespace tcmoe
