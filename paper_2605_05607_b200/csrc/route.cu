// Gate of the MoE layer (paper Sec. II-A: "topk experts selected by the gate network").
//   gate_logits_kernel : logits[T,E] = x[T,d] (bf16) * w_gate[d,E] (fp32), fp32 accumulation
//   topk_kernel        : key = logit + bias; k largest keys per token ordered by
//                        (key descending, expert index ascending); gate weights over the k keys
#include "common.cuh"

#include <cuda_bf16.h>

namespace tcmoe {

// ------------------------------------------------------------------------------------------------
// Gate logits: register-tiled fp32 GEMM.  256 threads; thread grid (256 / (BN/4)) x (BN/4);
// each thread owns TM x 4 outputs.  x tile is converted to fp32 and stored k-major in shared
// memory so that the inner product reads are conflict-free broadcasts.
// ------------------------------------------------------------------------------------------------
template <int BN>
struct GateCfg {
  static constexpr int TN = 4;
  static constexpr int TX = BN / TN;          // threads along experts
  static constexpr int TY = 256 / TX;         // threads along tokens
  static constexpr int BM = (BN >= 64) ? 64 : (BN >= 32 ? 64 : 128);
  static constexpr int TM = BM / TY;
  static constexpr int BK = 32;
};

template <int BN>
__global__ void __launch_bounds__(256) gate_logits_kernel(const __nv_bfloat16* __restrict__ x,
                                                          const float* __restrict__ wg,
                                                          float* __restrict__ logits, int T, int d, int E) {
  using C = GateCfg<BN>;
  constexpr int BM = C::BM, BK = C::BK, TM = C::TM, TN = C::TN;
  __shared__ float xs[BK][BM + 4];
  __shared__ float ws[BK][BN];
  const int tid = threadIdx.x;
  const int tx = tid % C::TX, ty = tid / C::TX;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < d; k0 += BK) {
    // x tile: BM rows x BK cols, 16-byte vectors of 8 bf16 (d % 8 == 0)
    for (int v = tid; v < BM * (BK / 8); v += 256) {
      const int r = v / (BK / 8), c = (v % (BK / 8)) * 8;
      const int row = m0 + r, col = k0 + c;
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (row < T && col < d) raw = __ldg(reinterpret_cast<const uint4*>(x + (size_t)row * d + col));
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f2 = __bfloat1622float2(p[q]);
        xs[c + 2 * q][r] = f2.x;
        xs[c + 2 * q + 1][r] = f2.y;
      }
    }
    for (int v = tid; v < BK * BN; v += 256) {
      const int kk = v / BN, nn = v % BN;
      const int row = k0 + kk, col = n0 + nn;
      ws[kk][nn] = (row < d && col < E) ? __ldg(wg + (size_t)row * E + col) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], b[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = xs[kk][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) b[j] = ws[kk][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int row = m0 + ty * TM + i;
    if (row >= T) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int col = n0 + tx * TN + j;
      if (col < E) logits[(size_t)row * E + col] = acc[i][j];
    }
  }
}

template <int BN>
static cudaError_t launch_gate_bn(const Shape& s, const void* x, const float* wg, float* logits, cudaStream_t st) {
  dim3 grid((s.T + GateCfg<BN>::BM - 1) / GateCfg<BN>::BM, (s.E + BN - 1) / BN);
  ProfileScope prof(KID_GATE, st);
  gate_logits_kernel<BN><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), wg, logits, s.T, s.d, s.E);
  return cudaGetLastError();
}

cudaError_t launch_gate_logits(const Shape& s, const void* x, const float* w_gate, float* logits, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  if (s.E <= 8) return launch_gate_bn<8>(s, x, w_gate, logits, st);
  if (s.E <= 32) return launch_gate_bn<32>(s, x, w_gate, logits, st);
  return launch_gate_bn<64>(s, x, w_gate, logits, st);
}

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
                                                   int32_t* status) {
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
                        int32_t* topk_idx, float* topk_w, int32_t* status, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  const int warps = 8;
  int blocks = (s.T + warps - 1) / warps;
  const int cap = sm_count() * 8;
  if (blocks > cap) blocks = cap;
  const int kpl = (s.E + 31) / 32;
  ProfileScope prof(KID_TOPK, st);
#define TCMOE_TOPK(KPL)                                                                                        \
  topk_kernel<KPL><<<blocks, warps * 32, 0, st>>>(logits, bias, (long long)bias_stride, topk_idx, topk_w, s.T, \
                                                  s.E, s.k, s.score_fn, status)
  if (kpl <= 1) TCMOE_TOPK(1);
  else if (kpl <= 2) TCMOE_TOPK(2);
  else if (kpl <= 4) TCMOE_TOPK(4);
  else if (kpl <= 8) TCMOE_TOPK(8);
  else if (kpl <= 16) TCMOE_TOPK(16);
  else TCMOE_TOPK(32);
#undef TCMOE_TOPK
  return cudaGetLastError();
}

}  // namespace tcmoe
