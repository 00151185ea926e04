// Backward pass of the layer for fixed routing (paper Sec. VI-A evaluates training: forward + backward of the layer
// defined in Sec. II-A; gate weight applied at the expert output, Sec. III-C).  With
//     y[t] = sum_j w[t, j] * FFN_e(x[t]),   FFN_e(a) = (silu(a W1[e]) * (a W3[e])) W2[e],   e = topk_idx[t, j]
// and the routing (topk_idx, topk_w) held constant, the gradients of a loss with dL/dy = dy are
//     dO[r]  = w_r * dy[t_r]                       one row per (token, expert) pair, expert-sorted
//     dH     = dO . W2[e]^T
//     dA1    = dH * a3 * silu'(a1),  dA3 = dH * silu(a1)          (a1 = a W1, a3 = a W3 recomputed)
//     dXs    = dA1 . W1[e]^T + dA3 . W3[e]^T       dx[t] = sum of the token's rows of dXs (the Combine of the backward)
//     dW1[e] = Xs^T . dA1,  dW3[e] = Xs^T . dA3,  dW2[e] = H^T . dO      (contractions over the expert's rows)
//
// Row space.  Every row buffer of the backward pass uses PADDED expert segments: expert e starts at poff[e], a
// multiple of 64, and its unused tail rows are zero.  The weight-gradient GEMMs contract over rows in blocks of 64,
// so no block mixes two experts and nothing has to be masked; the row GEMMs treat pad rows as ordinary rows (zero in,
// zero out).
//
// Sequence (one stream, no host round trip; every GEMM is a tcgen05 kernel):
//   offsets -> gather (Dispatch of x and of w * dy into the padded per-expert layout) -> zero the pad rows
//   -> dH (CTA pairs, W2 read K-major in place) -> GEMM-1 recomputed with the backward SwiGLU epilogue (h, dA1, dA3)
//   -> dW2 -> dXs (CTA pairs, two-part K walk over (dA1, W1^T), (dA3, W3^T)) -> Combine into dx -> dW1, dW3
#include "ffn_common.cuh"

#include <cuda_bf16.h>

namespace tcmoe {
namespace {

// poff[e] = sum over e' < e of the row count of e' rounded up to 64
__global__ void __launch_bounds__(1024) bwd_offsets_kernel(const int32_t* __restrict__ expert_counts, int32_t* poff, int E) {
  grid_dependency_sync();
  __shared__ int buf[1024];
  const int i = threadIdx.x;
  buf[i] = (i < E) ? ((expert_counts[i] + 63) & ~63) : 0;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {
    int a = 0;
    if (i >= off) a = buf[i - off];
    __syncthreads();
    buf[i] += a;
    __syncthreads();
  }
  if (i < E) poff[i + 1] = buf[i];
  if (i == 0) poff[0] = 0;
}

// Token-centric: a warp reads x[t] and dy[t] once and writes, for each of the token's pairs, the row of xs and the
// row of dO = w * dy at the pair's padded row; it also records that row (pair_prow) for the Combine of dx.
__global__ void __launch_bounds__(256) bwd_gather_kernel(const uint4* __restrict__ x, const uint4* __restrict__ dy,
                                                         const int32_t* __restrict__ topk_idx,
                                                         const float* __restrict__ topk_w,
                                                         const int32_t* __restrict__ pair_row,
                                                         const int32_t* __restrict__ expert_offsets,
                                                         const int32_t* __restrict__ poff, uint4* __restrict__ xs,
                                                         uint4* __restrict__ dos, int32_t* __restrict__ pair_prow, int T,
                                                         int E, int k, int n_rows, int vec_per_row) {
  grid_dependency_sync();
  __shared__ int s_prow[8][32];
  __shared__ float s_w[8][32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int wpb = blockDim.x >> 5;
  for (int t = blockIdx.x * wpb + wid; t < T; t += gridDim.x * wpb) {
    int prow = -1;
    float w = 0.f;
    if (lane < k) {
      const int e = __ldg(topk_idx + (size_t)t * k + lane);
      const int r = __ldg(pair_row + (size_t)t * k + lane);
      if (e >= 0 && e < E && r >= 0 && r < n_rows) {
        prow = __ldg(poff + e) + (r - __ldg(expert_offsets + e));
        w = __ldg(topk_w + (size_t)t * k + lane);
      }
      pair_prow[(size_t)t * k + lane] = prow;
    }
    __syncwarp();
    s_prow[wid][lane] = prow;
    s_w[wid][lane] = w;
    __syncwarp();
    const uint4* xr = x + (size_t)t * vec_per_row;
    const uint4* dr = dy + (size_t)t * vec_per_row;
    for (int v = lane; v < vec_per_row; v += 32) {
      const uint4 xv = __ldcs(xr + v), dv = __ldcs(dr + v);
      const __nv_bfloat162* dp = reinterpret_cast<const __nv_bfloat162*>(&dv);
      float2 f[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) f[q] = __bfloat1622float2(dp[q]);
      for (int j = 0; j < k; ++j) {
        const int pr = s_prow[wid][j];
        if (pr < 0) continue;
        const float wj = s_w[wid][j];
        uint4 o;
        __nv_bfloat162* op = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int q = 0; q < 4; ++q) op[q] = __floats2bfloat162_rn(wj * f[q].x, wj * f[q].y);
        xs[(size_t)pr * vec_per_row + v] = xv;
        dos[(size_t)pr * vec_per_row + v] = o;
      }
    }
    __syncwarp();
  }
}

// rows [poff[e] + count[e], poff[e + 1]) of xs and dO are zero: one block per expert, a warp per pad row
__global__ void __launch_bounds__(256) bwd_zero_pads_kernel(const int32_t* __restrict__ expert_counts,
                                                            const int32_t* __restrict__ poff, uint4* __restrict__ xs,
                                                            uint4* __restrict__ dos, int vec_per_row) {
  grid_dependency_sync();
  const int e = blockIdx.x;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int lo = __ldg(poff + e) + __ldg(expert_counts + e), hi = __ldg(poff + e + 1);
  const uint4 z = make_uint4(0u, 0u, 0u, 0u);
  for (int r = lo + wid; r < hi; r += 8)
    for (int v = lane; v < vec_per_row; v += 32) {
      xs[(size_t)r * vec_per_row + v] = z;
      dos[(size_t)r * vec_per_row + v] = z;
    }
}

}  // namespace

// rows of every padded row buffer for a shape: all pairs plus at most 63 pad rows per expert
size_t bwd_row_capacity(const Shape& s) { return (size_t)s.T * s.k + 64 * (size_t)s.E; }

cudaError_t launch_layer_backward(const Shape& s, const BwdArgs& a, cudaStream_t st) {
  if (s.T == 0) {   // no rows: every weight gradient is zero
    cudaError_t err;
    const size_t n13 = (size_t)s.E * s.d * s.f * 2;
    if ((err = cudaMemsetAsync(a.dw1, 0, n13, st)) != cudaSuccess) return err;
    if ((err = cudaMemsetAsync(a.dw3, 0, n13, st)) != cudaSuccess) return err;
    return cudaMemsetAsync(a.dw2, 0, n13, st);
  }
  const long long R = (long long)bwd_row_capacity(s);
  const int vec = s.d / 8;
  cudaError_t err;
  if ((err = launch_pdl(bwd_offsets_kernel, 1, 1024, 0, st, a.L.expert_counts, a.poff, s.E)) != cudaSuccess) return err;
  if ((err = launch_tile_prefix(s, a.L.expert_counts, a.mt_prefix, a.mp_prefix, st)) != cudaSuccess) return err;
  int blocks = (s.T + 7) / 8;
  const int cap = sm_count() * 8;
  if (blocks > cap) blocks = cap;
  {
    ProfileScope prof(KID_BWD, st);
    if ((err = launch_pdl(bwd_gather_kernel, blocks, 256, 0, st, static_cast<const uint4*>(a.x),
                          static_cast<const uint4*>(a.dy), a.topk_idx, a.topk_w, a.L.pair_row, a.L.expert_offsets,
                          a.poff, static_cast<uint4*>(a.xs), static_cast<uint4*>(a.dos), a.pair_prow, s.T, s.E, s.k,
                          s.T * s.k, vec)) != cudaSuccess)
      return err;
  }
  if ((err = launch_pdl(bwd_zero_pads_kernel, s.E, 256, 0, st, a.L.expert_counts, a.poff, static_cast<uint4*>(a.xs),
                        static_cast<uint4*>(a.dos), vec)) != cudaSuccess)
    return err;

  CUtensorMap m_w1, m_w3, m_w1t, m_w3t, m_w2t, m_xs, m_do, m_da1, m_da3;
  CUtensorMap r_xs, r_h, r_do, r_da1, r_da3;
  if (!ffn::make_weight_map(&m_w1, a.w1, s.E, s.d, s.f) || !ffn::make_weight_map(&m_w3, a.w3, s.E, s.d, s.f) ||
      !ffn::make_weight_map_kmajor(&m_w1t, a.w1, s.E, s.d, s.f) || !ffn::make_weight_map_kmajor(&m_w3t, a.w3, s.E, s.d, s.f) ||
      !ffn::make_weight_map_kmajor(&m_w2t, a.w2, s.E, s.f, s.d) || !ffn::make_act_map(&m_xs, a.xs, R, s.d) ||
      !ffn::make_act_map(&m_do, a.dos, R, s.d) || !ffn::make_act_map(&m_da1, a.da1, R, s.f) ||
      !ffn::make_act_map(&m_da3, a.da3, R, s.f) || !ffn::make_rows_map_mn(&r_xs, a.xs, R, s.d) ||
      !ffn::make_rows_map_mn(&r_h, a.h, R, s.f) || !ffn::make_rows_map_mn(&r_do, a.dos, R, s.d) ||
      !ffn::make_rows_map_mn(&r_da1, a.da1, R, s.f) || !ffn::make_rows_map_mn(&r_da3, a.da3, R, s.f))
    return cudaErrorInvalidValue;

  // dH = dO . W2^T : [R, d] x [d, f], the gate weight is already inside dO
  ffn::GemmParams g{};
  g.out = static_cast<__nv_bfloat16*>(a.dh);
  g.out_ld = s.f;
  g.expert_offsets = a.poff;
  g.tile_prefix = a.mp_prefix;
  g.E = s.E;
  g.K = s.d;
  g.N = s.f;
  g.n_tiles = (s.f + 255) / 256;
  g.status = a.status;
  {
    ProfileScope prof(KID_GEMM2, st);
    if ((err = ffn::launch_bwd_dh(g, m_w2t, m_do, st)) != cudaSuccess) return err;
  }
  // GEMM-1 recomputed, backward SwiGLU epilogue: h, dA1, dA3
  ffn::GemmParams r{};
  r.out = static_cast<__nv_bfloat16*>(a.h);
  r.out2 = static_cast<__nv_bfloat16*>(a.da1);
  r.out3 = static_cast<__nv_bfloat16*>(a.da3);
  r.dh = static_cast<const __nv_bfloat16*>(a.dh);
  r.out_ld = s.f;
  r.expert_offsets = a.poff;
  r.tile_prefix = a.mp_prefix;
  r.E = s.E;
  r.K = s.d;
  r.N = s.f;
  r.n_tiles = (s.f + 127) / 128;
  r.status = a.status;
  {
    ProfileScope prof(KID_GEMM1, st);
    if ((err = ffn::launch_bwd_glu(r, m_w1, m_w3, m_xs, st)) != cudaSuccess) return err;
  }
  // dW2[e] = H^T . dO
  if ((err = ffn::launch_wgrad_pair(r_h, r_do, a.poff, a.dw2, s.E, s.f, s.d, a.status, st)) != cudaSuccess) return err;
  // dXs = dA1 . W1^T + dA3 . W3^T : [R, f] x [f, d], twice into one accumulator
  ffn::GemmParams q{};
  q.out = static_cast<__nv_bfloat16*>(a.dxs);
  q.out_ld = s.d;
  q.expert_offsets = a.poff;
  q.tile_prefix = a.mp_prefix;
  q.E = s.E;
  q.K = s.f;
  q.N = s.d;
  q.n_tiles = (s.d + 255) / 256;
  q.k_split = (s.f + ffn::BK - 1) / ffn::BK;
  q.status = a.status;
  {
    ProfileScope prof(KID_GEMM2, st);
    if ((err = ffn::launch_bwd_dx(q, m_w1t, m_w3t, m_da1, m_da3, st)) != cudaSuccess) return err;
  }
  // dx[t] = sum of the token's rows of dXs: the Combine stage on the padded row numbers, un-weighted
  Layout Lp = a.L;
  Lp.pair_row = a.pair_prow;
  Shape sc = s;
  sc.flags &= ~1;
  if ((err = launch_combine_rows(sc, a.dxs, Lp, a.topk_idx, nullptr, nullptr, a.dx, (int)R, a.status, st)) != cudaSuccess)
    return err;
  // dW1[e] = Xs^T . dA1,  dW3[e] = Xs^T . dA3
  if ((err = ffn::launch_wgrad_pair(r_xs, r_da1, a.poff, a.dw1, s.E, s.d, s.f, a.status, st)) != cudaSuccess) return err;
  return ffn::launch_wgrad_pair(r_xs, r_da3, a.poff, a.dw3, s.E, s.d, s.f, a.status, st);
}

}  // namespace tcmoe
