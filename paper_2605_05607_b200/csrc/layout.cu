// Dispatch layout, dispatch and combine (paper Sec. III-D: switch routing rule
// group = expert / experts_per_group, AL tables built by a running counter, MV translation;
// Sec. IV-B TID table; Sec. III-C un-weighted reduction in Combine).
//
// The hardware of the paper hands out layout rows in arrival order.  Here the order is fixed to
// ascending token index so that the layout is a pure function of topk_idx: membership bitmasks
// (one bit per (expert, token) and per (group, token)) are built with order-independent atomicOr,
// an exclusive popcount scan along each mask row gives every token its rank, and a fill pass
// turns ranks into the row tables.  No atomics touch the result arrays.
#include "combine.cuh"

namespace tcmoe {

// ---- K2a: membership masks -------------------------------------------------------------------
__global__ void __launch_bounds__(256) build_masks_kernel(const int32_t* __restrict__ topk_idx, uint32_t* emask,
                                                          uint32_t* gmask, int T, int E, int k, int m, int W,
                                                          int32_t* status, int sparse) {
  grid_dependency_sync();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;  // warp w covers tokens 32w .. 32w+31
  const int lane = threadIdx.x & 31;
  const int word = t >> 5;
  const bool live = t < T;
  for (int j = 0; j < k; ++j) {
    int e = live ? __ldg(topk_idx + (size_t)t * k + j) : -1;
    if (live && (e < 0 || e >= E)) {
      if (!(sparse && e == -1)) report_error(status, DEV_INDEX_OUT_OF_RANGE, KID_MASKS, t, e);   // -1: unused slot
      e = -1;
    }
    // lanes that picked the same expert (group) fold their bits into one atomicOr
    const unsigned same_e = __match_any_sync(0xFFFFFFFFu, e);
    if (e >= 0 && lane == __ffs(same_e) - 1) atomicOr(&emask[(size_t)e * W + word], same_e);
    const int g = (e >= 0) ? e / m : -1;
    const unsigned same_g = __match_any_sync(0xFFFFFFFFu, g);
    if (g >= 0 && lane == __ffs(same_g) - 1) atomicOr(&gmask[(size_t)g * W + word], same_g);
  }
}

// ---- K2b: exclusive popcount prefix along every mask row; row totals -> counts ------------------
__global__ void __launch_bounds__(256) scan_masks_kernel(const uint32_t* __restrict__ emask,
                                                         const uint32_t* __restrict__ gmask, int32_t* eprefix,
                                                         int32_t* gprefix, int32_t* expert_counts,
                                                         int32_t* group_counts, int E, int W) {
  grid_dependency_sync();
  __shared__ int warp_sum[8];
  __shared__ int running_s;
  const int row = blockIdx.x;
  const uint32_t* mask = (row < E) ? emask + (size_t)row * W : gmask + (size_t)(row - E) * W;
  int32_t* prefix = (row < E) ? eprefix + (size_t)row * W : gprefix + (size_t)(row - E) * W;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x == 0) running_s = 0;
  __syncthreads();
  for (int base = 0; base < W; base += 256) {
    const int i = base + threadIdx.x;
    const int c = (i < W) ? __popc(mask[i]) : 0;
    int incl = c;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xFFFFFFFFu, incl, off);
      if (lane >= off) incl += n;
    }
    if (lane == 31) warp_sum[wid] = incl;
    __syncthreads();
    int warp_base = 0;
    for (int w = 0; w < wid; ++w) warp_base += warp_sum[w];
    const int running = running_s;
    if (i < W) prefix[i] = running + warp_base + incl - c;
    __syncthreads();
    if (threadIdx.x == 255) running_s = running + warp_base + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    if (row < E) expert_counts[row] = running_s;
    else group_counts[row - E] = running_s;
  }
}

// ---- K2c: offsets (exclusive scans over experts / groups) and the GEMM tile prefixes --------------
__global__ void __launch_bounds__(1024) offsets_kernel(const int32_t* __restrict__ expert_counts,
                                                       const int32_t* __restrict__ group_counts,
                                                       int32_t* expert_offsets, int32_t* group_offsets,
                                                       int32_t* mt_prefix, int32_t* mp_prefix, int E, int G) {
  grid_dependency_sync();
  __shared__ int buf[4][1024];
  const int i = threadIdx.x;
  const int ce = (i < E) ? expert_counts[i] : 0;
  const int cg = (i < G) ? group_counts[i] : 0;
  buf[0][i] = ce;
  buf[1][i] = cg;
  buf[2][i] = (ce + 127) >> 7;   // 128-row tiles (GEMM-1)
  buf[3][i] = (ce + 255) >> 8;   // 256-row CTA-pair tiles (GEMM-2)
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {  // Hillis-Steele inclusive scan, three lanes at once
    int a = 0, b = 0, c = 0, d = 0;
    if (i >= off) { a = buf[0][i - off]; b = buf[1][i - off]; c = buf[2][i - off]; d = buf[3][i - off]; }
    __syncthreads();
    buf[0][i] += a; buf[1][i] += b; buf[2][i] += c; buf[3][i] += d;
    __syncthreads();
  }
  if (i < E) { expert_offsets[i + 1] = buf[0][i]; mt_prefix[i + 1] = buf[2][i]; mp_prefix[i + 1] = buf[3][i]; }
  if (i < G) group_offsets[i + 1] = buf[1][i];
  if (i == 0) { expert_offsets[0] = 0; group_offsets[0] = 0; mt_prefix[0] = 0; mp_prefix[0] = 0; }
}

// ---- K2d: ranks -> row tables ----------------------------------------------------------------
__global__ void __launch_bounds__(256) fill_layout_kernel(const int32_t* __restrict__ topk_idx, Layout L,
                                                          LayoutScratch sc, int T, int E, int k, int G, int m) {
  grid_dependency_sync();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  const int word = t >> 5;
  const uint32_t below = (1u << (t & 31)) - 1u;
  for (int g = 0; g < G; ++g) {
    const uint32_t bits = sc.gmask[(size_t)g * sc.W + word];
    int a = -1;
    if (bits >> (t & 31) & 1u) {
      a = sc.gprefix[(size_t)g * sc.W + word] + __popc(bits & below);
      L.disp_token[L.group_offsets[g] + a] = t;  // TID table entry of the allocated row
    }
    L.al[(size_t)g * T + t] = a;
  }
  for (int j = 0; j < k; ++j) {
    const int e = __ldg(topk_idx + (size_t)t * k + j);
    if (e < 0 || e >= E) {          // unused slot (sparse top-k), or an index build_masks_kernel reported
      L.pair_row[(size_t)t * k + j] = -1;
      continue;
    }
    const int rank = sc.eprefix[(size_t)e * sc.W + word] + __popc(sc.emask[(size_t)e * sc.W + word] & below);
    const int r = L.expert_offsets[e] + rank;
    const int g = e / m;
    const uint32_t gbits = sc.gmask[(size_t)g * sc.W + word];
    const int a = sc.gprefix[(size_t)g * sc.W + word] + __popc(gbits & below);
    L.pair_row[(size_t)t * k + j] = r;
    L.row_pair[r] = t * k + j;
    L.row_src[r] = L.group_offsets[g] + a;
  }
}

// exclusive prefixes of 128-row tiles and 256-row pair tiles per expert, from the counts alone
__global__ void __launch_bounds__(1024) tile_prefix_kernel(const int32_t* __restrict__ expert_counts,
                                                           int32_t* mt_prefix, int32_t* mp_prefix, int E) {
  grid_dependency_sync();
  __shared__ int buf[2][1024];
  const int i = threadIdx.x;
  const int c = (i < E) ? expert_counts[i] : 0;
  buf[0][i] = (c + 127) >> 7;
  buf[1][i] = (c + 255) >> 8;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {
    int a = 0, b = 0;
    if (i >= off) { a = buf[0][i - off]; b = buf[1][i - off]; }
    __syncthreads();
    buf[0][i] += a; buf[1][i] += b;
    __syncthreads();
  }
  if (i < E) { mt_prefix[i + 1] = buf[0][i]; mp_prefix[i + 1] = buf[1][i]; }
  if (i == 0) { mt_prefix[0] = 0; mp_prefix[0] = 0; }
}

cudaError_t launch_tile_prefix(const Shape& s, const int32_t* expert_counts, int32_t* mt_prefix, int32_t* mp_prefix,
                               cudaStream_t st) {
  return launch_pdl(tile_prefix_kernel, 1, 1024, 0, st, expert_counts, mt_prefix, mp_prefix, s.E);
}

cudaError_t launch_layout(const Shape& s, const int32_t* topk_idx, const Layout& L, const LayoutScratch& sc,
                          int32_t* status, cudaStream_t st, bool masks_cleared) {
  const int m = s.E / s.G;
  cudaError_t err;
  if (!masks_cleared &&
      (err = cudaMemsetAsync(sc.emask, 0, sizeof(uint32_t) * (size_t)(s.E + s.G) * sc.W, st)) != cudaSuccess)
    return err;  // emask and gmask are adjacent
  const int tb = (s.T + 255) / 256;
  if (s.T > 0 && (err = launch_pdl(build_masks_kernel, tb, 256, 0, st, topk_idx, sc.emask, sc.gmask, s.T, s.E, s.k,
                                   m, sc.W, status, (s.flags & 4) ? 1 : 0)) != cudaSuccess)
    return err;
  if ((err = launch_pdl(scan_masks_kernel, s.E + s.G, 256, 0, st, sc.emask, sc.gmask, sc.eprefix, sc.gprefix,
                        L.expert_counts, L.group_counts, s.E, sc.W)) != cudaSuccess)
    return err;
  if ((err = launch_pdl(offsets_kernel, 1, 1024, 0, st, L.expert_counts, L.group_counts, L.expert_offsets,
                        L.group_offsets, sc.mt_prefix, sc.mp_prefix, s.E, s.G)) != cudaSuccess)
    return err;
  if (s.T > 0) return launch_pdl(fill_layout_kernel, tb, 256, 0, st, topk_idx, L, sc, s.T, s.E, s.k, s.G, m);
  return cudaSuccess;
}

// ---- K3: dispatch ------------------------------------------------------------------------------
// Token-centric: a warp reads (its part of) row x[t] once (16-byte vectors) and writes one copy per distinct
// group the token touches - the single-HBM image of "send once, the switch replicates per port".  With few tokens
// a row is split over `parts` warps (see combine_kernel).
__global__ void __launch_bounds__(256) dispatch_kernel(const uint4* __restrict__ x, uint4* __restrict__ xg,
                                                       const int32_t* __restrict__ al,
                                                       const int32_t* __restrict__ group_offsets, int T, int G,
                                                       int vec_per_row, int parts, int vec_per_part) {
  grid_dependency_sync();
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const long long units = (long long)T * parts;
  for (long long u = (long long)blockIdx.x * wpb + (threadIdx.x >> 5); u < units; u += (long long)gridDim.x * wpb) {
    const int t = (int)(u / parts), part = (int)(u % parts);
    const int v_lo = part * vec_per_part, v_hi = min(vec_per_row, v_lo + vec_per_part);
    const uint4* src = x + (size_t)t * vec_per_row;
    for (int g0 = 0; g0 < G; g0 += 32) {
      const int g = g0 + lane;
      int dst_row = -1;
      if (g < G) {
        const int a = __ldg(al + (size_t)g * T + t);
        if (a >= 0) dst_row = __ldg(group_offsets + g) + a;
      }
      unsigned live = __ballot_sync(0xFFFFFFFFu, dst_row >= 0);
      if (!live) continue;
      for (int v0 = v_lo; v0 < v_hi; v0 += 128) {
        uint4 buf[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int v = v0 + q * 32 + lane;
          if (v < v_hi) buf[q] = __ldcs(src + v);
        }
        for (unsigned rem = live; rem; rem &= rem - 1) {
          const int row = __shfl_sync(0xFFFFFFFFu, dst_row, __ffs(rem) - 1);
          uint4* dst = xg + (size_t)row * vec_per_row;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int v = v0 + q * 32 + lane;
            if (v < v_hi) __stcs(dst + v, buf[q]);
          }
        }
      }
    }
  }
}

static int row_parts(int T, int vec_per_row);

cudaError_t launch_dispatch(const Shape& s, const void* x, const Layout& L, void* xg, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  const int vec = s.d / 8;
  const int parts = row_parts(s.T, vec);
  const int vec_per_part = ((vec + parts - 1) / parts + 127) & ~127;   // whole 128-vector steps per part
  long long blocks = ((long long)s.T * parts + 7) / 8;
  const long long cap = (long long)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  ProfileScope prof(KID_DISPATCH, st);
  return launch_pdl(dispatch_kernel, (unsigned)blocks, 256, 0, st, static_cast<const uint4*>(x), static_cast<uint4*>(xg),
                    L.al, L.group_offsets, s.T, s.G, vec, parts, vec_per_part);
}

// ---- K3b: dispatch into the per-expert layout tensors ----------------------------------------------
// xs[r, :] = src[gather_idx[r] / gather_div, :] for every expert-sorted row r: the dense per-expert buffers that
// the destination's memory manager fills in the paper (Sec. III-D: one AL sub-table per local expert), which is
// what lets GEMM-1 read its rows as plain TMA tiles.  One warp per row, 16-byte vectors; the number of rows in
// use is read from the device (expert_offsets[E]).
__global__ void __launch_bounds__(256) permute_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ xs,
                                                           const int32_t* __restrict__ gather_idx, int gather_div,
                                                           const int32_t* __restrict__ expert_offsets, int E,
                                                           int src_rows, int vec_per_row, int32_t* status) {
  grid_dependency_sync();
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int rows = __ldg(expert_offsets + E);
  for (int r = blockIdx.x * wpb + (threadIdx.x >> 5); r < rows; r += gridDim.x * wpb) {
    int idx = __ldg(gather_idx + r);
    if (gather_div > 1) idx /= gather_div;
    uint4* dst = xs + (size_t)r * vec_per_row;
    if (idx < 0 || idx >= src_rows) {   // a table entry that is no row of the source: reported, the row zero-filled
      if (lane == 0) report_error(status, DEV_INDEX_OUT_OF_RANGE, KID_DISPATCH, r, idx);
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0u, 0u, 0u, 0u);
      continue;
    }
    const uint4* from = src + (size_t)idx * vec_per_row;
    for (int v0 = 0; v0 < vec_per_row; v0 += 128) {
      uint4 buf[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int v = v0 + q * 32 + lane;
        if (v < vec_per_row) buf[q] = __ldg(from + v);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int v = v0 + q * 32 + lane;
        if (v < vec_per_row) dst[v] = buf[q];
      }
    }
  }
}

cudaError_t launch_permute_rows(const Shape& s, const void* src, int src_rows, const int32_t* gather_idx,
                                int gather_div, const int32_t* expert_offsets, void* xs, int32_t* status,
                                cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  long long blocks = ((long long)s.T * s.k + 7) / 8;
  const long long cap = (long long)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  ProfileScope prof(KID_DISPATCH, st);
  return launch_pdl(permute_rows_kernel, (unsigned)blocks, 256, 0, st, static_cast<const uint4*>(src),
                    static_cast<uint4*>(xs), gather_idx, gather_div, expert_offsets, s.E, src_rows, s.d / 8, status);
}

// ---- K5: combine -----------------------------------------------------------------------------
// One warp per (token, column part); the per-token work is combine_token() (combine.cuh).  With few tokens a row
// is split over `parts` warps so that enough loads are in flight to reach the memory bandwidth (one warp per token
// leaves a 4096-token batch at a third of it).
template <int BATCH>
__global__ void __launch_bounds__(256, 3) combine_kernel(const CombineArgs c, int parts, int vec_per_part) {
  grid_dependency_sync();
  __shared__ int s_row[8][32];   // per warp: expert-sorted row of the slot at sorted position p
  __shared__ int s_dst[8][32];   // dispatched row (t, g) of that slot's group
  __shared__ float s_w[8][32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int wpb = blockDim.x >> 5;
  const long long units = (long long)c.T * parts;
  for (long long u = (long long)blockIdx.x * wpb + wid; u < units; u += (long long)gridDim.x * wpb) {
    const int t = (int)(u / parts), part = (int)(u % parts);
    combine_token<false, BATCH>(c, t, lane, s_row[wid], s_dst[wid], s_w[wid], part * vec_per_part,
                                (part + 1) * vec_per_part);
  }
}

// parts of a row so that about 32 warps per SM exist even for small batches (at most 8, at least 4 vectors per lane)
static int row_parts(int T, int vec_per_row) {
  int parts = 1;
  while (parts < 8 && (long long)T * parts < 32ll * sm_count() * 2 && vec_per_row / (parts * 2) >= 128) parts *= 2;
  return parts;
}

cudaError_t launch_combine(const Shape& s, const void* o, const Layout& L, const int32_t* topk_idx,
                           const float* topk_w, void* pg, void* y, int32_t* status, cudaStream_t st) {
  return launch_combine_rows(s, o, L, topk_idx, topk_w, pg, y, s.T * s.k, status, st);
}

// n_rows: rows of `o` (L.pair_row entries outside [0, n_rows) are reported and skipped)
cudaError_t launch_combine_rows(const Shape& s, const void* o, const Layout& L, const int32_t* topk_idx,
                                const float* topk_w, void* pg, void* y, int n_rows, int32_t* status, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  const int vec = s.d / 8;
  const int parts = row_parts(s.T, vec);
  const int vec_per_part = ((vec + parts - 1) / parts + 31) & ~31;   // whole warp-strides per part
  long long blocks = ((long long)s.T * parts + 7) / 8;
  const long long cap = (long long)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  ProfileScope prof(KID_COMBINE, st);
  CombineArgs c{static_cast<const uint4*>(o), static_cast<uint4*>(y), static_cast<uint4*>(pg), topk_idx, topk_w,
                L.pair_row, L.al, L.group_offsets, s.T, s.E, s.k, s.E / s.G, vec, (s.flags & 1) ? 1 : 0,
                n_rows, status};
  if (s.k <= 2) return launch_pdl(combine_kernel<2>, (unsigned)blocks, 256, 0, st, c, parts, vec_per_part);
  if (s.k <= 4) return launch_pdl(combine_kernel<4>, (unsigned)blocks, 256, 0, st, c, parts, vec_per_part);
  return launch_pdl(combine_kernel<8>, (unsigned)blocks, 256, 0, st, c, parts, vec_per_part);
}

// Last step of the layer when Combine ran inside GEMM-2's epilogue: the fp32 token accumulators
// become the bf16 output, 8 elements per thread.
__global__ void __launch_bounds__(256) round_rows_kernel(const float4* __restrict__ acc, uint4* __restrict__ y,
                                                         size_t n_vec) {
  grid_dependency_sync();
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
    const float4 a = __ldcs(acc + 2 * i), b = __ldcs(acc + 2 * i + 1);
    uint4 q;
    __nv_bfloat162 v;
    v = __floats2bfloat162_rn(a.x, a.y); q.x = *reinterpret_cast<uint32_t*>(&v);
    v = __floats2bfloat162_rn(a.z, a.w); q.y = *reinterpret_cast<uint32_t*>(&v);
    v = __floats2bfloat162_rn(b.x, b.y); q.z = *reinterpret_cast<uint32_t*>(&v);
    v = __floats2bfloat162_rn(b.z, b.w); q.w = *reinterpret_cast<uint32_t*>(&v);
    y[i] = q;
  }
}

cudaError_t launch_round_rows(const Shape& s, const float* acc, void* y, cudaStream_t st) {
  const size_t n_vec = (size_t)s.T * s.d / 8;
  if (n_vec == 0) return cudaSuccess;
  size_t blocks = (n_vec + 255) / 256;
  const size_t cap = (size_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  ProfileScope prof(KID_COMBINE, st);
  return launch_pdl(round_rows_kernel, (unsigned)blocks, 256, 0, st, reinterpret_cast<const float4*>(acc),
                    static_cast<uint4*>(y), n_vec);
}

}  // namespace tcmoe
