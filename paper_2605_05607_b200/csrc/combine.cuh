// Combine of ONE token by one warp (paper Sec. II-A aggregation; Sec. III-D reduction logic), shared by the
// combine kernel and by the Combine tasks of the tracker-paced layer kernel so that both produce the same bits.
// The k slots are visited group by group (ascending group, ascending slot inside a group): the rows of one
// group are summed first (the pre-reduction that the switch performs per output port), then the group partial
// joins the token's total; fp32 throughout.
#pragma once
#include "common.cuh"

#include <cuda_bf16.h>

namespace tcmoe {

__device__ __forceinline__ void add_bf16x8(float (&acc)[8], const uint4& raw, float w) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float2 f = __bfloat1622float2(p[q]);
    acc[2 * q] = fmaf(w, f.x, acc[2 * q]);
    acc[2 * q + 1] = fmaf(w, f.y, acc[2 * q + 1]);
  }
}
__device__ __forceinline__ uint4 pack_bf16x8(const float (&v)[8]) {
  uint4 out;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
  for (int q = 0; q < 4; ++q) p[q] = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
  return out;
}


// The row sums of one token for the 16-byte columns [v_begin, v_end): slots in (group, slot) order from s_row /
// s_dst / s_w, BATCH rows loaded at a time.
template <bool COHERENT, int BATCH>
__device__ __forceinline__ void combine_rows(const CombineArgs& c, int t, int lane, int kv, const int* s_row,
                                             const int* s_dst, const float* s_w, int v_begin, int v_end) {
  const int vec_per_row = c.vec_per_row;
  v_end = min(v_end, vec_per_row);   // [v_begin, v_end): the 16-byte columns of the row this warp sums
  for (int v = v_begin + lane; v < v_end; v += 32) {
    float total[8], part[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) { total[q] = 0.f; part[q] = 0.f; }
    int prev_dst = -1;
    for (int s0 = 0; s0 < kv; s0 += BATCH) {
      uint4 buf[BATCH];
#pragma unroll
      for (int q = 0; q < BATCH; ++q)   // all loads of the batch are in flight before the first use
        if (s0 + q < kv) {
          const uint4* src = c.o + (size_t)s_row[s0 + q] * vec_per_row + v;
          buf[q] = COHERENT ? __ldcg(src) : __ldcs(src);
        }
#pragma unroll
      for (int q = 0; q < BATCH; ++q) {
        if (s0 + q < kv) {
          const int dst = s_dst[s0 + q];
          if (dst != prev_dst && prev_dst >= 0) {   // a group is complete: emit its partial sum
            if (c.pg != nullptr) c.pg[(size_t)prev_dst * vec_per_row + v] = pack_bf16x8(part);
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) { total[cc] += part[cc]; part[cc] = 0.f; }
          }
          prev_dst = dst;
          add_bf16x8(part, buf[q], s_w[s0 + q]);
        }
      }
    }
    if (c.pg != nullptr && prev_dst >= 0) c.pg[(size_t)prev_dst * vec_per_row + v] = pack_bf16x8(part);
#pragma unroll
    for (int cc = 0; cc < 8; ++cc) total[cc] += part[cc];
    c.y[(size_t)t * vec_per_row + v] = pack_bf16x8(total);
  }
}

// s_row / s_dst / s_w: 32 entries each of shared memory owned by the calling warp.  [v_begin, v_end) restricts the
// call to a range of 16-byte columns (several warps may share one token: the order of additions per element is
// the same whoever sums it).  COHERENT: rows of o are read
// with loads that see what other thread blocks of the SAME kernel wrote (the tracker-paced kernel); otherwise
// streaming loads.  BATCH (2, 4 or 8): rows loaded at a time; any value is correct for any k, the one that matches
// k wastes no issue slots on absent slots (a top-2 layer through the 8-row form runs at a third of the bandwidth).
template <bool COHERENT, int BATCH>
__device__ __forceinline__ void combine_token(const CombineArgs& c, int t, int lane, int* s_row, int* s_dst, float* s_w,
                                              int v_begin = 0, int v_end = 0x7FFFFFFF) {
  const int k = c.k;
  // lane j < k owns slot j; order slots by (group, slot)
  int my_g = 0x7FFFFFFF, my_row = 0, my_dst = 0;
  float my_w = 1.f;
  if (lane < k) {
    const int e = __ldg(c.topk_idx + (size_t)t * k + lane);
    // e < 0: unused slot of a sparse top-k table, sorts behind every real slot and is not read.  An expert
    // index or a row outside its table (the layout builder reported it and wrote row -1) is skipped the
    // same way, so no table entry is ever used as an address unchecked.
    if (e >= 0 && e < c.E) {
      const int r = __ldg(c.pair_row + (size_t)t * k + lane);
      const int a = __ldg(c.al + (size_t)(e / c.m) * c.T + t);
      if (r >= 0 && r < c.n_rows && a >= 0) {
        my_g = e / c.m;
        my_row = r;
        my_dst = __ldg(c.group_offsets + my_g) + a;
        if (c.weighted) my_w = __ldg(c.topk_w + (size_t)t * k + lane);
      } else {
        report_error(c.status, DEV_INDEX_OUT_OF_RANGE, KID_COMBINE, t, r);
      }
    } else if (e >= c.E) {
      report_error(c.status, DEV_INDEX_OUT_OF_RANGE, KID_COMBINE, t, e);
    }
  }
  const int kv = __popc(__ballot_sync(0xFFFFFFFFu, lane < k && my_g != 0x7FFFFFFF));   // slots in use
  int my_pos = 0;  // number of slots that come before mine
  for (int j = 0; j < k; ++j) {
    const int gj = __shfl_sync(0xFFFFFFFFu, my_g, j);
    if (gj < my_g || (gj == my_g && j < lane)) ++my_pos;
  }
  __syncwarp();
  if (lane < k) { s_row[my_pos] = my_row; s_dst[my_pos] = my_dst; s_w[my_pos] = my_w; }
  __syncwarp();
  combine_rows<COHERENT, BATCH>(c, t, lane, kv, s_row, s_dst, s_w, v_begin, v_end);
  __syncwarp();
}

}  // namespace tcmoe
