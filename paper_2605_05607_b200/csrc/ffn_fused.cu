// Expert FFN as ONE persistent kernel paced by a tile tracker (paper Sec. IV "token-centric kernel fusion":
// tiles of 128 tokens move through the stages of the layer as soon as the stage before has produced them;
// Sec. IV-B/C: tracker tables record which tiles are complete, persistent thread blocks poll them, with a
// synchronisation tile size of 128 tokens, Sec. VII-C).
//
// Tasks are GEMM-1 tiles (128 rows x 128 columns of h: gathered A, W1 | W3, SwiGLU epilogue) and GEMM-2 tiles
// (128 rows x 256 columns of o: A = rows of h, W2, gate weight in the epilogue), both on the single-CTA UMMA
// form (all tcgen05 instructions of a kernel share one cta_group).  The task list interleaves them by blocks of
// up to 16 row tiles of one expert:   G1(b0) G1(b1) G2(b0) G1(b2) G2(b1) ... G2(last)
// so that a GEMM-2 tile is scheduled one block after the GEMM-1 tiles it depends on.  The tracker is one
// counter per 128-row tile of h: every epilogue warp of a GEMM-1 tile adds 1 after its rows are stored
// (release); the gather warps of a GEMM-2 tile wait until the counter shows all 4 * n1 parts (acquire).  Every
// dependency points to an earlier task and every CTA takes its tasks in order, so the waits cannot form a
// cycle; they are bounded all the same.
//
// Pipeline, barriers and epilogues are those of the two separate kernels (ffn_gemm1.cu).  On one GPU this
// form removes the launch boundary between the GEMMs and lets GEMM-2 read h while it is still in L2; it gives
// up the CTA-pair form of GEMM-2.  Measured against the two-kernel path in the design notes.
#include "ffn_common.cuh"

#include <atomic>

namespace tcmoe {
namespace ffn {
namespace {

constexpr int NSTAGE = 4;
constexpr int A_BYTES = BM * BK * 2;         // 16 KiB
constexpr int B_BYTES = UMMA_N * BK * 2;     // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_BARS = 2 * NSTAGE + 4;
constexpr int STAGE_OUT_WARP = 32 * 144;
constexpr int SMEM_BYTES = 1024 + NSTAGE * STAGE_BYTES + NUM_BARS * 8 + 64 + 4 * STAGE_OUT_WARP;
constexpr int THREADS = 320;
constexpr int GATHER_THREADS = 128;
constexpr int M_BLOCK = 16;                  // row tiles per task block
constexpr uint32_t IDESC = idesc_bf16(BM);

struct Task {
  int type;        // 0: GEMM-1 tile, 1: GEMM-2 tile
  int e, n0, row0, rows;
  int mt_global;   // index of the 128-row tile of h among all tiles (tracker slot)
};

__device__ __forceinline__ Task decode_task(int w, const FusedParams& p, const int32_t* blk_start,
                                            const int4* blk_info, int nb) {
  int lo = 0, hi = nb;   // blk_start[lo] <= w < blk_start[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(blk_start + mid) <= w) lo = mid; else hi = mid;
  }
  const int4 info = __ldg(blk_info + lo);   // {type, expert, first row tile, row tiles}
  const int local = w - __ldg(blk_start + lo);
  Task t;
  t.type = info.x;
  t.e = info.y;
  const int mt = info.z + local % info.w;     // row tile fastest: CTAs running together share the weight tile
  t.n0 = (local / info.w) * (t.type ? 256 : 128);
  const int e0 = __ldg(p.expert_offsets + t.e), e1 = __ldg(p.expert_offsets + t.e + 1);
  t.row0 = e0 + mt * BM;
  t.rows = min(BM, e1 - t.row0);
  t.mt_global = __ldg(p.mt_prefix + t.e) + mt;
  return t;
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__global__ void __launch_bounds__(THREADS, 1)
ffn_fused_kernel(const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w3,
                 const __grid_constant__ CUtensorMap map_w2, const FusedParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NSTAGE * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  int* abort_s = reinterpret_cast<int*>(tmem_slot + 1);
  const uint32_t stage_base = ptx::smem_u32(tmem_slot + 16);   // 16-byte aligned

  const uint32_t smem_base = ptx::smem_u32(smem);
  const uint32_t bar_base = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (NSTAGE + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * NSTAGE + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * NSTAGE + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), GATHER_THREADS + 1);   // every gather thread's copies + the TMA thread (expect_tx)
      ptx::mbar_init(empty_bar(s), 1);                   // tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tfull_bar(b), 1);      // tcgen05.commit
      ptx::mbar_init(tempty_bar(b), 4);     // one lane per epilogue warp
    }
    ptx::fence_mbar_init();
  }
  if (warp == 4 && lane == 0) {
    ptx::prefetch_tensormap(&map_w1);
    ptx::prefetch_tensormap(&map_w3);
    ptx::prefetch_tensormap(&map_w2);
  }
  if (warp == 5) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
    ptx::tmem_relinquish();
  }
  grid_dependency_sync();   // nothing above touches global data
  if (threadIdx.x == 0) *abort_s = p.status[ST_ABORT];
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Task list of this CTA.  Default: every CTA walks the interleaved list (tasks blockIdx, blockIdx + grid, ...).
  // SM partition (Sec. IV: thread blocks are divided among the stages): the first `p.part_g1` CTAs take only
  // GEMM-1 tiles, the others only GEMM-2 tiles, each group walking the list of its own kind; the GEMM-2 group is
  // paced purely by the tracker, the GEMM-1 group never waits.
  const bool part = p.part_g1 > 0;
  const int kind = part ? ((int)blockIdx.x < p.part_g1 ? 0 : 1) : 0;
  const int32_t* tbl_start = part ? p.blk_start + (size_t)(1 + kind) * p.tbl_stride : p.blk_start;
  const int4* tbl_info = part ? p.blk_info + (size_t)(1 + kind) * p.tbl_stride : p.blk_info;
  const int nb = __ldg(p.n_blocks + (part ? 1 + kind : 0));
  const int total = __ldg(tbl_start + nb);
  const int first = part ? (kind ? (int)blockIdx.x - p.part_g1 : (int)blockIdx.x) : (int)blockIdx.x;
  const int stride = part ? (kind ? (int)gridDim.x - p.part_g1 : p.part_g1) : (int)gridDim.x;
  const int KB1 = (p.d + BK - 1) / BK, KB2 = (p.f + BK - 1) / BK;
  volatile int* abort_flag = abort_s;
  const volatile int* global_abort = p.status + ST_ABORT;

  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, KID_GEMM1, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };

  if (warp < 4) {
    // ================================ epilogue ================================
    int tl = 0;
    for (int w = first; w < total && !*abort_flag; w += stride, ++tl) {
      const Task t = decode_task(w, p, tbl_start, tbl_info, nb);
      const int buf = tl & 1;
      if (!ptx::mbar_wait_warp<true>(tfull_bar(buf), (tl >> 1) & 1, abort_flag, global_abort)) { timeout(1); break; }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UMMA_N);
      // rows are transposed through shared memory, 64 output columns at a time, and stored as whole
      // 128-byte segments (8 lanes per row, 4 rows per instruction)
      const uint32_t stage = stage_base + (uint32_t)(warp * STAGE_OUT_WARP);
      const int srow = lane >> 3, piece = lane & 7;
      if (t.type == 1) {
        // ---- GEMM-2 tile: o = gate weight * acc, 256 columns
        const int lrow = warp * 32 + lane;
        float wr = 1.f;
        if (lrow < t.rows && p.topk_w != nullptr) wr = __ldg(p.topk_w + __ldg(p.row_pair + (size_t)t.row0 + lrow));
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t acc0[32], acc1[32];
          ptx::tmem_ld32(taddr + cc * 64, acc0);
          ptx::tmem_ld32(taddr + cc * 64 + 32, acc1);
          ptx::tmem_ld_wait_on(acc0);
          ptx::tmem_ld_wait_on(acc1);
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            ptx::st_shared_v4(stage + lane * 144 + v * 16,
                              pack2(wr * __uint_as_float(acc0[v * 8]), wr * __uint_as_float(acc0[v * 8 + 1])),
                              pack2(wr * __uint_as_float(acc0[v * 8 + 2]), wr * __uint_as_float(acc0[v * 8 + 3])),
                              pack2(wr * __uint_as_float(acc0[v * 8 + 4]), wr * __uint_as_float(acc0[v * 8 + 5])),
                              pack2(wr * __uint_as_float(acc0[v * 8 + 6]), wr * __uint_as_float(acc0[v * 8 + 7])));
            ptx::st_shared_v4(stage + lane * 144 + 64 + v * 16,
                              pack2(wr * __uint_as_float(acc1[v * 8]), wr * __uint_as_float(acc1[v * 8 + 1])),
                              pack2(wr * __uint_as_float(acc1[v * 8 + 2]), wr * __uint_as_float(acc1[v * 8 + 3])),
                              pack2(wr * __uint_as_float(acc1[v * 8 + 4]), wr * __uint_as_float(acc1[v * 8 + 5])),
                              pack2(wr * __uint_as_float(acc1[v * 8 + 6]), wr * __uint_as_float(acc1[v * 8 + 7])));
          }
          __syncwarp();
          const int col = t.n0 + cc * 64 + piece * 8;
          if (col < p.d) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = i * 4 + srow;
              if (warp * 32 + r < t.rows) {
                const uint4 q = ptx::ld_shared_v4(stage + r * 144 + piece * 16);
                *reinterpret_cast<uint4*>(p.o + (size_t)(t.row0 + warp * 32 + r) * (size_t)p.d + col) = q;
              }
            }
          }
          __syncwarp();
        }
      } else {
        // ---- GEMM-1 tile: SwiGLU of the W1 / W3 halves, 128 columns of h
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t a1[32], a3[32];
          ptx::tmem_ld32(taddr + c * 32, a1);
          ptx::tmem_ld32(taddr + 128 + c * 32, a3);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t q[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = v * 8 + 2 * i;
              q[i] = pack2(silu_mul(__uint_as_float(a1[j]), __uint_as_float(a3[j])),
                           silu_mul(__uint_as_float(a1[j + 1]), __uint_as_float(a3[j + 1])));
            }
            ptx::st_shared_v4(stage + lane * 144 + (c & 1) * 64 + v * 16, q[0], q[1], q[2], q[3]);
          }
          if (c & 1) {
            __syncwarp();
            const int col = t.n0 + (c - 1) * 32 + piece * 8;
            if (col < p.f) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int r = i * 4 + srow;
                if (warp * 32 + r < t.rows) {
                  const uint4 q = ptx::ld_shared_v4(stage + r * 144 + piece * 16);
                  *reinterpret_cast<uint4*>(p.h + (size_t)(t.row0 + warp * 32 + r) * (size_t)p.f + col) = q;
                }
              }
            }
            __syncwarp();
          }
        }
        // tracker: this warp's 32 rows x 128 columns of the h tile are stored
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(p.done + t.mt_global, 1);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(buf));
    }
  } else if (warp == 4) {
    // ================================ TMA producer (weights) ================================
    if (lane == 0) {
      uint32_t it = 0;
      for (int w = first; w < total && !*abort_flag; w += stride) {
        const Task t = decode_task(w, p, tbl_start, tbl_info, nb);
        const int KB = t.type ? KB2 : KB1;
        const CUtensorMap* lo_map = t.type ? &map_w2 : &map_w1;
        const CUtensorMap* hi_map = t.type ? &map_w2 : &map_w3;
        const int hi_n = t.type ? t.n0 + 128 : t.n0;
        bool ok = true;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag, global_abort)) {
            timeout(2); ok = false; break;
          }
          const uint32_t sb = smem_base + s * STAGE_BYTES + A_BYTES;
          ptx::mbar_arrive_expect_tx(full_bar(s), B_BYTES);
          const int k0 = kb * BK;
          ptx::tma_load_3d(sb, lo_map, full_bar(s), t.n0, k0, t.e);
          ptx::tma_load_3d(sb + 8192, lo_map, full_bar(s), t.n0 + 64, k0, t.e);
          ptx::tma_load_3d(sb + 16384, hi_map, full_bar(s), hi_n, k0, t.e);
          ptx::tma_load_3d(sb + 24576, hi_map, full_bar(s), hi_n + 64, k0, t.e);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    // ================================ UMMA issuer ================================
    if (lane == 0) {
      const uint64_t a_base = desc_base(16, 1024);
      const uint64_t b_base = desc_base(BK * 128, 1024);
      uint32_t it = 0;
      int tl = 0;
      for (int w = first; w < total && !*abort_flag; w += stride, ++tl) {
        const Task t = decode_task(w, p, tbl_start, tbl_info, nb);
        const int KB = t.type ? KB2 : KB1;
        const int buf = tl & 1;
        if (!ptx::mbar_wait(tempty_bar(buf), ((tl >> 1) & 1) ^ 1, abort_flag, global_abort)) { timeout(3); break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * UMMA_N);
        bool ok = true;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait(full_bar(s), (it / NSTAGE) & 1, abort_flag, global_abort)) {
            timeout(4); ok = false; break;
          }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t ad = desc_at(a_base, sa), bd = desc_at(b_base, sb);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            ptx::umma_bf16(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 128), IDESC, (kb | k) != 0);
          ptx::umma_commit(empty_bar(s));
        }
        if (!ok) break;
        ptx::umma_commit(tfull_bar(buf));
      }
    }
  } else {
    // ================================ A gather producers ================================
    const int gt = threadIdx.x - 192;     // 0..127
    const int chunk = gt & 7;             // 16-byte chunk of the 128-byte K row
    const int rbase = gt >> 3;            // rows rbase + 16 j
    uint32_t it = 0;
    for (int w = first; w < total && !*abort_flag; w += stride) {
      const Task t = decode_task(w, p, tbl_start, tbl_info, nb);
      const int KB = t.type ? KB2 : KB1;
      const int K = t.type ? p.f : p.d;
      const uint8_t* base = static_cast<const uint8_t*>(t.type ? (const void*)p.h : p.x);
      const size_t ld_bytes = (size_t)(t.type ? p.f : p.x_ld) * 2;
      bool ok = true;
      if (t.type == 1) {
        // tracker: the tile of h this task reads is complete once all 4 * n1 parts have been counted
        if (lane == 0) {
          const int want = 4 * p.n1;
          uint64_t t0 = 0;
          for (uint32_t i = 0; ld_acquire(p.done + t.mt_global) < want; ++i) {
            if ((i & 63u) == 63u) {
              if (*abort_flag || *global_abort) { ok = false; break; }
              const uint64_t now = ptx::globaltimer_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > 2000000000ull) { timeout(7); ok = false; break; }
            }
          }
        }
        ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
      }
      const uint8_t* src[8];
      uint32_t live = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int lr = rbase + 16 * j;
        src[j] = base;
        if (lr < t.rows) {
          int idx = t.row0 + lr;   // GEMM-2: the rows of h in place
          if (t.type == 0) {
            idx = __ldg(p.gather_idx + idx);
            if (p.gather_div > 1) idx /= p.gather_div;
            if (idx < 0 || idx >= p.x_rows) {   // a table entry that is no row of the source: zero-filled
              report_error(p.status, DEV_INDEX_OUT_OF_RANGE, KID_GEMM1, t.row0 + lr, idx);
              continue;
            }
          }
          src[j] = base + (size_t)idx * ld_bytes;
          live |= 1u << j;
        }
      }
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % NSTAGE;
        if (!ptx::mbar_wait(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag, global_abort)) {
          timeout(5); ok = false; break;
        }
        const uint32_t sa = smem_base + s * STAGE_BYTES;
        const int col = kb * 128 + chunk * 16;   // byte offset inside the source row
        const bool kin = col < K * 2;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int lr = rbase + 16 * j;
          const uint32_t dst = sa + lr * 128 + ((chunk ^ (lr & 7)) << 4);
          const bool on = kin && ((live >> j) & 1u);
          ptx::cp_async_16(dst, on ? (const void*)(src[j] + col) : (const void*)base, on ? 16u : 0u);
        }
        ptx::cp_async_arrive_noinc(full_bar(s));
      }
      if (!ok) break;
    }
    ptx::cp_async_wait_all();
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);   // abort path only: let copies in flight land
  }
  __syncthreads();
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Task blocks (one thread: at most E + P / 2048 blocks of each kind).  Three tables, `stride` entries apart:
// 0: both kinds interleaved in emission order, 1: the GEMM-1 blocks alone, 2: the GEMM-2 blocks alone.
__global__ void ffn_task_table_kernel(const int32_t* __restrict__ expert_counts, int E, int n1, int n2,
                                      int32_t* blk_start, int4* blk_info, int32_t* n_blocks, int stride) {
  grid_dependency_sync();
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int nb = 0, acc = 0, nb1 = 0, acc1 = 0, nb2 = 0, acc2 = 0;
  int32_t *s1 = blk_start + stride, *s2 = blk_start + 2 * stride;
  int4 *i1 = blk_info + stride, *i2 = blk_info + 2 * stride;
  int pe = -1, pm0 = 0, pmc = 0;   // previous GEMM-1 block, whose GEMM-2 block follows the next GEMM-1 block
  auto emit2 = [&](int e, int m0, int mc) {
    blk_start[nb] = acc; blk_info[nb] = make_int4(1, e, m0, mc); acc += mc * n2; ++nb;
    s2[nb2] = acc2; i2[nb2] = make_int4(1, e, m0, mc); acc2 += mc * n2; ++nb2;
  };
  for (int e = 0; e < E; ++e) {
    const int M = (expert_counts[e] + BM - 1) / BM;
    for (int m0 = 0; m0 < M; m0 += M_BLOCK) {
      const int mc = min(M_BLOCK, M - m0);
      blk_start[nb] = acc; blk_info[nb] = make_int4(0, e, m0, mc); acc += mc * n1; ++nb;
      s1[nb1] = acc1; i1[nb1] = make_int4(0, e, m0, mc); acc1 += mc * n1; ++nb1;
      if (pe >= 0) emit2(pe, pm0, pmc);
      pe = e; pm0 = m0; pmc = mc;
    }
  }
  if (pe >= 0) emit2(pe, pm0, pmc);
  blk_start[nb] = acc; s1[nb1] = acc1; s2[nb2] = acc2;
  n_blocks[0] = nb; n_blocks[1] = nb1; n_blocks[2] = nb2;
}

}  // namespace

size_t fused_max_blocks(int T, int k, int E) { return 2 * ((size_t)E + ((size_t)T * k) / (BM * M_BLOCK) + 2); }

cudaError_t launch_ffn_fused(const FusedParams& p, const int32_t* expert_counts, int32_t* blk_start, int4* blk_info,
                             int32_t* n_blocks, size_t done_entries, const CUtensorMap& m_w1, const CUtensorMap& m_w3,
                             const CUtensorMap& m_w2, cudaStream_t st) {
  static std::atomic<bool> attr_set[MAX_DEVICES];
  const int dev = current_device();
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(ffn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  cudaError_t err = cudaMemsetAsync(p.done, 0, done_entries * sizeof(int32_t), st);
  if (err != cudaSuccess) return err;
  if ((err = launch_pdl(ffn_task_table_kernel, 1, 32, 0, st, expert_counts, p.E, p.n1, p.n2, blk_start, blk_info,
                        n_blocks, p.tbl_stride)) != cudaSuccess)
    return err;
  ProfileScope prof(KID_GEMM1, st);
  return launch_pdl(ffn_fused_kernel, sm_count(), THREADS, SMEM_BYTES, st, m_w1, m_w3, m_w2, p);
}

}  // namespace ffn
}  // namespace tcmoe
