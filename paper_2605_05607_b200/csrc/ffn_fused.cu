// The layer's stages as ONE persistent kernel paced by a token tracker (paper Sec. IV "token-centric kernel
// fusion": tiles of 128 tokens move through the stages of the layer as soon as the stage before has produced
// them; Sec. IV-B: tracker tables record what is complete, Sec. IV-C: persistent thread blocks fetch tasks and
// poll the tracker; synchronisation tile of 128 tokens, Sec. VII-C).
//
// Tasks
//   Dispatch  (optional) 16 rows of the per-expert layout tensors xs (Sec. III-D): xs[r] = x[token of row r]
//   GEMM-1    128 rows x 128 columns of h: A = rows of x gathered in the prologue (or rows of xs in place when
//             Dispatch tasks run), B = W1 | W3, SwiGLU epilogue
//   GEMM-2    128 rows x 256 columns of o: A = rows of h, B = W2, gate weight in the epilogue (Sec. III-C)
//   Combine   (optional) one token: the two-level sum of its rows of o, un-permuted into y
// Both GEMMs use the single-CTA UMMA form (all tcgen05 instructions of a kernel share one cta_group).
//
// Tracker (all counters in global memory, zeroed before the launch)
//   Tile Status table, one entry per 128-row tile of an expert (Sec. IV-B):
//     DAcc    rows of the tile written by Dispatch       -> GEMM-1 of the tile may start at rows-in-tile
//             (the paper counts bytes, tsize x bsize; rows x bsize here)
//     TBCnt1  parts of the h tile stored by GEMM-1        -> GEMM-2 of the tile may start at 4 warps x n1 tiles
//     TBCnt2  parts of the o tile stored by GEMM-2        -> at 4 warps x n2 tiles the warp that completed the
//             tile walks its token ids (the TID table: row_pair / k) and bumps
//   Output Readiness table, one entry per token:
//     nReady  complete rows of o of the token             -> Combine of the token may run at nReady == topk
// Every counter is bumped after the data it covers has been stored and fenced (the visibility rule of Sec. IV-B),
// and read with an acquire load; every wait is bounded.
//
// Schedule.  GEMM tasks: every CTA walks the interleaved list  G1(b0) G1(b1) G2(b0) G1(b2) G2(b1) ... of blocks of
// up to 16 row tiles of one expert, so a GEMM-2 tile is scheduled one block after the GEMM-1 tiles it needs; with
// the SM partition (Sec. IV-C) the first group of CTAs walks only GEMM-1 tiles and the second only GEMM-2 tiles.
// Dispatch units and Combine chunks (a few tokens) are handed out in order from two queue counters to four worker
// warps per CTA (with the partition: Dispatch to the workers of the GEMM-1 group, Combine to those of the GEMM-2
// group); when a CTA has finished its GEMM tasks all of its warps take Combine chunks.  Every dependency points to
// work that is earlier in its list and every list is taken in order by warps that wait for nothing else, so the
// waits cannot form a cycle as long as all CTAs of the grid are resident (the grid is sized from the occupancy
// query for that reason).
//
// Pipeline, barriers and epilogues are those of ffn_gemm1.cu.  Results equal the separate kernels bit for bit.
#include "ffn_common.cuh"

#include <algorithm>
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
#ifndef TCMOE_FUSED_WORKERS
#define TCMOE_FUSED_WORKERS 4
#endif
constexpr int NWARPS = 10 + TCMOE_FUSED_WORKERS;   // 0-3 epilogue, 4 TMA, 5 UMMA, 6-9 gather, 10-13 Dispatch / Combine workers
constexpr int THREADS = NWARPS * 32;
constexpr int COMB_BYTES = NWARPS * 3 * 32 * 4;   // per warp: slot order tables of combine_token()
constexpr int SMEM_BYTES = 1024 + NSTAGE * STAGE_BYTES + NUM_BARS * 8 + 64 + 4 * STAGE_OUT_WARP + COMB_BYTES;
constexpr int GATHER_THREADS = 128;
constexpr int M_BLOCK = 16;                  // row tiles per task block
constexpr int DISPATCH_UNIT = 16;            // rows per Dispatch task
constexpr uint32_t IDESC = idesc_bf16(BM);
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

struct Task {
  int type;        // 0: GEMM-1 tile, 1: GEMM-2 tile
  int e, n0, row0, rows;
  int mt_global;   // index of the 128-row tile among all tiles (tracker slot)
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
// tracker updates: the add is a release (everything this thread observed or wrote before it, including what it
// synchronised with through __syncwarp, is visible to whoever acquires the new value)
__device__ __forceinline__ void add_release(int32_t* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int add_acq_rel(int32_t* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
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
  int* comb_s = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(tmem_slot + 16) + 4 * STAGE_OUT_WARP);

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
  // GEMM task list of this CTA.  Default: every CTA walks the interleaved list (tasks blockIdx, blockIdx + grid, ...).
  // SM partition (Sec. IV-C: thread blocks are divided among the stages): the first `p.part_g1` CTAs take only
  // GEMM-1 tiles, the others only GEMM-2 tiles, each group walking the list of its own kind; the GEMM-2 group is
  // paced purely by the tracker.
  const bool part = p.part_g1 > 0;
  const int kind = part ? ((int)blockIdx.x < p.part_g1 ? 0 : 1) : 0;
  const int32_t* tbl_start = part ? p.blk_start + (size_t)(1 + kind) * p.tbl_stride : p.blk_start;
  const int4* tbl_info = part ? p.blk_info + (size_t)(1 + kind) * p.tbl_stride : p.blk_info;
  const int nb = __ldg(p.n_blocks + (part ? 1 + kind : 0));
  const int total = __ldg(tbl_start + nb);
  const int first = part ? (kind ? (int)blockIdx.x - p.part_g1 : (int)blockIdx.x) : (int)blockIdx.x;
  const int stride = part ? (kind ? (int)gridDim.x - p.part_g1 : p.part_g1) : (int)gridDim.x;
  const int KB1 = (p.d + BK - 1) / BK, KB2 = (p.f + BK - 1) / BK;
  const bool dispatched = p.dacc != nullptr;   // GEMM-1 reads the rows Dispatch wrote to xs
  volatile int* abort_flag = abort_s;
  const volatile int* global_abort = p.status + ST_ABORT;

  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, KID_GEMM1, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };
  // bounded wait of one warp on a tracker counter (lane 0 polls, all lanes get the result)
  auto wait_counter = [&](const int32_t* ctr, int want, int detail) -> bool {
    int ok = 1;
    if (lane == 0) {
      uint64_t t0 = 0;
      for (uint32_t i = 0; ld_acquire(ctr) < want; ++i) {
        if ((i & 63u) == 63u) {
          if (*abort_flag || *global_abort) { ok = 0; break; }
          const uint64_t now = ptx::globaltimer_ns();
          if (t0 == 0) t0 = now;
          else if (now - t0 > WAIT_LIMIT_NS) { timeout(detail); ok = 0; break; }
        }
      }
    }
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    __syncwarp();
    return ok != 0;
  };

  // ---- Combine tasks: chunks of up to 32 tokens handed out in order; lane i watches token i of the chunk ------------
  int* s_row = comb_s + warp * 96;
  int* s_dst = s_row + 32;
  float* s_w = reinterpret_cast<float*>(s_row + 64);
  auto combine_worker = [&](uint32_t sleep_ns) {
    if (p.nready == nullptr) return;
    const int per = p.chunk_tokens;                       // 1..32 tokens per chunk
    const int chunks = (p.T + per - 1) / per;
    while (!*abort_flag) {
      int c = 0;
      if (lane == 0) c = atomicAdd(p.queue + 1, 1);
      c = __shfl_sync(0xFFFFFFFFu, c, 0);
      if (c >= chunks) break;
      const int my_t = c * per + lane;
      const bool mine = lane < per && my_t < p.T;
      unsigned pending = __ballot_sync(0xFFFFFFFFu, mine);
      uint64_t t0 = 0;
      int ok = 1;
      while (pending && ok) {
        // Output Readiness table: a token is ready when all topk rows of o are complete
        const int rdy = mine ? ld_acquire(p.nready + my_t) : 0;
        const unsigned ready = __ballot_sync(0xFFFFFFFFu, rdy >= p.k) & pending;
        for (unsigned rem = ready; rem; rem &= rem - 1) {
          const int t = c * per + (__ffs(rem) - 1);
          if (p.k <= 2) combine_token<true, 2>(p.comb, t, lane, s_row, s_dst, s_w);
          else if (p.k <= 4) combine_token<true, 4>(p.comb, t, lane, s_row, s_dst, s_w);
          else combine_token<true, 8>(p.comb, t, lane, s_row, s_dst, s_w);
        }
        pending &= ~ready;
        if (pending && !ready) {
          __nanosleep(sleep_ns);
          if (lane == 0) {
            if (*abort_flag || *global_abort) ok = 0;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) { timeout(8); ok = 0; }
          }
          ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
        } else if (lane == 0) {
          t0 = 0;
        }
      }
      if (!ok) break;
    }
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
        if (p.nready != nullptr) {
          // tracker: this warp's 32 rows x 256 columns of the o tile are stored.  The warp whose part completes
          // the tile (TBCnt2 == 4 warps x n2 column tiles) walks the tile's token ids and bumps the Output
          // Readiness entry of each (the acquire half of its own add makes the other parts' stores precede
          // the bumps it releases).
          __syncwarp();
          int old = 0;
          if (lane == 0) old = add_acq_rel(p.tbcnt2 + t.mt_global, 1);
          old = __shfl_sync(0xFFFFFFFFu, old, 0);
          if (old == 4 * p.n2 - 1) {
            for (int r = lane; r < t.rows; r += 32)
              add_release(p.nready + __ldg(p.row_pair + (size_t)t.row0 + r) / p.k, 1);
          }
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
        // tracker: this warp's 32 rows x 128 columns of the h tile are stored (TBCnt1)
        __syncwarp();
        if (lane == 0) add_release(p.done + t.mt_global, 1);
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
    __syncwarp();
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
    __syncwarp();
  } else if (warp < 10) {
    // ================================ A gather producers ================================
    const int gt = threadIdx.x - 192;     // 0..127
    const int chunk = gt & 7;             // 16-byte chunk of the 128-byte K row
    const int rbase = gt >> 3;            // rows rbase + 16 j
    uint32_t it = 0;
    for (int w = first; w < total && !*abort_flag; w += stride) {
      const Task t = decode_task(w, p, tbl_start, tbl_info, nb);
      const int KB = t.type ? KB2 : KB1;
      const int K = t.type ? p.f : p.d;
      const bool in_place = t.type == 1 || dispatched;   // rows of h, or rows of xs: already in expert-sorted order
      const uint8_t* base = static_cast<const uint8_t*>(t.type ? (const void*)p.h : (dispatched ? (const void*)p.xs : p.x));
      const size_t ld_bytes = (size_t)(t.type ? p.f : (dispatched ? p.d : p.x_ld)) * 2;
      bool ok = true;
      // tracker: GEMM-2 waits for the h tile (TBCnt1: all 4 x n1 parts), GEMM-1 for the rows Dispatch writes (DAcc)
      if (t.type == 1) ok = wait_counter(p.done + t.mt_global, 4 * p.n1, 7);
      else if (dispatched) ok = wait_counter(p.dacc + t.mt_global, t.rows, 6);
      if (!ok) break;
      const uint8_t* src[8];
      uint32_t live = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int lr = rbase + 16 * j;
        src[j] = base;
        if (lr < t.rows) {
          int idx = t.row0 + lr;
          if (!in_place) {
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
  } else {
    // ================================ Dispatch / Combine workers ================================
    const bool do_dispatch = dispatched && (!part || kind == 0);
    const bool do_combine = !part || kind == 1;
    if (do_dispatch) {
      // Dispatch tasks: units of 16 expert-sorted rows, handed out in order so that tiles complete in the order
      // GEMM-1 asks for them.  xs[r] = x[token of row r]; then DAcc of the row's tile += rows written.
      const int n_tiles = __ldg(p.mt_prefix + p.E);
      const int units = n_tiles * (BM / DISPATCH_UNIT);
      const int vec_per_row = p.d / 8;
      while (!*abort_flag) {
        int u = 0;
        if (lane == 0) u = atomicAdd(p.queue, 1);
        u = __shfl_sync(0xFFFFFFFFu, u, 0);
        if (u >= units) break;
        const int mt_global = u / (BM / DISPATCH_UNIT);
        int lo = 0, hi = p.E;   // mt_prefix[lo] <= mt_global < mt_prefix[hi]
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (__ldg(p.mt_prefix + mid) <= mt_global) lo = mid; else hi = mid;
        }
        const int e0 = __ldg(p.expert_offsets + lo), e1 = __ldg(p.expert_offsets + lo + 1);
        const int row0 = e0 + (mt_global - __ldg(p.mt_prefix + lo)) * BM + (u % (BM / DISPATCH_UNIT)) * DISPATCH_UNIT;
        const int rows = max(0, min(DISPATCH_UNIT, e1 - row0));
        for (int r = 0; r < rows; ++r) {
          int idx = __ldg(p.gather_idx + row0 + r);
          if (p.gather_div > 1) idx /= p.gather_div;
          uint4* dst = reinterpret_cast<uint4*>(p.xs) + (size_t)(row0 + r) * vec_per_row;
          if (idx < 0 || idx >= p.x_rows) {   // a table entry that is no row of the source: reported, zero-filled
            if (lane == 0) report_error(p.status, DEV_INDEX_OUT_OF_RANGE, KID_DISPATCH, row0 + r, idx);
            for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0u, 0u, 0u, 0u);
            continue;
          }
          const uint4* from = static_cast<const uint4*>(p.x) + (size_t)idx * (p.x_ld / 8);
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
        __syncwarp();
        if (lane == 0 && rows > 0) add_release(p.dacc + mt_global, rows);
      }
    }
    if (do_combine) combine_worker(20000);
  }

  // a CTA that has finished its GEMM tasks lends all of its warps to the Combine tasks that are left
  if (warp < 10) combine_worker(2000);

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

// Persistent grid: as many CTAs as are resident at once (one per SM when the kernel has the device to itself),
// because tasks wait for tasks of other CTAs.
int fused_grid() {
  static std::atomic<int> grid_of[MAX_DEVICES];   // 0 = not computed yet; recomputing gives the same value
  std::atomic<int>& cached = grid_of[current_device()];
  int g = cached.load(std::memory_order_relaxed);
  if (g == 0) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ffn_fused_kernel, THREADS, SMEM_BYTES) != cudaSuccess ||
        per_sm <= 0) {
      (void)cudaGetLastError();
      per_sm = 1;
    }
    g = sm_count() * (per_sm < 1 ? per_sm : 1);   // one CTA per SM: each holds all 512 TMEM columns
    cached.store(g, std::memory_order_relaxed);
  }
  return g;
}

size_t tile_slots(int T, int k, int E) { return (size_t)T * k / BM + (size_t)E + 1; }

}  // namespace

size_t fused_max_blocks(int T, int k, int E) { return 2 * ((size_t)E + ((size_t)T * k) / (BM * M_BLOCK) + 2); }

// tracker region: DAcc | TBCnt1 | TBCnt2 (one entry per 128-row tile each) | nReady (per token) | 2 queue counters
size_t fused_tracker_words(int T, int k, int E) { return 3 * tile_slots(T, k, E) + (size_t)T + 2; }

cudaError_t launch_ffn_fused(FusedParams p, const int32_t* expert_counts, int32_t* blk_start, int4* blk_info,
                             int32_t* n_blocks, int32_t* tracker, const CUtensorMap& m_w1, const CUtensorMap& m_w3,
                             const CUtensorMap& m_w2, cudaStream_t st) {
  static std::atomic<bool> attr_set[MAX_DEVICES];
  const int dev = current_device();
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(ffn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  const size_t slots = tile_slots(p.T, p.k, p.E);
  const bool with_dispatch = p.xs != nullptr, with_combine = p.comb.y != nullptr;
  p.dacc = with_dispatch ? tracker : nullptr;
  p.done = tracker + slots;
  p.tbcnt2 = tracker + 2 * slots;
  p.nready = with_combine ? tracker + 3 * slots : nullptr;
  p.queue = tracker + 3 * slots + p.T;
  // Combine chunks: about four per warp of the grid, so that the tokens left when the GEMM tasks end (most of them:
  // a token is complete only when its last expert is) spread over every warp of every CTA
  const long long warps = (long long)fused_grid() * NWARPS;
  p.chunk_tokens = (int)std::max(1ll, std::min(32ll, (long long)p.T / (4 * warps)));
  cudaError_t err = cudaMemsetAsync(tracker, 0, fused_tracker_words(p.T, p.k, p.E) * sizeof(int32_t), st);
  if (err != cudaSuccess) return err;
  if ((err = launch_pdl(ffn_task_table_kernel, 1, 32, 0, st, expert_counts, p.E, p.n1, p.n2, blk_start, blk_info,
                        n_blocks, p.tbl_stride)) != cudaSuccess)
    return err;
  ProfileScope prof(KID_GEMM1, st);
  return launch_pdl(ffn_fused_kernel, fused_grid(), THREADS, SMEM_BYTES, st, m_w1, m_w3, m_w2, p);
}

}  // namespace ffn
}  // namespace tcmoe
