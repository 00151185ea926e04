// Weight gradients of the expert FFN (the backward pass of GEMM-1 / GEMM-2; paper Sec. VI-A evaluates training,
// forward + backward, of the layer of Sec. II-A):
//     dW[e][m, n] = sum over the rows r of expert e of  A[r, m] * B[r, n]
// with (A, B) = (xs, dA1) for W1, (xs, dA3) for W3 and (h, dO) for W2.  The contraction runs over the expert's rows,
// so both operands are read "MN-major" (the row index is K): TMA boxes of 64 columns x 64 rows with the 128-byte
// swizzle, two for the 128-column A tile and four for the 256-column B tile, exactly the layout the forward GEMMs
// use for their weight operand.  All row buffers live in the PADDED row space of the backward pass (every expert's
// segment is a multiple of 64 rows, pad rows are zero), so every 64-row K block is clean and needs no masking.
//
// One persistent CTA per SM (tcgen05 cta_group::1): warps 0-3 epilogue (TMEM -> bf16 rows of dW), warp 4 TMA
// producer, warp 5 UMMA issuer and TMEM owner; 4 stages of 48 KiB, accumulators double-buffered in TMEM.  Tasks
// (expert, m-tile of 128, n-tile of 256) are walked expert-major with the m-tile fastest, so the CTAs running
// together share one expert's rows in L2.  An expert without rows gets zeros.  Every wait is bounded.
#include "ffn_common.cuh"

#include <atomic>

namespace tcmoe {
namespace ffn {
namespace {

constexpr int NSTAGE = 4;
constexpr int A_BYTES = BM * BK * 2;         // 16 KiB: two slabs of 64 columns x 64 rows
constexpr int B_BYTES = UMMA_N * BK * 2;     // 32 KiB: four slabs
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_BARS = 2 * NSTAGE + 4;
constexpr int STAGE_OUT_WARP = 32 * 144;
constexpr int SMEM_BYTES = 1024 + NSTAGE * STAGE_BYTES + NUM_BARS * 8 + 64 + 4 * STAGE_OUT_WARP;
constexpr int THREADS = 192;
// D fp32, A / B bf16, both MN-major, N = 256, M = 128
constexpr uint32_t IDESC = idesc_bf16(BM) | (1u << 15);

struct WgradParams {
  const int32_t* poff;   // [E + 1] padded row offsets (multiples of 64)
  __nv_bfloat16* out;    // [E, M, N]
  int E, M, N;
  int32_t* status;
};

__global__ void __launch_bounds__(THREADS, 1)
wgrad_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const WgradParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NSTAGE * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  int* abort_s = reinterpret_cast<int*>(tmem_slot + 1);
  const uint32_t stage_base = ptx::smem_u32(tmem_slot + 16);

  const uint32_t smem_base = ptx::smem_u32(smem);
  const uint32_t bar_base = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (NSTAGE + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * NSTAGE + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * NSTAGE + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), 1);     // the TMA thread (expect_tx)
      ptx::mbar_init(empty_bar(s), 1);    // tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tfull_bar(b), 1);
      ptx::mbar_init(tempty_bar(b), 4);
    }
    ptx::fence_mbar_init();
  }
  if (warp == 4 && lane == 0) {
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
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
  const int mt = (p.M + BM - 1) / BM, nt = (p.N + UMMA_N - 1) / UMMA_N;
  const int per_expert = mt * nt;
  const int total = p.E * per_expert;
  volatile int* abort_flag = abort_s;
  const volatile int* global_abort = p.status + ST_ABORT;
  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, KID_WGRAD, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };
  struct Task { int e, m0, n0, row0, kb; };
  auto task_of = [&](int w) {
    Task t;
    t.e = w / per_expert;
    const int rem = w - t.e * per_expert;
    t.m0 = (rem % mt) * BM;
    t.n0 = (rem / mt) * UMMA_N;
    t.row0 = __ldg(p.poff + t.e);
    t.kb = (__ldg(p.poff + t.e + 1) - t.row0) / BK;
    return t;
  };

  if (warp < 4) {
    // ================================ epilogue ================================
    int tl = 0;
    for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x, ++tl) {
      const Task t = task_of(w);
      const int buf = tl & 1;
      if (!ptx::mbar_wait_warp<true>(tfull_bar(buf), (tl >> 1) & 1, abort_flag, global_abort)) { timeout(1); break; }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UMMA_N);
      const uint32_t stage = stage_base + (uint32_t)(warp * STAGE_OUT_WARP);
      const int srow = lane >> 3, piece = lane & 7;
      const int rows = min(BM, p.M - t.m0);   // rows of dW[e] in this tile
      __nv_bfloat16* out = p.out + ((size_t)t.e * p.M + t.m0) * (size_t)p.N;
      const bool empty = t.kb == 0;           // an expert without rows: the accumulator was never written
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t acc0[32], acc1[32];
        ptx::tmem_ld32(taddr + cc * 64, acc0);
        ptx::tmem_ld32(taddr + cc * 64 + 32, acc1);
        ptx::tmem_ld_wait_on(acc0);
        ptx::tmem_ld_wait_on(acc1);
        if (empty) {
#pragma unroll
          for (int j = 0; j < 32; ++j) { acc0[j] = 0u; acc1[j] = 0u; }
        }
        // transpose 64 columns through shared memory (rows padded to 144 bytes) and store whole 128-byte segments
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          ptx::st_shared_v4(stage + lane * 144 + v * 16,
                            pack2(__uint_as_float(acc0[v * 8]), __uint_as_float(acc0[v * 8 + 1])),
                            pack2(__uint_as_float(acc0[v * 8 + 2]), __uint_as_float(acc0[v * 8 + 3])),
                            pack2(__uint_as_float(acc0[v * 8 + 4]), __uint_as_float(acc0[v * 8 + 5])),
                            pack2(__uint_as_float(acc0[v * 8 + 6]), __uint_as_float(acc0[v * 8 + 7])));
          ptx::st_shared_v4(stage + lane * 144 + 64 + v * 16,
                            pack2(__uint_as_float(acc1[v * 8]), __uint_as_float(acc1[v * 8 + 1])),
                            pack2(__uint_as_float(acc1[v * 8 + 2]), __uint_as_float(acc1[v * 8 + 3])),
                            pack2(__uint_as_float(acc1[v * 8 + 4]), __uint_as_float(acc1[v * 8 + 5])),
                            pack2(__uint_as_float(acc1[v * 8 + 6]), __uint_as_float(acc1[v * 8 + 7])));
        }
        __syncwarp();
        const int col = t.n0 + cc * 64 + piece * 8;
        if (col < p.N) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = i * 4 + srow;
            if (warp * 32 + r < rows) {
              const uint4 q = ptx::ld_shared_v4(stage + r * 144 + piece * 16);
              *reinterpret_cast<uint4*>(out + (size_t)(warp * 32 + r) * (size_t)p.N + col) = q;
            }
          }
        }
        __syncwarp();
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(buf));
    }
  } else if (warp == 4) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      uint32_t it = 0;
      for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x) {
        const Task t = task_of(w);
        bool ok = true;
        for (int kb = 0; kb < t.kb; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag, global_abort)) {
            timeout(2); ok = false; break;
          }
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          ptx::mbar_arrive_expect_tx(full_bar(s), STAGE_BYTES);
          const int r0 = t.row0 + kb * BK;
          ptx::tma_load_2d(sa, &map_a, full_bar(s), t.m0, r0);
          ptx::tma_load_2d(sa + 8192, &map_a, full_bar(s), t.m0 + 64, r0);
#pragma unroll
          for (int c = 0; c < 4; ++c) ptx::tma_load_2d(sb + c * 8192, &map_b, full_bar(s), t.n0 + c * 64, r0);
        }
        if (!ok) break;
      }
    }
  } else {
    // ================================ UMMA issuer ================================
    if (lane == 0) {
      const uint64_t ab_base = desc_base(BK * 128, 1024);   // MN-major: slabs 8 KiB apart, 8-row groups 1 KiB apart
      uint32_t it = 0;
      int tl = 0;
      for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x, ++tl) {
        const Task t = task_of(w);
        const int buf = tl & 1;
        if (!ptx::mbar_wait(tempty_bar(buf), ((tl >> 1) & 1) ^ 1, abort_flag, global_abort)) { timeout(3); break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * UMMA_N);
        bool ok = true;
        for (int kb = 0; kb < t.kb; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait(full_bar(s), (it / NSTAGE) & 1, abort_flag, global_abort)) {
            timeout(4); ok = false; break;
          }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t ad = desc_at(ab_base, sa), bd = desc_at(ab_base, sb);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)   // 16 rows of K = two 8-row atoms = 2 KiB further in both operands
            ptx::umma_bf16(d_tmem, ad + (uint64_t)(k * 128), bd + (uint64_t)(k * 128), IDESC, (kb | k) != 0);
          ptx::umma_commit(empty_bar(s));
        }
        if (!ok) break;
        ptx::umma_commit(tfull_bar(buf));
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);   // abort path only: let bulk copies in flight land
  }
  __syncthreads();
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

// a, b: row buffers [rows_cap, M] / [rows_cap, N] in the padded row space; dw: [E, M, N] bf16 (fully written).
cudaError_t launch_wgrad(const CUtensorMap& m_a, const CUtensorMap& m_b, const int32_t* poff, void* dw, int E, int M,
                         int N, int32_t* status, cudaStream_t st) {
  static std::atomic<bool> attr_set[MAX_DEVICES];
  const int dev = current_device();
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  WgradParams p{poff, static_cast<__nv_bfloat16*>(dw), E, M, N, status};
  ProfileScope prof(KID_WGRAD, st);
  return launch_pdl(wgrad_kernel, sm_count(), THREADS, SMEM_BYTES, st, m_a, m_b, p);
}

}  // namespace ffn
}  // namespace tcmoe
