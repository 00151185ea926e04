// Gate logits on the tensor cores (paper Sec. II-A: the gate network that selects the experts):
//     logits[T, E] = x[T, d] (bf16) * w_gate[d, E] (fp32), fp32 result.
//
// x is bf16, so every product x * w is exact once w is written as hi + mid + lo with three bf16
// terms (8 + 8 + 8 mantissa bits cover fp32's 24).  The kernel therefore runs ONE bf16 UMMA
// accumulation over K' = 3 d: iteration j multiplies k-block j / 3 of x with k-block j / 3 of
// split j % 3, all into the same fp32 accumulator in TMEM.  The fp32 ALUs would need 2 T d E flop
// (120 GFLOP, 3.7 ms for the DeepSeek-V3-shaped layer); the tensor pipe does 3x that in ~0.3 ms.
//
// One CTA per (128-token tile, 256-expert tile); warps 0-3 epilogue (TMEM -> fp32 stores), warp 4
// TMA producer, warp 5 UMMA issuer and TMEM owner.  Two schedules:
//  - E <= 128 ("side by side"): the hi / mid / lo slabs of a k-block sit next to each other as
//    columns of one B tile (3 x ceil(E/64) slabs <= 6), x is loaded once per k-block, one or two
//    UMMAs fill separate accumulator column groups and the epilogue adds the three groups;
//    d/64 iterations of (A 16 KB + B <= 48 KB), 3 stages.
//  - larger E: the three terms are accumulated in place, 3 d/64 iterations of (A 16 KB + B 32 KB),
//    4 stages (the accumulators of 3 x 256 columns would not fit the 512 TMEM columns).
#include "ffn_common.cuh"

#include <atomic>

namespace tcmoe {
namespace {

using namespace ffn;

constexpr int A_BYTES = BM * BK * 2;
constexpr int MAX_STAGES = 4;
constexpr int NUM_BARS = 2 * MAX_STAGES + 1;
constexpr int RING_BYTES = 4 * (A_BYTES + 4 * 8192);   // = 3 * (A_BYTES + 6 * 8192) = 192 KiB
constexpr int SMEM_BYTES = 1024 + RING_BYTES + NUM_BARS * 8 + 64;
constexpr int THREADS = 192;

// w_gate fp32 [d, E] -> bf16 [3, d, Epad]: hi, mid, lo terms, zero in the padding columns
__global__ void __launch_bounds__(256) split_gate_kernel(const float* __restrict__ wg, __nv_bfloat16* __restrict__ out,
                                                         int d, int E, int Epad) {
  grid_dependency_sync();
  const size_t n = (size_t)d * Epad;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / Epad), col = (int)(i % Epad);
    float w = (col < E) ? __ldg(wg + (size_t)row * E + col) : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16_rn(w);
    w = __fsub_rn(w, __bfloat162float(hi));          // exact
    const __nv_bfloat16 mid = __float2bfloat16_rn(w);
    w = __fsub_rn(w, __bfloat162float(mid));         // exact
    out[i] = hi;
    out[n + i] = mid;
    out[2 * n + i] = __float2bfloat16_rn(w);
  }
}

struct GateParams {
  float* logits;
  int T, E, KB, n_tiles;
  int side_by_side;   // 1: hi | mid | lo as column groups of one B tile (E <= 128)
  int32_t* status;
};

__global__ void __launch_bounds__(THREADS, 1)
gate_umma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const GateParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + RING_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  int* abort_s = reinterpret_cast<int*>(tmem_slot + 1);

  const uint32_t smem_base = ptx::smem_u32(smem);
  const uint32_t bar_base = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
  const uint32_t done_bar = bar_base + 8u * (2 * MAX_STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mt = blockIdx.x / p.n_tiles, nt = blockIdx.x % p.n_tiles;
  const int row0 = mt * BM, n0 = nt * UMMA_N;
  const int ncols = min(UMMA_N, ((p.E - n0) + 63) & ~63);   // expert columns of this tile, in 64-column slabs
  const int nslab = ncols >> 6;
  const bool sbs = p.side_by_side != 0;
  const int bslabs = sbs ? 3 * nslab : nslab;            // B slabs per stage
  const int NSTAGE = sbs ? 3 : 4;
  const int STAGE_BYTES = A_BYTES + (sbs ? 6 : 4) * 8192;
  const int iters = sbs ? p.KB : 3 * p.KB;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(done_bar, 1);
    ptx::fence_mbar_init();
  }
  if (warp == 4 && lane == 0) {
    ptx::prefetch_tensormap(&map_x);
    ptx::prefetch_tensormap(&map_w);
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
  volatile int* abort_flag = abort_s;
  const volatile int* global_abort = p.status + ST_ABORT;
  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, KID_GATE, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };

  if (warp < 4) {
    // ================================ epilogue ================================
    if (!*abort_flag) {
      if (!ptx::mbar_wait_warp<true>(done_bar, 0, abort_flag, global_abort)) {
        timeout(1);
      } else {
        ptx::tc_fence_after();
        const int row = row0 + warp * 32 + lane;
        const bool valid = row < p.T;
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
        float* out = p.logits + (size_t)(valid ? row : 0) * p.E + n0;
        const bool vec = (p.E & 3) == 0;
        for (int c = 0; c < ncols; c += 32) {
          uint32_t acc[32];
          ptx::tmem_ld32(taddr + c, acc);
          if (sbs) {   // logits = (hi + mid) + lo: the three column groups are ncols apart
            uint32_t mid[32], lo[32];
            ptx::tmem_ld32(taddr + ncols + c, mid);
            ptx::tmem_ld32(taddr + 2 * ncols + c, lo);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int v = 0; v < 32; ++v)
              acc[v] = __float_as_uint(__fadd_rn(__fadd_rn(__uint_as_float(acc[v]), __uint_as_float(mid[v])),
                                                 __uint_as_float(lo[v])));
          }
          ptx::tmem_ld_wait();
          if (valid) {
            if (vec) {
#pragma unroll
              for (int v = 0; v < 8; ++v)
                if (n0 + c + v * 4 < p.E)
                  *reinterpret_cast<uint4*>(out + c + v * 4) =
                      make_uint4(acc[v * 4], acc[v * 4 + 1], acc[v * 4 + 2], acc[v * 4 + 3]);
            } else {
#pragma unroll
              for (int v = 0; v < 32; ++v)
                if (n0 + c + v < p.E) out[c + v] = __uint_as_float(acc[v]);
            }
          }
        }
        ptx::tc_fence_before();
      }
    }
  } else if (warp == 4) {
    // ================================ TMA producer ================================
    if (lane == 0 && !*abort_flag) {
      int slab_col[6], slab_split[6];   // slab c = (split c / nslab, 64-column slab c % nslab), hoisted out of the loop
#pragma unroll
      for (int c = 0; c < 6; ++c) {
        slab_col[c] = n0 + (c % nslab) * 64;
        slab_split[c] = c / nslab;
      }
      int s = 0, ph = 1;
      for (int it = 0; it < iters; ++it) {
        if (!ptx::mbar_wait(empty_bar(s), ph, abort_flag, global_abort)) { timeout(2); break; }
        const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
        const int kb = sbs ? it : it / 3, split0 = sbs ? 0 : it - kb * 3;
        ptx::mbar_arrive_expect_tx(full_bar(s), A_BYTES + bslabs * 8192);
        ptx::tma_load_2d(sa, &map_x, full_bar(s), kb * BK, row0);
#pragma unroll
        for (int c = 0; c < 6; ++c)
          if (c < bslabs) ptx::tma_load_3d(sb + c * 8192, &map_w, full_bar(s), slab_col[c], kb * BK, split0 + slab_split[c]);
        if (++s == NSTAGE) { s = 0; ph ^= 1; }
      }
    }
  } else {
    // ================================ UMMA issuer ================================
    if (lane == 0 && !*abort_flag) {
      const uint64_t a_base = desc_base(16, 1024);
      const uint64_t b_base = desc_base(BK * 128, 1024);
      auto idesc_n = [](int n) {
        return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      };
      const int n_first = min(bslabs, 4) * 64, n_second = (bslabs - min(bslabs, 4)) * 64;   // columns per UMMA
      bool ok = true;
      int s = 0, ph = 0;
      for (int it = 0; it < iters; ++it) {
        if (!ptx::mbar_wait(full_bar(s), ph, abort_flag, global_abort)) { timeout(3); ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
        const uint64_t ad = desc_at(a_base, sa), bd = desc_at(b_base, sb);
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          ptx::umma_bf16(tmem_base, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 128), idesc_n(n_first), (it | k) != 0);
          if (n_second > 0)   // slabs 4, 5 start 4 * 8 KiB into the B tile and 256 columns into the accumulator
            ptx::umma_bf16(tmem_base + 256, ad + (uint64_t)(k * 2), bd + (uint64_t)(2048 + k * 128), idesc_n(n_second),
                           (it | k) != 0);
        }
        ptx::umma_commit(empty_bar(s));
        if (++s == NSTAGE) { s = 0; ph ^= 1; }
      }
      if (ok) ptx::umma_commit(done_bar);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);   // abort path: let bulk copies in flight land
  }
  __syncthreads();
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

size_t gate_split_bytes(int d, int E) { return (size_t)3 * d * ((E + 63) & ~63) * 2; }

cudaError_t launch_gate_logits(const Shape& s, const void* x, const float* w_gate, float* logits, void* wsplit,
                               int32_t* status, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  // per device; several host threads may get here at once: setting the attribute twice is harmless
  static std::atomic<bool> attr_set[MAX_DEVICES];
  const int dev = current_device();
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(gate_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  const int Epad = (s.E + 63) & ~63;
  CUtensorMap m_x, m_w;
  {
    cuuint64_t dims[2] = {(cuuint64_t)s.d, (cuuint64_t)s.T};
    cuuint64_t strides[1] = {(cuuint64_t)s.d * 2};
    cuuint32_t box[2] = {BK, BM};
    if (!ffn::encode_tiled(&m_x, false, 2, x, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    cuuint64_t dims[3] = {(cuuint64_t)Epad, (cuuint64_t)s.d, 3};
    cuuint64_t strides[2] = {(cuuint64_t)Epad * 2, (cuuint64_t)Epad * s.d * 2};
    cuuint32_t box[3] = {64, BK, 1};
    if (!ffn::encode_tiled(&m_w, false, 3, wsplit, dims, strides, box)) return cudaErrorInvalidValue;
  }
  ProfileScope prof(KID_GATE, st);
  const size_t n = (size_t)s.d * Epad;
  int sb = (int)((n + 255) / 256);
  if (sb > sm_count() * 8) sb = sm_count() * 8;
  cudaError_t err = launch_pdl(split_gate_kernel, sb, 256, 0, st, w_gate, static_cast<__nv_bfloat16*>(wsplit), s.d, s.E,
                               Epad);
  if (err != cudaSuccess) return err;
  GateParams p;
  p.logits = logits;
  p.T = s.T;
  p.E = s.E;
  p.KB = (s.d + BK - 1) / BK;
  p.n_tiles = (s.E + UMMA_N - 1) / UMMA_N;
  p.side_by_side = s.E <= 128 ? 1 : 0;
  p.status = status;
  const int grid = ((s.T + BM - 1) / BM) * p.n_tiles;
  return launch_pdl(gate_umma_kernel, grid, THREADS, SMEM_BYTES, st, m_x, m_w, p);
}

}  // namespace tcmoe
