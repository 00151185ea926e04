// Expert FFN as a grouped GEMM on the 5th-generation tensor cores (paper Sec. II-A GEMM-1 /
// GEMM-2; Sec. III-C: gate weight applied in GEMM-2's epilogue; Sec. IV-C: persistent thread
// blocks that fetch tile tasks instead of relying on the hardware block scheduler; Sec. VI-H:
// 128-token tiles).
//
//   MODE 0 (GEMM-1 + SwiGLU): h[r, n] = silu(a_r . W1[e][:, n]) * (a_r . W3[e][:, n])
//       A rows are GATHERED (a_r = src[gather_idx[r] / gather_div]) by cp.async into the 128-byte
//       swizzled K-major layout the UMMA descriptor expects; B = 64-column slabs of W1 and W3
//       loaded by TMA side by side so that ONE 128x256x16 UMMA produces both products.
//   MODE 1 (GEMM-2 + gate weight): o[r, n] = w_r * (h_r . W2[e][:, n]);  A and B both by TMA.
//
// One persistent CTA per SM walks tile tasks (expert, n-tile, m-tile) decoded from the device-side
// prefix of 128-row tiles per expert, so no routing-dependent quantity ever visits the host.
// Warp roles: 0-3 epilogue (TMEM -> registers -> global), 4 TMA producer, 5 UMMA issuer and TMEM
// owner, 6-9 A-gather producers (MODE 0).  Accumulators are double-buffered in TMEM (2 x 256
// columns) so the epilogue of tile i overlaps the main loop of tile i+1.  Every wait is bounded.
#include "common.cuh"
#include "ptx.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

namespace tcmoe {

namespace {

constexpr int BM = 128;                 // rows per tile (the paper's tsize)
constexpr int BK = 64;                  // K per pipeline stage = one 128-byte swizzle row of bf16
constexpr int UMMA_N = 256;
constexpr int NSTAGE = 4;
constexpr int A_BYTES = BM * BK * 2;    // 16 KiB
constexpr int B_BYTES = UMMA_N * BK * 2;  // 32 KiB = four 64-column slabs of 8 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int GATHER_LAG = 2;           // cp.async groups kept in flight per gather thread
constexpr int MAX_E = 1024;
constexpr int NUM_BARS = 2 * NSTAGE + 4;
constexpr int SMEM_BYTES = 1024 + NSTAGE * STAGE_BYTES + NUM_BARS * 8 + 64 + 2 * (MAX_E + 1) * 4;

struct GemmParams {
  const __nv_bfloat16* a_src;   // MODE 0 gather source
  int a_ld;
  const int32_t* gather_idx;
  int gather_div;
  __nv_bfloat16* out;
  int out_ld;
  const float* topk_w;          // MODE 1 epilogue weights (NULL: 1)
  const int32_t* row_pair;
  const int32_t* expert_offsets;
  const int32_t* mt_prefix;
  int E, K, N, n_tiles;
  int32_t* status;
};

struct Tile {
  int e, n0, row0, rows;
};

__device__ __forceinline__ Tile decode_tile(int w, const int* mtp, const int* eoff, int E, int n_tiles, int bn_out) {
  int lo = 0, hi = E;  // mtp[lo] * n_tiles <= w < mtp[hi] * n_tiles
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (mtp[mid] * n_tiles <= w) lo = mid; else hi = mid;
  }
  const int local = w - mtp[lo] * n_tiles;
  const int mt = mtp[lo + 1] - mtp[lo];
  Tile t;
  t.e = lo;
  t.n0 = (local / mt) * bn_out;
  t.row0 = eoff[lo] + (local % mt) * BM;
  t.rows = min(BM, eoff[lo + 1] - t.row0);
  return t;
}

// 64-bit shared-memory matrix descriptors (sm_100 format: version 1, 128-byte swizzle).
//  A, K-major : rows of 128 B; 8-row groups 1024 B apart (SBO); LBO unused.
//  B, MN-major: 64-column slabs; inside a slab 8 K-rows of 128 B form a 1024-B atom, atoms of
//               successive K 1024 B apart (SBO); slabs BK*128 B apart (LBO).
__device__ __forceinline__ uint64_t desc_base(uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) | ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) |
         (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t desc_at(uint64_t base, uint32_t smem_addr) {
  return base | (uint64_t)((smem_addr & 0x3FFFF) >> 4);
}

// instruction descriptor: D fp32, A/B bf16, A K-major, B MN-major, N = 256, M = 128
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                           ((uint32_t)(UMMA_N >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ float silu_mul(float a, float b) { return __fdividef(a, 1.f + __expf(-a)) * b; }

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int MODE>
__global__ void __launch_bounds__(MODE == 0 ? 320 : 192, 1)
ffn_gemm_kernel(const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
                const __grid_constant__ CUtensorMap map_a, const GemmParams p) {
  constexpr int BN_OUT = (MODE == 0) ? 128 : 256;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NSTAGE * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  int* abort_s = reinterpret_cast<int*>(tmem_slot + 1);
  int* mtp_s = reinterpret_cast<int*>(tmem_slot + 16);
  int* eoff_s = mtp_s + (MAX_E + 1);

  const uint32_t smem_base = ptx::smem_u32(smem);
  const uint32_t bar_base = ptx::smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (NSTAGE + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * NSTAGE + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * NSTAGE + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  for (int i = threadIdx.x; i <= p.E; i += blockDim.x) {
    mtp_s[i] = p.mt_prefix[i];
    eoff_s[i] = p.expert_offsets[i];
  }
  if (threadIdx.x == 0) {
    *abort_s = p.status[ST_ABORT];
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), MODE == 0 ? 1 + 4 : 1);  // TMA thread (+ one lane per gather warp)
      ptx::mbar_init(empty_bar(s), 1);                     // tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tfull_bar(b), 1);                     // tcgen05.commit
      ptx::mbar_init(tempty_bar(b), 4);                    // one lane per epilogue warp
    }
    ptx::fence_mbar_init();
  }
  if (warp == 4 && lane == 0) {
    ptx::prefetch_tensormap(&map_b0);
    if (MODE == 0) ptx::prefetch_tensormap(&map_b1);
    else ptx::prefetch_tensormap(&map_a);
  }
  if (warp == 5) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = mtp_s[p.E] * p.n_tiles;
  const int KB = (p.K + BK - 1) / BK;
  volatile int* abort_flag = abort_s;

  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, MODE == 0 ? KID_GEMM1 : KID_GEMM2, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };

  if (warp < 4) {
    // ================================ epilogue ================================
    int tl = 0;
    for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x, ++tl) {
      const Tile t = decode_tile(w, mtp_s, eoff_s, p.E, p.n_tiles, BN_OUT);
      const int buf = tl & 1;
      const bool ready = ptx::mbar_wait(tfull_bar(buf), (tl >> 1) & 1, abort_flag);
      if (!__all_sync(0xFFFFFFFFu, ready)) { timeout(1); break; }  // warp-uniform: tcgen05.ld is .aligned
      ptx::tc_fence_after();
      const int lrow = warp * 32 + lane;
      const bool valid = lrow < t.rows;
      const size_t grow = (size_t)t.row0 + lrow;
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UMMA_N);
      __nv_bfloat16* orow = p.out + grow * (size_t)p.out_ld + t.n0;
      if (MODE == 0) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t a1[32], a3[32];
          ptx::tmem_ld32(taddr + c * 32, a1);
          ptx::tmem_ld32(taddr + 128 + c * 32, a3);
          ptx::tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (t.n0 + c * 32 + v * 8 < p.N) {
                uint4 q;
                uint32_t* qq = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int j = v * 8 + 2 * i;
                  qq[i] = pack2(silu_mul(__uint_as_float(a1[j]), __uint_as_float(a3[j])),
                                silu_mul(__uint_as_float(a1[j + 1]), __uint_as_float(a3[j + 1])));
                }
                *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = q;
              }
            }
          }
        }
      } else {
        float wr = 1.f;
        if (valid && p.topk_w != nullptr) wr = __ldg(p.topk_w + __ldg(p.row_pair + grow));
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          uint32_t acc[32];
          ptx::tmem_ld32(taddr + c * 32, acc);
          ptx::tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (t.n0 + c * 32 + v * 8 < p.N) {
                uint4 q;
                uint32_t* qq = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int j = v * 8 + 2 * i;
                  qq[i] = pack2(wr * __uint_as_float(acc[j]), wr * __uint_as_float(acc[j + 1]));
                }
                *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = q;
              }
            }
          }
        }
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
        const Tile t = decode_tile(w, mtp_s, eoff_s, p.E, p.n_tiles, BN_OUT);
        bool ok = true;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag)) { timeout(2); ok = false; break; }
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          ptx::mbar_arrive_expect_tx(full_bar(s), MODE == 0 ? B_BYTES : A_BYTES + B_BYTES);
          const int k0 = kb * BK;
          if (MODE == 0) {
            ptx::tma_load_3d(sb, &map_b0, full_bar(s), t.n0, k0, t.e);
            ptx::tma_load_3d(sb + 8192, &map_b0, full_bar(s), t.n0 + 64, k0, t.e);
            ptx::tma_load_3d(sb + 16384, &map_b1, full_bar(s), t.n0, k0, t.e);
            ptx::tma_load_3d(sb + 24576, &map_b1, full_bar(s), t.n0 + 64, k0, t.e);
          } else {
            ptx::tma_load_2d(sa, &map_a, full_bar(s), k0, t.row0);
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tma_load_3d(sb + c * 8192, &map_b0, full_bar(s), t.n0 + c * 64, k0, t.e);
          }
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
      for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x, ++tl) {
        const int buf = tl & 1;
        if (!ptx::mbar_wait(tempty_bar(buf), ((tl >> 1) & 1) ^ 1, abort_flag)) { timeout(3); break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * UMMA_N);
        bool ok = true;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait(full_bar(s), (it / NSTAGE) & 1, abort_flag)) { timeout(4); ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t ad = desc_at(a_base, sa), bd = desc_at(b_base, sb);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)  // K = 16 per UMMA: A +32 B inside the swizzle row, B +2 atoms
            ptx::umma_bf16(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 128), IDESC, (kb | k) != 0);
          ptx::umma_commit(empty_bar(s));   // frees the stage when these UMMAs have read it
        }
        if (!ok) break;
        ptx::umma_commit(tfull_bar(buf));   // accumulator complete
      }
    }
  } else if (MODE == 0) {
    // ================================ A gather producers ================================
    const int gt = threadIdx.x - 192;     // 0..127
    const int chunk = gt & 7;             // 16-byte chunk of the 128-byte K row
    const int rbase = gt >> 3;            // rows rbase + 16 j
    uint32_t it = 0;
    for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x) {
      const Tile t = decode_tile(w, mtp_s, eoff_s, p.E, p.n_tiles, BN_OUT);
      const __nv_bfloat16* src[8];
      uint32_t live = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int lr = rbase + 16 * j;
        src[j] = p.a_src;
        if (lr < t.rows) {
          int idx = __ldg(p.gather_idx + t.row0 + lr);
          if (p.gather_div > 1) idx /= p.gather_div;
          src[j] = p.a_src + (size_t)idx * p.a_ld;
          live |= 1u << j;
        }
      }
      bool ok = true;
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % NSTAGE;
        if (!ptx::mbar_wait(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag)) { timeout(5); ok = false; break; }
        const uint32_t sa = smem_base + s * STAGE_BYTES;
        const int col = kb * BK + chunk * 8;
        const bool kin = col < p.K;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int lr = rbase + 16 * j;
          const uint32_t dst = sa + lr * 128 + ((chunk ^ (lr & 7)) << 4);
          const bool on = kin && ((live >> j) & 1u);
          ptx::cp_async_16(dst, on ? (const void*)(src[j] + col) : (const void*)p.a_src, on ? 16u : 0u);
        }
        ptx::cp_async_commit();
        if (it >= GATHER_LAG) {
          ptx::cp_async_wait<GATHER_LAG>();
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(full_bar((it - GATHER_LAG) % NSTAGE));
        }
      }
      if (!ok) break;
    }
    ptx::cp_async_wait<0>();
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      const uint32_t first = it >= GATHER_LAG ? it - GATHER_LAG : 0;
      for (uint32_t i = first; i < it; ++i) ptx::mbar_arrive(full_bar(i % NSTAGE));
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // abort path only: give bulk copies still in flight time to land before the CTA retires
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 weights [E, K, N] row-major: box = 64 (N) x 64 (K) x 1, 128-byte swizzle, zero fill
bool make_weight_map(CUtensorMap* map, const void* base, int E, int K, int N) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)K, (cuuint64_t)E};
  cuuint64_t strides[2] = {(cuuint64_t)N * 2, (cuuint64_t)N * K * 2};
  cuuint32_t box[3] = {64, BK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 activations [rows, K] row-major: box = 64 (K) x 128 rows
bool make_act_map(CUtensorMap* map, const void* base, int rows, int K) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {BK, BM};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        n <= 0)
      n = 148;
  }
  return n;
}

cudaError_t launch_expert_ffn(const Shape& s, const FfnArgs& a, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e1 = cudaFuncSetAttribute(ffn_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    cudaError_t e2 = cudaFuncSetAttribute(ffn_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e1 != cudaSuccess) return e1;
    if (e2 != cudaSuccess) return e2;
    attr_set = true;
  }
  const int P = s.T * s.k;
  CUtensorMap m_w1, m_w3, m_w2, m_h;
  if (!make_weight_map(&m_w1, a.w1, s.E, s.d, s.f) || !make_weight_map(&m_w3, a.w3, s.E, s.d, s.f) ||
      !make_weight_map(&m_w2, a.w2, s.E, s.f, s.d) || !make_act_map(&m_h, a.h, P, s.f))
    return cudaErrorInvalidValue;
  const int grid = sm_count();

  GemmParams g1{};
  g1.a_src = static_cast<const __nv_bfloat16*>(a.a_src);
  g1.a_ld = s.d;
  g1.gather_idx = a.gather_idx;
  g1.gather_div = a.gather_div;
  g1.out = static_cast<__nv_bfloat16*>(a.h);
  g1.out_ld = s.f;
  g1.expert_offsets = a.expert_offsets;
  g1.mt_prefix = a.mt_prefix;
  g1.E = s.E;
  g1.K = s.d;
  g1.N = s.f;
  g1.n_tiles = (s.f + 127) / 128;
  g1.status = a.status;
  {
    ProfileScope prof(KID_GEMM1, st);
    ffn_gemm_kernel<0><<<grid, 320, SMEM_BYTES, st>>>(m_w1, m_w3, m_h, g1);
  }
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;

  GemmParams g2{};
  g2.out = static_cast<__nv_bfloat16*>(a.o);
  g2.out_ld = s.d;
  g2.topk_w = a.topk_w;
  g2.row_pair = a.row_pair;
  g2.expert_offsets = a.expert_offsets;
  g2.mt_prefix = a.mt_prefix;
  g2.E = s.E;
  g2.K = s.f;
  g2.N = s.d;
  g2.n_tiles = (s.d + 255) / 256;
  g2.status = a.status;
  {
    ProfileScope prof(KID_GEMM2, st);
    ffn_gemm_kernel<1><<<grid, 192, SMEM_BYTES, st>>>(m_w2, m_w2, m_h, g2);
  }
  return cudaGetLastError();
}

}  // namespace tcmoe
