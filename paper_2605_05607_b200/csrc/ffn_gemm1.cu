// GEMM-1 of the expert FFN with the SwiGLU epilogue (paper Sec. II-A "GEMM-1"; Sec. IV: the
// dispatch gather is the GEMM's prologue, tiles of 128 tokens):
//     h[r, n] = silu(a_r . W1[e][:, n]) * (a_r . W3[e][:, n]),   a_r = src[gather_idx[r] / gather_div]
//
// A rows are GATHERED (they are arbitrary rows of the dispatched buffer, or of x itself in the
// fused layer) by cp.async into the 128-byte swizzled K-major layout the UMMA descriptor expects;
// B = two 64-column slabs of W1 and the same two of W3 loaded by TMA side by side, so that ONE
// 128 x 256 x 16 UMMA yields both products (accumulator columns [0,128) = a.W1, [128,256) = a.W3).
//
// One persistent CTA per SM (tcgen05 cta_group::1) walks tile tasks decoded from the device-side
// tile prefix, so no routing-dependent quantity visits the host.  Warp roles: 0-3 epilogue
// (TMEM -> registers -> SwiGLU -> global), 4 TMA producer, 5 UMMA issuer and TMEM owner, 6-9 gather
// producers.  Accumulators are double-buffered in TMEM (2 x 256 columns): the epilogue of tile i
// overlaps the main loop of tile i+1.  Every wait is bounded.
//
// Pipeline: 4 stages, each an A tile (16 KiB, gathered) and a B tile (32 KiB, TMA) behind one
// full / one empty barrier.  The gather threads never wait for their own copies: after issuing the
// cp.async copies of a stage each thread posts cp.async.mbarrier.arrive.noinc on the stage's full
// barrier, so the barrier completes exactly when the last row has landed (and the TMA bytes are
// in), independent of how far the issuing threads have moved on.  An earlier form published a
// stage only when the copies of two later stages had been issued (commit groups, wait, proxy
// fence, arrive): the publication then trailed the tensor pipe by one stage and the kernel ran
// 8-11 % (K = 4096) to 30 % (K = 7168, rows gathered from DRAM) slower; deeper or split A / B
// rings on that form recovered only part of it and cost a second wait per k-block.
//
// CTA-pair (cta_group::2) variants of this kernel were measured and not kept.  With lagged
// publication they lost by 20-60 %; with self-arriving copies (the peer CTA's arrivals relayed to the
// leader's barrier by one thread, with a RELAXED cluster-scope arrive: a releasing one waits for the
// copies the SM has in flight and held the kernel at 0.83 us per stage) the paired form reaches the
// same UMMA rate as this kernel and then loses 4 % to the padding of 256-row tiles.  TMA
// tile::gather4 as the gather engine sustains only one 4-row instruction per ~40 ns.
#include "ffn_common.cuh"

#include <atomic>

namespace tcmoe {
namespace ffn {
namespace {

constexpr int NSTAGE = 4;
constexpr int A_BYTES = BM * BK * 2;         // 16 KiB
constexpr int B_BYTES = UMMA_N * BK * 2;     // 32 KiB = four 64-column slabs of 8 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_BARS = 2 * NSTAGE + 4;
constexpr int STAGE_OUT_WARP = 32 * 144;     // epilogue transpose buffer of one warp: 32 rows x (128 + 16) bytes
constexpr int TABLE_BYTES = (2 * (MAX_E + 1) * 4 + 15) & ~15;
constexpr int COLSCALE_WARP = UMMA_N * 4;     // FP8: one warp's copy of the tile's 128 + 128 output-column scales
constexpr int SMEM_BYTES =
    1024 + NSTAGE * STAGE_BYTES + NUM_BARS * 8 + 64 + TABLE_BYTES + 4 * STAGE_OUT_WARP + 4 * COLSCALE_WARP;
constexpr int THREADS = 320;
constexpr int GATHER_THREADS = 128;
constexpr int BN_OUT = 128;
constexpr uint32_t IDESC = idesc_bf16(BM);
// The producers (TMA thread, 128 gather threads) wait for a free stage with a suspend-time hint: parked in hardware
// instead of polling.  At the board's power limit the layer's time follows energy: GEMM-1 alone in a loop on the
// DeepSeek-V3 shape 15.78 -> 15.50 ms with the hint (two alternations, same box), a single cold launch 13.41 -> 13.48.
// The UMMA thread's wait for a full stage is on the critical path and keeps the plain form (hinting it too gives the
// gain back).
constexpr uint32_t FEED_HINT = 1000;
constexpr uint32_t IDESC_F8 = idesc_e4m3(BM);

// FP8 = true: A rows and weights are E4M3 codes, a stage holds 128 elements of K (the same 128
// bytes per row), W1 / W3 come K-major from [E, N, K] as two 128-row boxes, and the epilogue applies
// a_scale[source row] * b_scale[e, n] before the SwiGLU; h is written as bf16 either way.
//
// PLAIN = true turns the kernel into a single-CTA form of GEMM-2 (Sec. II-A "GEMM-2", gate weight in the
// epilogue, Sec. III-C): the "gather" reads the rows of h in place (gather_idx = NULL), both halves of
// the 256-column B tile come from the one weight map (map_w1), the epilogue writes
// o[r, n] = w_r * acc[r, n] for 256 columns.  Used instead of the CTA-pair kernel when experts are small
// (128-row tiles pad far less than 256-row pair tiles when most experts hold fewer than 128 rows).
template <bool FP8, bool PLAIN>
__global__ void __launch_bounds__(THREADS, 1)
ffn_gemm1_kernel(const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w3,
                 const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NSTAGE * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  int* abort_s = reinterpret_cast<int*>(tmem_slot + 1);
  int* tp_s = reinterpret_cast<int*>(tmem_slot + 16);
  int* eoff_s = tp_s + (MAX_E + 1);
  const uint32_t stage_base = ptx::smem_u32(tp_s) + TABLE_BYTES;   // 16-byte aligned
  float* colscale_base = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(tp_s) + TABLE_BYTES + 4 * STAGE_OUT_WARP);

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
  }
  if (warp == 5) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
    ptx::tmem_relinquish();
  }
  grid_dependency_sync();   // nothing above touches global data
  for (int i = threadIdx.x; i <= p.E; i += blockDim.x) {
    tp_s[i] = p.tile_prefix[i];
    eoff_s[i] = p.expert_offsets[i];
  }
  if (threadIdx.x == 0) *abort_s = p.status[ST_ABORT];
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = tp_s[p.E] * p.n_tiles;
  constexpr int BK_ELEMS = FP8 ? 2 * BK : BK;   // K elements per stage: 128 bytes per row either way
  const int KB = (p.K + BK_ELEMS - 1) / BK_ELEMS;
  volatile int* abort_flag = abort_s;
  const volatile int* global_abort = p.status + ST_ABORT;

  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, PLAIN ? KID_GEMM2 : KID_GEMM1, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };
  auto tile_of = [&](int w) { return decode_tile(w, tp_s, eoff_s, p.E, p.n_tiles, PLAIN ? 2 * BN_OUT : BN_OUT, BM, 0); };

  if (warp < 4) {
    // ================================ epilogue ================================
    int tl = 0;
    for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x, ++tl) {
      const Tile t = tile_of(w);
      const int buf = tl & 1;
      if (!ptx::mbar_wait_warp<true>(tfull_bar(buf), (tl >> 1) & 1, abort_flag, global_abort)) { timeout(1); break; }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UMMA_N);
      // A thread owns one accumulator row; 32 threads storing 16 bytes each to 32 different rows
      // would cost 32 memory transactions per instruction.  The warp transposes 64 output columns
      // at a time through shared memory (rows padded to 144 bytes: conflict-free both ways) and
      // stores whole 128-byte row segments, 8 lanes per row, 4 rows per instruction.
      const uint32_t stage = stage_base + (uint32_t)(warp * STAGE_OUT_WARP);
      const int srow = lane >> 3, piece = lane & 7;
      if (PLAIN) {
        // ---- GEMM-2 form: o = (gate weight x row scale) * acc * column scale, 256 columns
        const int lrow = warp * 32 + lane;
        float wr = 1.f;
        if (lrow < t.rows) {
          const size_t grow = (size_t)t.row0 + lrow;
          if (p.topk_w != nullptr) wr = __ldg(p.topk_w + __ldg(p.row_pair + grow));
          if (FP8) wr *= __ldg(p.a_scale + grow);
        }
        float* sb_col = colscale_base + warp * UMMA_N;
        if (FP8) {
          const float* g = p.b_scale + (size_t)t.e * p.N + t.n0;
#pragma unroll
          for (int i = 0; i < UMMA_N / 32; ++i) {
            const int n = lane + 32 * i;
            sb_col[n] = (t.n0 + n < p.N) ? __ldg(g + n) : 0.f;
          }
          __syncwarp();
        }
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t acc0[32], acc1[32];
          ptx::tmem_ld32(taddr + cc * 64, acc0);
          ptx::tmem_ld32(taddr + cc * 64 + 32, acc1);
          ptx::tmem_ld_wait_on(acc0);
          ptx::tmem_ld_wait_on(acc1);
          if (FP8) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int n = cc * 64 + j;
              acc0[j] = __float_as_uint(__uint_as_float(acc0[j]) * sb_col[n]);
              acc1[j] = __float_as_uint(__uint_as_float(acc1[j]) * sb_col[n + 32]);
            }
          }
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
          if (col < p.N) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = i * 4 + srow;
              if (warp * 32 + r < t.rows) {
                const uint4 q = ptx::ld_shared_v4(stage + r * 144 + piece * 16);
                *reinterpret_cast<uint4*>(p.out + (size_t)(t.row0 + warp * 32 + r) * (size_t)p.out_ld + col) = q;
              }
            }
          }
          __syncwarp();
        }
      } else {
        // ---- GEMM-1 form: SwiGLU of the W1 / W3 halves, 128 output columns
      float sa = 1.f;   // FP8: scale of this thread's row (the gather source row)
      float* s1 = colscale_base + warp * UMMA_N;   // this warp's copy of the W1 / W3 column scales (0 beyond N)
      float* s3 = s1 + 128;
      if (FP8) {
        const int lrow = warp * 32 + lane;
        if (lrow < t.rows) {
          int idx = __ldg(p.gather_idx + t.row0 + lrow);
          if (p.gather_div > 1) idx /= p.gather_div;
          sa = (idx >= 0 && idx < p.a_rows) ? __ldg(p.a_scale + idx) : 0.f;
        }
        const size_t g = (size_t)t.e * p.N + t.n0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int n = lane + 32 * i;
          const bool in = t.n0 + n < p.N;
          s1[n] = in ? (__ldg(p.b_scale + g + n)) : 0.f;
          s3[n] = in ? (__ldg(p.b_scale2 + g + n)) : 0.f;
        }
        __syncwarp();
      }
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
            float u0 = __uint_as_float(a1[j]), u1 = __uint_as_float(a1[j + 1]);
            float g0 = __uint_as_float(a3[j]), g1 = __uint_as_float(a3[j + 1]);
            if (FP8) {
              const int n = c * 32 + j;
              u0 *= sa * s1[n];
              g0 *= sa * s3[n];
              u1 *= sa * s1[n + 1];
              g1 *= sa * s3[n + 1];
            }
            q[i] = pack2(silu_mul(u0, g0), silu_mul(u1, g1));
          }
          ptx::st_shared_v4(stage + lane * 144 + (c & 1) * 64 + v * 16, q[0], q[1], q[2], q[3]);
        }
        if (c & 1) {
          __syncwarp();
          const int col = t.n0 + (c - 1) * 32 + piece * 8;
          if (col < p.N) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = i * 4 + srow;           // row of this warp's 32
              if (warp * 32 + r < t.rows) {
                const uint4 q = ptx::ld_shared_v4(stage + r * 144 + piece * 16);
                *reinterpret_cast<uint4*>(p.out + (size_t)(t.row0 + warp * 32 + r) * (size_t)p.out_ld + col) = q;
              }
            }
          }
          __syncwarp();
        }
      }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(buf));
    }
  } else if (warp == 4) {
    // ================================ TMA producer (weights) ================================
    if (lane == 0) {
      uint32_t it = 0;
      for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x) {
        const Tile t = tile_of(w);
        bool ok = true;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait<false, FEED_HINT>(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag, global_abort)) {
            timeout(2); ok = false; break;
          }
          const uint32_t sb = smem_base + s * STAGE_BYTES + A_BYTES;
          ptx::mbar_arrive_expect_tx(full_bar(s), B_BYTES);
          const int k0 = kb * BK_ELEMS;
          const CUtensorMap* hi_map = PLAIN ? &map_w1 : &map_w3;   // second 128 accumulator columns
          const int hi_n = PLAIN ? t.n0 + 128 : t.n0;
          if (FP8) {   // K-major boxes of 128 output columns x 128 bytes of K
            ptx::tma_load_3d(sb, &map_w1, full_bar(s), k0, t.n0, t.e);
            ptx::tma_load_3d(sb + 16384, hi_map, full_bar(s), k0, hi_n, t.e);
          } else {     // MN-major slabs of 64 output columns x 64 rows of K
            ptx::tma_load_3d(sb, &map_w1, full_bar(s), t.n0, k0, t.e);
            ptx::tma_load_3d(sb + 8192, &map_w1, full_bar(s), t.n0 + 64, k0, t.e);
            ptx::tma_load_3d(sb + 16384, hi_map, full_bar(s), hi_n, k0, t.e);
            ptx::tma_load_3d(sb + 24576, hi_map, full_bar(s), hi_n + 64, k0, t.e);
          }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    // ================================ UMMA issuer ================================
    if (lane == 0) {
      const uint64_t a_base = desc_base(16, 1024);
      const uint64_t b_base = FP8 ? desc_base(16, 1024) : desc_base(BK * 128, 1024);   // K-major : MN-major
      uint32_t it = 0;
      int tl = 0;
      for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x, ++tl) {
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
          for (int k = 0; k < 4; ++k) {   // 32 bytes of K per UMMA (16 bf16 / 32 E4M3): +32 B inside the swizzle row
            if (FP8) ptx::umma_f8(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), IDESC_F8, (kb | k) != 0);
            else ptx::umma_bf16(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 128), IDESC, (kb | k) != 0);   // B: +2 atoms
          }
          ptx::umma_commit(empty_bar(s));   // free the stage when these UMMAs have read it
        }
        if (!ok) break;
        ptx::umma_commit(tfull_bar(buf));   // accumulator complete
      }
    }
  } else {
    // ================================ A gather producers ================================
    const int gt = threadIdx.x - 192;     // 0..127
    const int chunk = gt & 7;             // 16-byte chunk of the 128-byte K row
    const int rbase = gt >> 3;            // rows rbase + 16 j
    uint32_t it = 0;
    for (int w = blockIdx.x; w < total && !*abort_flag; w += gridDim.x) {
      const Tile t = tile_of(w);
      constexpr int ELEM = FP8 ? 1 : 2;   // bytes per element of the source rows
      const uint8_t* src[8];
      const uint8_t* base = static_cast<const uint8_t*>(p.a_src);
      uint32_t live = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int lr = rbase + 16 * j;
        src[j] = base;
        if (lr < t.rows) {
          int idx = t.row0 + lr;   // PLAIN: the rows of h in place
          if (!PLAIN) {
            idx = __ldg(p.gather_idx + idx);
            if (p.gather_div > 1) idx /= p.gather_div;
            if (idx < 0 || idx >= p.a_rows) {   // a table entry that is no row of the source: zero-filled
              report_error(p.status, DEV_INDEX_OUT_OF_RANGE, KID_GEMM1, t.row0 + lr, idx);
              continue;
            }
          }
          src[j] = base + (size_t)idx * p.a_ld * ELEM;
          live |= 1u << j;
        }
      }
      bool ok = true;
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % NSTAGE;
        if (!ptx::mbar_wait<false, FEED_HINT>(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag, global_abort)) {
          timeout(5); ok = false; break;
        }
        const uint32_t sa = smem_base + s * STAGE_BYTES;
        const int col = kb * 128 + chunk * 16;   // byte offset inside the source row
        const bool kin = col < p.K * ELEM;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int lr = rbase + 16 * j;
          const uint32_t dst = sa + lr * 128 + ((chunk ^ (lr & 7)) << 4);
          const bool on = kin && ((live >> j) & 1u);
          ptx::cp_async_16(dst, on ? (const void*)(src[j] + col) : (const void*)base, on ? 16u : 0u);
        }
        // one arrival on the stage's full barrier once the copies above have landed; the thread
        // itself goes straight on to the next stage
        ptx::cp_async_arrive_noinc(full_bar(s));
      }
      if (!ok) break;
    }
    ptx::cp_async_wait_all();   // nothing may still be in flight towards shared memory at exit
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

}  // namespace

namespace {
template <bool FP8, bool PLAIN>
cudaError_t launch_form(const GemmParams& p, const CUtensorMap& m_a, const CUtensorMap& m_b, cudaStream_t st) {
  // per device; several host threads may get here at once: setting the attribute twice is harmless
  static std::atomic<bool> attr_set[MAX_DEVICES];
  const int dev = current_device();
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(ffn_gemm1_kernel<FP8, PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  ProfileScope prof(PLAIN ? KID_GEMM2 : KID_GEMM1, st);
  return launch_pdl(ffn_gemm1_kernel<FP8, PLAIN>, sm_count(), THREADS, SMEM_BYTES, st, m_a, m_b, p);
}
}  // namespace

cudaError_t launch_gemm1(const GemmParams& p, const CUtensorMap& m_w1, const CUtensorMap& m_w3, bool fp8,
                         cudaStream_t st) {
  return fp8 ? launch_form<true, false>(p, m_w1, m_w3, st) : launch_form<false, false>(p, m_w1, m_w3, st);
}

// GEMM-2 through the single-CTA kernel (128-row tiles): p.a_src = h (or its E4M3 copy), p.a_ld = f,
// p.tile_prefix = the 128-row tile prefix, p.n_tiles = ceil(N / 256); m_w2 is the weight map.
cudaError_t launch_gemm2_single(const GemmParams& p, const CUtensorMap& m_w2, bool fp8, cudaStream_t st) {
  return fp8 ? launch_form<true, true>(p, m_w2, m_w2, st) : launch_form<false, true>(p, m_w2, m_w2, st);
}

}  // namespace ffn
}  // namespace tcmoe
