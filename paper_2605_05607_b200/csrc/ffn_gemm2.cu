// GEMM-2 of the expert FFN with the gate weight in the epilogue (paper Sec. II-A "GEMM-2";
// Sec. III-C: expert i scales its output by w_i in GEMM-2's epilogue so that Combine can be an
// un-weighted reduction):
//     o[r, n] = w_r * (h_r . W2[e][:, n])
//
// The same kernel, with GLU = true, is the CTA-pair form of GEMM-1 (Sec. II-A "GEMM-1") on rows that Dispatch
// has already placed in expert-sorted order (the per-expert layout tensors of Sec. III-D):
//     h[r, n] = silu(a_r . W1[e][:, n]) * (a_r . W3[e][:, n])
// CTA 0 of the pair then holds the 128-column tile of W1 and CTA 1 the same tile of W3, so the pair's 256
// accumulator columns are [a.W1 | a.W3] for every row and the epilogue applies SwiGLU to column c and c + 128.
//
// Both operands come by TMA (h rows are contiguous in expert-sorted order).  CTAs work in pairs
// (cluster of 2, tcgen05 cta_group::2): each CTA holds 128 rows of h and one half of the
// 256-column W2 tile; one UMMA of M = 256 spans the pair, so every weight byte is fetched and read
// from shared memory once per 256 rows.  Rank 0 of the pair (the leader) issues every UMMA.
//
// Barrier ownership in a pair:
//   full[s]    leader's copy: the leader announces the bytes of both CTAs, both CTAs' TMA loads
//              credit it
//   empty[s]   each CTA's own copy, signalled by the leader's tcgen05.commit (one commit per CTA)
//   tfull[b]   each CTA's own copy (accumulator buffer b complete), same
//   tempty[b]  leader's copy: the 4 epilogue warps of each CTA arrive when buffer b is drained
//
// Warp roles: 0-3 epilogue, 4 TMA producer, 5 UMMA issuer (leader only) and TMEM owner.
// Accumulators are double-buffered in TMEM; every wait is bounded; neither CTA retires before its
// peer has stopped touching its shared memory and TMEM (cluster barrier at the end).
#include "ffn_common.cuh"

#include <atomic>

namespace tcmoe {
namespace ffn {
namespace {

constexpr int NSTAGE = 6;
constexpr int A_BYTES = BM * BK * 2;            // 16 KiB: this CTA's 128 rows
constexpr int B_BYTES = (UMMA_N / 2) * BK * 2;  // 16 KiB: this CTA's half of the B tile (two 64-column slabs)
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_BARS = 2 * NSTAGE + 4;
constexpr int STAGE_OUT_WARP = 32 * 144;          // epilogue transpose buffer of one warp: 32 rows x (128 + 16) bytes
constexpr int TABLE_BYTES = (2 * (MAX_E + 1) * 4 + 15) & ~15;
constexpr int COLSCALE_WARP = UMMA_N * 4;          // FP8: one warp's copy of the tile's 256 output-column scales
constexpr int SMEM_BYTES =
    1024 + NSTAGE * STAGE_BYTES + NUM_BARS * 8 + 64 + TABLE_BYTES + 4 * STAGE_OUT_WARP + 4 * COLSCALE_WARP;
constexpr int THREADS = 192;
constexpr uint32_t IDESC = idesc_bf16(2 * BM);
constexpr uint32_t IDESC_F8 = idesc_e4m3(2 * BM);
constexpr uint32_t IDESC_BK = idesc_bf16(2 * BM) & ~(1u << 16);   // bf16 with a K-major B operand
constexpr uint32_t IDESC_WG = idesc_bf16(2 * BM) | (1u << 15);    // bf16 with both operands MN-major
constexpr uint32_t HINT = 4000;   // try_wait suspend-time hint (ns), see ptx::mbar_try_wait

// RED = false: rows go to o (bf16), Combine is a later pass.  RED = true: Combine happens here
// (Sec. IV: the fused pipeline reduces expert outputs as GEMM-2 produces them): each weighted row is
// added into the fp32 accumulator row of its token with vector reductions; o is never written.
// FP8 = true: h rows and weights are E4M3 codes, a stage holds 128 elements of K (the same 128 bytes
// per row), W2 comes K-major from [E, N, K] as one 128-row box per CTA, and the epilogue applies
// a_scale[row] * b_scale[e, n] together with the gate weight.
// MODE selects the epilogue and the operand walk:
//   PAIR_PLAIN    o = row weight x acc (GEMM-2; also dH = dO . W2^T of the backward pass): map_b0 = map_b1 = the weight,
//                 CTA `rank` takes columns n0 + 128 * rank
//   PAIR_GLU      GEMM-1 with the SwiGLU epilogue (see the head of this file): map_b0 = W1, map_b1 = W3, 128 output
//                 columns per tile
//   PAIR_GLU_BWD  the same GEMM recomputed in the backward pass: from a1 = a.W1, a3 = a.W3 and the incoming dh tile the
//                 epilogue writes h, da1 = dh * a3 * silu'(a1) and da3 = dh * silu(a1)
//   PAIR_WGRAD    dW[e] = A_e^T . B_e over the rows of expert e in the padded row space (segments start at poff[e], a multiple of 64, pad
//                 rows zero, so no block of 64 rows mixes experts and an expert without rows gets zeros): a task is a
//                 256 x 256 tile of one expert's gradient (p.K = its row count M, p.N its columns), the K walk runs over
//                 the expert's rows in blocks of 64, both operands are MN-major boxes of 64 columns x 64 rows; CTA `rank`
//                 holds rows m0 + 128 * rank of the tile and columns n0 + 128 * rank of B
//   PAIR_KSPLIT   acc = A0 . B0 + A1 . B1 (dX = dA1 . W1^T + dA3 . W3^T): the first p.k_split k-blocks come from
//                 (map_h, map_b0), the rest from (map_a1, map_b1); plain epilogue
// BKMAJ: the bf16 weight operand is read K-major (one box of 128 columns x 64 K per CTA and stage), which is how
// W^T looks when W is stored [K, N] with N contiguous: the backward GEMMs read the forward weights in place.
enum { PAIR_PLAIN = 0, PAIR_GLU = 1, PAIR_GLU_BWD = 2, PAIR_KSPLIT = 3, PAIR_WGRAD = 4 };

template <bool RED, bool FP8, int MODE, bool BKMAJ>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
ffn_gemm2_kernel(const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
                 const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_a1,
                 const GemmParams p) {
  constexpr bool GLU = MODE == PAIR_GLU || MODE == PAIR_GLU_BWD;
  constexpr bool KMAJ = FP8 || BKMAJ;   // the weight operand is K-major in shared memory
  static_assert(!(MODE != PAIR_PLAIN && (RED || FP8)), "only the plain form has the reducing / FP8 variants");
  constexpr int BN_OUT = GLU ? 128 : 256;
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
  const int rank = (int)ptx::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), 1);       // leader TMA thread (expect_tx for both CTAs)
      ptx::mbar_init(empty_bar(s), 1);      // tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tfull_bar(b), 1);      // tcgen05.commit
      ptx::mbar_init(tempty_bar(b), 8);     // one lane per epilogue warp, both CTAs
    }
    ptx::fence_mbar_init();
  }
  if (warp == 4 && lane == 0) {
    ptx::prefetch_tensormap(&map_b0);
    ptx::prefetch_tensormap(&map_b1);
    ptx::prefetch_tensormap(&map_h);
    if (MODE == PAIR_KSPLIT) ptx::prefetch_tensormap(&map_a1);
  }
  if (warp == 5) {
    ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), 512);
    ptx::tmem_relinquish_pair();
  }
  grid_dependency_sync();   // nothing above touches global data
  for (int i = threadIdx.x; i <= p.E; i += blockDim.x) {
    tp_s[i] = p.tile_prefix[i];
    eoff_s[i] = p.expert_offsets[i];
  }
  if (threadIdx.x == 0) *abort_s = p.status[ST_ABORT];
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();   // the peer's barriers are initialised before anything signals them
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  constexpr bool WGRAD = MODE == PAIR_WGRAD;
  const int wg_mt = (p.K + 2 * BM - 1) / (2 * BM), wg_per_expert = wg_mt * p.n_tiles;   // weight-gradient tiles per expert
  const int total = WGRAD ? p.E * wg_per_expert : tp_s[p.E] * p.n_tiles;
  constexpr int BK_ELEMS = FP8 ? 2 * BK : BK;   // K elements per stage: 128 bytes per row either way
  const int KB = MODE == PAIR_KSPLIT ? 2 * p.k_split : (p.K + BK_ELEMS - 1) / BK_ELEMS;
  volatile int* abort_flag = abort_s;
  const volatile int* global_abort = p.status + ST_ABORT;

  auto timeout = [&](int detail) {
    report_error(p.status, DEV_TIMEOUT, GLU ? KID_GEMM1 : KID_GEMM2, detail, blockIdx.x);
    p.status[ST_ABORT] = 1;
    *abort_flag = 1;
  };
  auto tile_of = [&](int w) {
    if (WGRAD) {   // (expert, m-tile of 256, n-tile of 256), m-tile fastest: neighbours share the B rows in L2
      Tile t;
      t.e = w / wg_per_expert;
      const int rem = w - t.e * wg_per_expert;
      const int m0 = (rem % wg_mt) * 2 * BM + rank * BM;
      t.n0 = (rem / wg_mt) * BN_OUT;
      t.row0 = eoff_s[t.e];                                  // first (padded) row of the expert: start of the K walk
      t.kb = (eoff_s[t.e + 1] - t.row0) / BK;
      t.rows = min(BM, p.K - m0);                            // rows of dW[e] this CTA owns (<= 0: none)
      t.out_row0 = t.e * p.K + m0;
      return t;
    }
    return decode_tile(w, tp_s, eoff_s, p.E, p.n_tiles, BN_OUT, 2 * BM, rank);
  };

  if (warp < 4) {
    // ================================ epilogue (both CTAs) ================================
    int tl = 0;
    for (int w = cluster_id; w < total && !*abort_flag; w += num_clusters, ++tl) {
      const Tile t = tile_of(w);
      const int buf = tl & 1;
      if (!ptx::mbar_wait_warp<false, HINT>(tfull_bar(buf), (tl >> 1) & 1, abort_flag, global_abort)) { timeout(1); break; }
      ptx::tc_fence_after();
      const int lrow = warp * 32 + lane;
      const bool valid = lrow < t.rows;
      const size_t grow = (size_t)(valid ? t.row0 + lrow : 0);
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UMMA_N);
      float* yrow = nullptr;
      float wr = 1.f;
      if (valid && !GLU && !WGRAD && (RED || p.topk_w != nullptr)) {
        const int pair = __ldg(p.row_pair + grow);
        if (p.topk_w != nullptr) wr = __ldg(p.topk_w + pair);
        if (FP8) wr *= __ldg(p.a_scale + grow);   // row scale of h joins the gate weight
        if (RED) yrow = p.y_acc + (size_t)(pair / p.y_div) * (size_t)p.N + t.n0;
      }
      // FP8: the tile's output-column scales, one copy per warp (0 beyond N), staged while the
      // main loop of this tile may still be running
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
      if (MODE == PAIR_GLU_BWD) {
        // backward of SwiGLU on the recomputed pre-activations: a thread owns one row and walks its 128 columns 32 at
        // a time; dh comes from global memory (64 bytes of the row per step), h / da1 / da3 go straight back
        const size_t rowoff = grow * (size_t)p.out_ld + t.n0;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t a1[32], a3[32];
          ptx::tmem_ld32(taddr + c * 32, a1);
          ptx::tmem_ld32(taddr + 128 + c * 32, a3);
          ptx::tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              const int col = t.n0 + c * 32 + v * 8;
              if (col < p.N) {
                const size_t at = rowoff + c * 32 + v * 8;
                const uint4 dq = *reinterpret_cast<const uint4*>(p.dh + at);
                const __nv_bfloat162* dp = reinterpret_cast<const __nv_bfloat162*>(&dq);
                uint32_t qh[4], q1[4], q3[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int j = v * 8 + 2 * i;
                  const float2 dhv = __bfloat1622float2(dp[i]);
                  float hh[2], d1[2], d3[2];
#pragma unroll
                  for (int u = 0; u < 2; ++u) {
                    const float x1 = __uint_as_float(a1[j + u]), x3 = __uint_as_float(a3[j + u]);
                    const float dv = u ? dhv.y : dhv.x;
                    const float sg = __fdividef(1.f, 1.f + __expf(-x1));
                    const float sl = x1 * sg;
                    hh[u] = sl * x3;
                    d3[u] = dv * sl;
                    d1[u] = dv * x3 * (sg * (1.f + x1 * (1.f - sg)));
                  }
                  qh[i] = pack2(hh[0], hh[1]);
                  q1[i] = pack2(d1[0], d1[1]);
                  q3[i] = pack2(d3[0], d3[1]);
                }
                *reinterpret_cast<uint4*>(p.out + at) = make_uint4(qh[0], qh[1], qh[2], qh[3]);
                *reinterpret_cast<uint4*>(p.out2 + at) = make_uint4(q1[0], q1[1], q1[2], q1[3]);
                *reinterpret_cast<uint4*>(p.out3 + at) = make_uint4(q3[0], q3[1], q3[2], q3[3]);
              }
            }
          }
        }
      } else if (GLU) {
        // SwiGLU of the W1 half (columns 0..127) and the W3 half (128..255): 128 columns of h, transposed
        // through shared memory 64 columns at a time and stored as whole 128-byte row segments
        const uint32_t stage = stage_base + (uint32_t)(warp * STAGE_OUT_WARP);
        const int srow = lane >> 3, piece = lane & 7;
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
        }
      } else if (RED) {
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          uint32_t acc[32];
          ptx::tmem_ld32(taddr + c * 32, acc);
          ptx::tmem_ld_wait();
          if (FP8) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int n = c * 32 + j;
              acc[j] = __float_as_uint(__uint_as_float(acc[j]) * sb_col[n]);
            }
          }
          if (valid) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (t.n0 + c * 32 + v * 8 < p.N) {
                float* dst = yrow + c * 32 + v * 8;
                ptx::red_add_v4(dst, wr * __uint_as_float(acc[v * 8]), wr * __uint_as_float(acc[v * 8 + 1]),
                                wr * __uint_as_float(acc[v * 8 + 2]), wr * __uint_as_float(acc[v * 8 + 3]));
                ptx::red_add_v4(dst + 4, wr * __uint_as_float(acc[v * 8 + 4]), wr * __uint_as_float(acc[v * 8 + 5]),
                                wr * __uint_as_float(acc[v * 8 + 6]), wr * __uint_as_float(acc[v * 8 + 7]));
              }
            }
          }
        }
      } else {
        // A thread owns one accumulator row, but 32 threads storing 16 bytes each to 32 different
        // rows cost 32 memory transactions per instruction.  The warp therefore transposes 64
        // columns at a time through shared memory (rows padded to 144 bytes: conflict-free both
        // ways) and stores whole 128-byte row segments, 8 lanes per row, 4 rows per instruction.
        const uint32_t stage = stage_base + (uint32_t)(warp * STAGE_OUT_WARP);
        const int srow = lane >> 3, piece = lane & 7;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t acc0[32], acc1[32];
          ptx::tmem_ld32(taddr + cc * 64, acc0);
          ptx::tmem_ld32(taddr + cc * 64 + 32, acc1);
          ptx::tmem_ld_wait_on(acc0);
          ptx::tmem_ld_wait_on(acc1);
          if (WGRAD && t.kb == 0) {   // an expert without rows: the accumulator was never written
#pragma unroll
            for (int j = 0; j < 32; ++j) { acc0[j] = 0u; acc1[j] = 0u; }
          }
          if (FP8) {   // per-output-column weight scales
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
              const int r = i * 4 + srow;           // row of this warp's 32
              if (warp * 32 + r < t.rows) {
                const uint4 q = ptx::ld_shared_v4(stage + r * 144 + piece * 16);
                *reinterpret_cast<uint4*>(p.out + (size_t)(t.out_row0 + warp * 32 + r) * (size_t)p.out_ld + col) = q;
              }
            }
          }
          __syncwarp();
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      // "accumulator buffer drained": the tcgen05.ld results are in registers (wait::ld above), so a
      // relaxed arrival is enough; a releasing one would first wait for this warp's row stores to
      // become visible cluster-wide, which on short-K tiles stalls the next-but-one main loop
      // (K = 512: 860 -> 1049 TFLOP/s with the relaxed form)
      if (lane == 0) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(tempty_bar(buf), 0));
    }
  } else if (warp == 4) {
    // ================================ TMA producer (both CTAs) ================================
    if (lane == 0) {
      uint32_t it = 0;
      for (int w = cluster_id; w < total && !*abort_flag; w += num_clusters) {
        const Tile t = tile_of(w);
        bool ok = true;
        const int KBt = WGRAD ? t.kb : KB;
        for (int kb = 0; kb < KBt; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait<false, HINT>(empty_bar(s), ((it / NSTAGE) & 1) ^ 1, abort_flag, global_abort)) {
            timeout(2); ok = false; break;
          }
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          const uint32_t lead_full = ptx::mapa(full_bar(s), 0);
          // the leader announces the bytes of both CTAs; the peer's copies only complete them
          if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);
          if (WGRAD) {   // four MN-major boxes of 64 columns x 64 rows: this CTA's 128 rows of A^T and 128 columns of B
            const int r0 = t.row0 + kb * BK, ma = t.out_row0 - t.e * p.K;
            ptx::tma_load_2d_pair(sa, &map_h, lead_full, ma, r0);
            ptx::tma_load_2d_pair(sa + 8192, &map_h, lead_full, ma + 64, r0);
            ptx::tma_load_2d_pair(sb, &map_b0, lead_full, t.n0 + rank * 128, r0);
            ptx::tma_load_2d_pair(sb + 8192, &map_b0, lead_full, t.n0 + rank * 128 + 64, r0);
            continue;
          }
          const bool second = MODE == PAIR_KSPLIT && kb >= p.k_split;     // second (A, B) pair of the K walk
          const int k0 = (second ? kb - p.k_split : kb) * BK_ELEMS;
          ptx::tma_load_2d_pair(sa, second ? &map_a1 : &map_h, lead_full, k0, t.row0);
          const CUtensorMap* map_b = MODE == PAIR_KSPLIT ? (second ? &map_b1 : &map_b0) : (rank == 0 ? &map_b0 : &map_b1);
          const int nb = GLU ? t.n0 : t.n0 + rank * 128;   // this CTA's 128 columns of the B tile
          if (KMAJ) {   // one K-major box: this CTA's 128 output columns x 128 bytes of K
            ptx::tma_load_3d_pair(sb, map_b, lead_full, k0, nb, t.e);
          } else {     // two MN-major slabs of 64 output columns x 64 rows of K
            ptx::tma_load_3d_pair(sb, map_b, lead_full, nb, k0, t.e);
            ptx::tma_load_3d_pair(sb + 8192, map_b, lead_full, nb + 64, k0, t.e);
          }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    // ================================ UMMA issuer (leader CTA only) ================================
    if (rank == 0 && lane == 0) {
      const uint64_t a_base = desc_base(16, 1024);
      const uint64_t b_base = KMAJ ? desc_base(16, 1024) : desc_base(BK * 128, 1024);   // K-major : MN-major
      uint32_t it = 0;
      int tl = 0;
      for (int w = cluster_id; w < total && !*abort_flag; w += num_clusters, ++tl) {
        const int buf = tl & 1;
        if (!ptx::mbar_wait_cluster<HINT>(tempty_bar(buf), ((tl >> 1) & 1) ^ 1, abort_flag, global_abort)) {
          timeout(3); break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * UMMA_N);
        bool ok = true;
        const int KBt = WGRAD ? tile_of(w).kb : KB;
        for (int kb = 0; kb < KBt; ++kb, ++it) {
          const int s = it % NSTAGE;
          if (!ptx::mbar_wait_cluster<HINT>(full_bar(s), (it / NSTAGE) & 1, abort_flag, global_abort)) {
            timeout(4); ok = false; break;
          }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t ad = desc_at(WGRAD ? b_base : a_base, sa), bd = desc_at(b_base, sb);   // WGRAD: A is MN-major too
          auto bd_a = [](uint64_t d, int k) { return d + (uint64_t)(k * 128); };               // 16 rows of K = 2 KiB
#pragma unroll
          for (int k = 0; k < 4; ++k) {   // 32 bytes of K per UMMA (16 bf16 / 32 E4M3): +32 B inside the swizzle row
            if (FP8) ptx::umma_f8_pair(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), IDESC_F8, (kb | k) != 0);
            else if (WGRAD) ptx::umma_bf16_pair(d_tmem, bd_a(ad, k), bd + (uint64_t)(k * 128), IDESC_WG, (kb | k) != 0);
            else if (BKMAJ) ptx::umma_bf16_pair(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), IDESC_BK, (kb | k) != 0);
            else ptx::umma_bf16_pair(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 128), IDESC, (kb | k) != 0);   // B: +2 atoms
          }
          // free the stage in both CTAs once these UMMAs have read it
          ptx::umma_commit_pair(ptx::mapa(empty_bar(s), 0));
          ptx::umma_commit_pair(ptx::mapa(empty_bar(s), 1));
        }
        if (!ok) break;
        ptx::umma_commit_pair(ptx::mapa(tfull_bar(buf), 0));   // accumulator complete, both halves
        ptx::umma_commit_pair(ptx::mapa(tfull_bar(buf), 1));
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag || *global_abort) {
    // abort path only: give bulk copies still in flight time to land before the CTAs retire
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  ptx::cluster_sync();   // neither CTA leaves while its peer may still touch its shared memory / TMEM
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, 512);
  }
}

// Persistent grid: two CTAs per resident cluster, at most one CTA per SM.
int pair_grid() {
  static std::atomic<int> grid_of[MAX_DEVICES];   // 0 = not computed yet; recomputing gives the same value
  std::atomic<int>& cached = grid_of[current_device()];
  int g = cached.load(std::memory_order_relaxed);
  if (g == 0) {
    int clusters = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sm_count() & ~1);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&clusters, ffn_gemm2_kernel<false, false, PAIR_PLAIN, false>, &cfg) != cudaSuccess || clusters <= 0) {
      (void)cudaGetLastError();
      clusters = sm_count() / 2;
    }
    g = 2 * min(clusters, sm_count() / 2);
    cached.store(g, std::memory_order_relaxed);
  }
  return g;
}

}  // namespace

namespace {
cudaError_t set_pair_attributes() {
  // per device; several host threads may get here at once: setting the attribute twice is harmless
  static std::atomic<bool> attr_set[MAX_DEVICES];
  const int dev = current_device();
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, false, PAIR_PLAIN, false>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<true, false, PAIR_PLAIN, false>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, true, PAIR_PLAIN, false>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<true, true, PAIR_PLAIN, false>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, false, PAIR_GLU, false>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, false, PAIR_PLAIN, true>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, false, PAIR_GLU_BWD, false>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, false, PAIR_KSPLIT, true>, attr, SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_gemm2_kernel<false, false, PAIR_WGRAD, false>, attr, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  return cudaSuccess;
}
}  // namespace

cudaError_t launch_gemm2(const GemmParams& p, const CUtensorMap& m_w2, const CUtensorMap& m_h, bool fp8,
                         cudaStream_t st) {
  cudaError_t e = set_pair_attributes();
  if (e != cudaSuccess) return e;
  ProfileScope prof(KID_GEMM2, st);
  const bool red = p.y_acc != nullptr;
  const int g = pair_grid();
  if (fp8) {
    if (red) return launch_pdl(ffn_gemm2_kernel<true, true, PAIR_PLAIN, false>, g, THREADS, SMEM_BYTES, st, m_w2, m_w2, m_h, m_h, p);
    return launch_pdl(ffn_gemm2_kernel<false, true, PAIR_PLAIN, false>, g, THREADS, SMEM_BYTES, st, m_w2, m_w2, m_h, m_h, p);
  }
  if (red) return launch_pdl(ffn_gemm2_kernel<true, false, PAIR_PLAIN, false>, g, THREADS, SMEM_BYTES, st, m_w2, m_w2, m_h, m_h, p);
  return launch_pdl(ffn_gemm2_kernel<false, false, PAIR_PLAIN, false>, g, THREADS, SMEM_BYTES, st, m_w2, m_w2, m_h, m_h, p);
}

// GEMM-1 on CTA pairs: m_xs maps the expert-sorted activation rows [P, K]; p.tile_prefix = the 256-row pair-tile
// prefix, p.n_tiles = ceil(N / 128), p.out = h.
cudaError_t launch_gemm1_pair(const GemmParams& p, const CUtensorMap& m_w1, const CUtensorMap& m_w3,
                              const CUtensorMap& m_xs, cudaStream_t st) {
  cudaError_t e = set_pair_attributes();
  if (e != cudaSuccess) return e;
  ProfileScope prof(KID_GEMM1, st);
  return launch_pdl(ffn_gemm2_kernel<false, false, PAIR_GLU, false>, pair_grid(), THREADS, SMEM_BYTES, st, m_w1, m_w3, m_xs,
                    m_xs, p);
}

// Backward pass, all on CTA pairs (see bwd.cu for the sequence):
//   launch_bwd_dh    dh = dO . W2^T          A = dO rows (m_do), B = W2 read K-major (m_w2t), N = f, K = d
//   launch_bwd_glu   GEMM-1 recomputed with the backward SwiGLU epilogue: p.dh in, p.out = h, p.out2 = dA1, p.out3 = dA3
//   launch_bwd_dx    dXs = dA1 . W1^T + dA3 . W3^T   A = (m_da1, m_da3), B = (m_w1t, m_w3t) K-major, p.k_split k-blocks each
cudaError_t launch_bwd_dh(const GemmParams& p, const CUtensorMap& m_w2t, const CUtensorMap& m_do, cudaStream_t st) {
  cudaError_t e = set_pair_attributes();
  if (e != cudaSuccess) return e;
  return launch_pdl(ffn_gemm2_kernel<false, false, PAIR_PLAIN, true>, pair_grid(), THREADS, SMEM_BYTES, st, m_w2t, m_w2t,
                    m_do, m_do, p);
}
cudaError_t launch_bwd_glu(const GemmParams& p, const CUtensorMap& m_w1, const CUtensorMap& m_w3, const CUtensorMap& m_xs,
                           cudaStream_t st) {
  cudaError_t e = set_pair_attributes();
  if (e != cudaSuccess) return e;
  return launch_pdl(ffn_gemm2_kernel<false, false, PAIR_GLU_BWD, false>, pair_grid(), THREADS, SMEM_BYTES, st, m_w1, m_w3,
                    m_xs, m_xs, p);
}
cudaError_t launch_bwd_dx(const GemmParams& p, const CUtensorMap& m_w1t, const CUtensorMap& m_w3t, const CUtensorMap& m_da1,
                          const CUtensorMap& m_da3, cudaStream_t st) {
  cudaError_t e = set_pair_attributes();
  if (e != cudaSuccess) return e;
  return launch_pdl(ffn_gemm2_kernel<false, false, PAIR_KSPLIT, true>, pair_grid(), THREADS, SMEM_BYTES, st, m_w1t, m_w3t,
                    m_da1, m_da3, p);
}

// Weight gradient on CTA pairs: dw[e] = A_e^T . B_e, A = [rows, M], B = [rows, N] in the padded row space (maps with
// boxes of 64 columns x 64 rows), dw [E, M, N] bf16, fully written.
cudaError_t launch_wgrad_pair(const CUtensorMap& m_a, const CUtensorMap& m_b, const int32_t* poff, void* dw, int E, int M,
                              int N, int32_t* status, cudaStream_t st) {
  cudaError_t e = set_pair_attributes();
  if (e != cudaSuccess) return e;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(dw);
  p.out_ld = N;
  p.expert_offsets = poff;
  p.tile_prefix = poff;      // not used by this mode (the table load needs a valid array)
  p.E = E;
  p.K = M;                   // rows of dw[e]
  p.N = N;
  p.n_tiles = (N + 255) / 256;
  p.status = status;
  ProfileScope prof(KID_WGRAD, st);
  return launch_pdl(ffn_gemm2_kernel<false, false, PAIR_WGRAD, false>, pair_grid(), THREADS, SMEM_BYTES, st, m_b, m_b, m_a,
                    m_a, p);
}

}  // namespace ffn
}  // namespace tcmoe
