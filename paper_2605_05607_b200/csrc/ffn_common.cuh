// Pieces shared by the two expert-FFN GEMM kernels (paper Sec. II-A GEMM-1 / GEMM-2): tile
// geometry, the device-side task decode, UMMA descriptors and small epilogue helpers.
#pragma once
#include "combine.cuh"
#include "common.cuh"
#include "ptx.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

namespace tcmoe {
namespace ffn {

constexpr int BM = 128;       // rows per CTA tile (the paper's tsize: 128-token tiles, Sec. VII-C)
constexpr int BK = 64;        // K per pipeline stage = one 128-byte swizzle row of bf16
constexpr int UMMA_N = 256;   // accumulator columns per tile
constexpr int MAX_E = 1024;

struct GemmParams {
  const void* a_src;            // GEMM-1 gather source (xg or x): bf16, or E4M3 codes in the FP8 form
  int a_ld;                     // elements per source row
  int a_rows;                   // rows of the gather source: indices outside [0, a_rows) are reported, not read
  const int32_t* gather_idx;    // row_src, or row_pair with gather_div = k (token = row_pair / k)
  int gather_div;
  __nv_bfloat16* out;
  int out_ld;
  const float* topk_w;          // GEMM-2 epilogue weights (NULL: 1)
  const int32_t* row_pair;
  const int32_t* expert_offsets;
  const int32_t* tile_prefix;   // exclusive prefix of tiles per expert (128-row tiles for GEMM-1,
                                // 256-row CTA-pair tiles for GEMM-2)
  int E, K, N, n_tiles;
  int32_t* status;
  // FP8 form only: per-row scale of the A operand (indexed like the A rows: gather source rows
  // for GEMM-1, expert-sorted rows for GEMM-2) and per-(expert, output column) scales of B
  const float* a_scale;
  const float* b_scale;         // [E, N]   (GEMM-1: W1)
  const float* b_scale2;        // [E, N]   (GEMM-1: W3)
  float* y_acc;                 // GEMM-2 with Combine in its epilogue: fp32 [T, N] accumulator, token
  int y_div;                    // of row r = row_pair[r] / y_div (NULL: rows go to `out`)
  // backward pass (pair kernel modes PAIR_GLU_BWD / PAIR_KSPLIT)
  const __nv_bfloat16* dh;      // [rows, N] incoming gradient of h (same leading dimension as out)
  __nv_bfloat16* out2;          // dA1 [rows, N]
  __nv_bfloat16* out3;          // dA3 [rows, N]
  int k_split;                  // k-blocks taken from each of the two (A, B) pairs
};

struct Tile {
  int e, n0, row0, rows;
  int out_row0, kb;   // weight-gradient tiles of the pair kernel: first output row of this CTA, k-blocks of the task
};

// Task w -> (expert, m-group, n-tile, m-tile in group): expert-major; inside an expert the m-tiles
// are taken in groups of M_GROUP, and inside a group the order is n-tile, m-tile fastest.  CTAs
// that run at the same time then share the weight tile (same expert, same n) in L2, and the
// activation rows that must stay in L2 while the n-tiles sweep over them are bounded by one
// m-group (a popular expert with hundreds of m-tiles would otherwise cycle all of its rows through
// L2 once per n-tile).  `rows_per_tile` is 128 (one CTA) or 256 (a CTA pair; CTA `rank` owns the
// rank-th half).  rows <= 0: nothing of this CTA is valid.
constexpr int M_GROUP_ROWS = 2048;   // rows of one m-group

__device__ __forceinline__ Tile decode_tile(int w, const int* tp, const int* eoff, int E, int n_tiles, int bn_out,
                                            int rows_per_tile, int rank) {
  int lo = 0, hi = E;  // tp[lo] * n_tiles <= w < tp[hi] * n_tiles
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tp[mid] * n_tiles <= w) lo = mid; else hi = mid;
  }
  int local = w - tp[lo] * n_tiles;
  const int mt = tp[lo + 1] - tp[lo];
  const int mg = M_GROUP_ROWS / rows_per_tile;          // m-tiles per full group
  const int g = local / (mg * n_tiles);                 // group index
  local -= g * mg * n_tiles;
  const int gsize = min(mg, mt - g * mg);               // m-tiles in this group
  Tile t;
  t.e = lo;
  t.n0 = (local / gsize) * bn_out;
  t.row0 = eoff[lo] + (g * mg + local % gsize) * rows_per_tile + rank * BM;
  t.rows = min(BM, eoff[lo + 1] - t.row0);
  t.out_row0 = t.row0;
  t.kb = 0;
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

// instruction descriptor of the FP8 form: D fp32, A/B E4M3 (format code 0), both K-major, N = 256, M = m
__host__ __device__ constexpr uint32_t idesc_e4m3(int m) {
  return (1u << 4) | (0u << 7) | (0u << 10) | (0u << 15) | (0u << 16) | ((uint32_t)(UMMA_N >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

// instruction descriptor: D fp32, A/B bf16, A K-major, B MN-major, N = 256, M = m
__host__ __device__ constexpr uint32_t idesc_bf16(int m) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(UMMA_N >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ float silu_mul(float a, float b) { return __fdividef(a, 1.f + __expf(-a)) * b; }

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Parameters of the tracker-paced kernel (ffn_fused.cu)
struct FusedParams {
  const void* x;                // GEMM-1 gather source (xg or x), bf16
  int x_ld;
  int x_rows;                   // rows of x: gather indices outside [0, x_rows) are reported, not read
  const int32_t* gather_idx;
  int gather_div;
  __nv_bfloat16* h;             // [P, f] intermediate
  __nv_bfloat16* o;             // [P, d] out
  const float* topk_w;          // GEMM-2 epilogue weights (NULL: 1)
  const int32_t* row_pair;
  const int32_t* expert_offsets;
  const int32_t* mt_prefix;     // [E+1] 128-row tile prefix: tracker slot base per expert
  // three task tables `tbl_stride` entries apart: interleaved, GEMM-1 blocks alone, GEMM-2 blocks alone
  const int32_t* blk_start;     // [3][tbl_stride] cumulative task counts of the task blocks (n_blocks + 1 used)
  const int4* blk_info;         // [3][tbl_stride] {0: GEMM-1 / 1: GEMM-2, expert, first row tile, row tiles}
  const int32_t* n_blocks;      // [3] device scalars
  int tbl_stride;
  int part_g1;                  // SM partition: CTAs [0, part_g1) take GEMM-1 tiles, the rest GEMM-2 tiles; 0: none
  // Tracker (Sec. IV-B), all zeroed before the launch.  Tile Status table, one entry per 128-row tile:
  int32_t* dacc;                //   DAcc   rows of the tile that Dispatch has written (NULL: no Dispatch tasks)
  int32_t* done;                //   TBCnt1 parts of the h tile stored by GEMM-1 (4 warps x n1 column tiles)
  int32_t* tbcnt2;              //   TBCnt2 parts of the o tile stored by GEMM-2 (4 warps x n2 column tiles)
  int32_t* nready;              // Output Readiness table: complete rows of o per token (NULL: no Combine tasks)
  int32_t* queue;               // [2] next Dispatch unit, next Combine chunk (work handed out in order)
  __nv_bfloat16* xs;            // per-expert layout tensors [P, d] written by the Dispatch tasks (with dacc)
  CombineArgs comb;             // Combine tasks (with nready)
  int T, k;
  int chunk_tokens;             // tokens per Combine chunk (1..32)
  int E, d, f, n1, n2;          // n1 = ceil(f / 128) GEMM-1 column tiles, n2 = ceil(d / 256) GEMM-2 column tiles
  int32_t* status;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// tensor maps (ffn.cu).  encode_tiled is the one place that calls cuTensorMapEncodeTiled; it keeps the most recent maps,
// keyed by every argument of the encode, and clear_map_cache forgets them.
bool encode_tiled(CUtensorMap* map, bool bytes, int rank, const void* base, const cuuint64_t* dims,
                  const cuuint64_t* strides, const cuuint32_t* box);
void clear_map_cache();
bool make_weight_map(CUtensorMap* map, const void* base, int E, int K, int N);
bool make_act_map(CUtensorMap* map, const void* base, long long rows, int K);
bool make_weight_map_fp8(CUtensorMap* map, const void* base, int E, int N, int K);
bool make_act_map_fp8(CUtensorMap* map, const void* base, int rows, int K);
bool make_weight_map_kmajor(CUtensorMap* map, const void* base, int E, int rows, int cols);
bool make_rows_map_mn(CUtensorMap* map, const void* base, long long rows, int cols);
cudaError_t launch_wgrad_pair(const CUtensorMap& m_a, const CUtensorMap& m_b, const int32_t* poff, void* dw, int E, int M,
                              int N, int32_t* status, cudaStream_t st);

// fp8 = false: bf16 operands, weights [E, K, N] (B MN-major).  fp8 = true: E4M3 operands, weights
// [E, N, K] (B K-major), 128 elements of K per pipeline stage, scales applied in the epilogue.
cudaError_t launch_gemm1(const GemmParams& p, const CUtensorMap& m_w1, const CUtensorMap& m_w3, bool fp8,
                         cudaStream_t st);
cudaError_t launch_gemm2(const GemmParams& p, const CUtensorMap& m_w2, const CUtensorMap& m_h, bool fp8,
                         cudaStream_t st);
cudaError_t launch_gemm1_pair(const GemmParams& p, const CUtensorMap& m_w1, const CUtensorMap& m_w3,
                              const CUtensorMap& m_xs, cudaStream_t st);
cudaError_t launch_bwd_dh(const GemmParams& p, const CUtensorMap& m_w2t, const CUtensorMap& m_do, cudaStream_t st);
cudaError_t launch_bwd_glu(const GemmParams& p, const CUtensorMap& m_w1, const CUtensorMap& m_w3, const CUtensorMap& m_xs,
                           cudaStream_t st);
cudaError_t launch_bwd_dx(const GemmParams& p, const CUtensorMap& m_w1t, const CUtensorMap& m_w3t, const CUtensorMap& m_da1,
                          const CUtensorMap& m_da3, cudaStream_t st);
size_t fused_max_blocks(int T, int k, int E);   // capacity of blk_start (+1) / blk_info for a shape
size_t fused_tracker_words(int T, int k, int E);   // int32 words of the tracker region (dacc | done | tbcnt2 | nready | queue)
cudaError_t launch_ffn_fused(FusedParams p, const int32_t* expert_counts, int32_t* blk_start, int4* blk_info,
                             int32_t* n_blocks, int32_t* tracker, const CUtensorMap& m_w1, const CUtensorMap& m_w3,
                             const CUtensorMap& m_w2, cudaStream_t st);
// GEMM-2 on 128-row single-CTA tiles (small experts): p.a_src / p.a_ld = h rows, no Combine-in-epilogue form
cudaError_t launch_gemm2_single(const GemmParams& p, const CUtensorMap& m_w2, bool fp8, cudaStream_t st);

}  // namespace ffn
}  // namespace tcmoe
