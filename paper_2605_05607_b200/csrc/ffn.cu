// Host side of the expert FFN: TMA tensor maps and the two GEMM launches
// (GEMM-1 + SwiGLU in ffn_gemm1.cu, GEMM-2 + gate weight in ffn_gemm2.cu).
#include "ffn_common.cuh"

#include <atomic>
#include <mutex>

namespace tcmoe {
namespace ffn {

namespace {

EncodeTiledFn encode_fn() {
  static std::atomic<EncodeTiledFn> cached{nullptr};   // looked up once; a second lookup gives the same address
  EncodeTiledFn fn = cached.load(std::memory_order_acquire);
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(sym);
      cached.store(fn, std::memory_order_release);
    }
  }
  return fn;
}

// A tensor map is a pure function of (address, element size, rank, extents, strides, box): the same arguments give
// the same 128 bytes, whatever the memory holds.  The layer asks for the same handful of maps on every call (weights,
// workspace regions), so the most recent ones are kept, keyed by exactly those arguments.
struct MapKey {
  const void* base;
  int bytes, rank;
  cuuint64_t dims[3], strides[2];
  cuuint32_t box[3];
  bool operator==(const MapKey& o) const {
    return base == o.base && bytes == o.bytes && rank == o.rank && dims[0] == o.dims[0] && dims[1] == o.dims[1] &&
           dims[2] == o.dims[2] && strides[0] == o.strides[0] && strides[1] == o.strides[1] && box[0] == o.box[0] &&
           box[1] == o.box[1] && box[2] == o.box[2];
  }
};
struct MapEntry {
  MapKey key;
  CUtensorMap map;
};
constexpr int MAP_CACHE_ENTRIES = 64;
std::mutex g_map_mutex;
MapEntry g_map_cache[MAP_CACHE_ENTRIES];
int g_map_count = 0, g_map_next = 0;   // entries in use, next slot to overwrite (round robin)

}  // namespace

// Every map of this library: bf16 (bytes = 0) or one-byte (bytes = 1) elements, 128-byte swizzle, no interleave,
// 256-byte L2 promotion, zero fill outside the tensor.
bool encode_tiled(CUtensorMap* map, bool bytes, int rank, const void* base, const cuuint64_t* dims,
                  const cuuint64_t* strides, const cuuint32_t* box) {
  MapKey key{};
  key.base = base;
  key.bytes = bytes ? 1 : 0;
  key.rank = rank;
  for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides[i];
  {
    std::lock_guard<std::mutex> lock(g_map_mutex);
    for (int i = 0; i < g_map_count; ++i)
      if (g_map_cache[i].key == key) { *map = g_map_cache[i].map; return true; }
  }
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint32_t estr[3] = {1, 1, 1};
  if (fn(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
         const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  std::lock_guard<std::mutex> lock(g_map_mutex);
  MapEntry& e = g_map_cache[g_map_next];
  e.key = key;
  e.map = *map;
  g_map_next = (g_map_next + 1) % MAP_CACHE_ENTRIES;
  if (g_map_count < MAP_CACHE_ENTRIES) ++g_map_count;
  return true;
}

void clear_map_cache() {
  std::lock_guard<std::mutex> lock(g_map_mutex);
  g_map_count = 0;
  g_map_next = 0;
}

// bf16 weights [E, K, N] row-major: box = 64 (N) x 64 (K) x 1, 128-byte swizzle, zero fill
bool make_weight_map(CUtensorMap* map, const void* base, int E, int K, int N) {
  cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)K, (cuuint64_t)E};
  cuuint64_t strides[2] = {(cuuint64_t)N * 2, (cuuint64_t)N * K * 2};
  cuuint32_t box[3] = {64, BK, 1};
  return encode_tiled(map, false, 3, base, dims, strides, box);
}

// bf16 activations [rows, K] row-major: box = 64 (K) x 128 rows
bool make_act_map(CUtensorMap* map, const void* base, long long rows, int K) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {BK, BM};
  return encode_tiled(map, false, 2, base, dims, strides, box);
}

// E4M3 weights [E, N, K] (K contiguous): box = 128 bytes of K x 128 output columns x 1, 128-byte swizzle
bool make_weight_map_fp8(CUtensorMap* map, const void* base, int E, int N, int K) {
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)N, (cuuint64_t)E};
  cuuint64_t strides[2] = {(cuuint64_t)K, (cuuint64_t)N * K};
  cuuint32_t box[3] = {128, 128, 1};
  return encode_tiled(map, true, 3, base, dims, strides, box);
}

// E4M3 activations [rows, K]: box = 128 bytes of K x 128 rows
bool make_act_map_fp8(CUtensorMap* map, const void* base, int rows, int K) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K};
  cuuint32_t box[2] = {128, BM};
  return encode_tiled(map, true, 2, base, dims, strides, box);
}

// bf16 weights [E, K, N] read as the TRANSPOSED operand of a backward GEMM: the same memory seen as [E, N' = K, K' = N]
// with K' contiguous; box = 64 (K') x 128 (N') x 1, 128-byte swizzle.  `rows` = N', `cols` = K'.
bool make_weight_map_kmajor(CUtensorMap* map, const void* base, int E, int rows, int cols) {
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)E};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)rows * cols * 2};
  cuuint32_t box[3] = {64, 128, 1};
  return encode_tiled(map, false, 3, base, dims, strides, box);
}

// bf16 rows [rows, cols] read with the row index as K (weight gradients): box = 64 columns x 64 rows
bool make_rows_map_mn(CUtensorMap* map, const void* base, long long rows, int cols) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, 64};
  return encode_tiled(map, false, 2, base, dims, strides, box);
}

}  // namespace ffn

using ffn::make_weight_map;
using ffn::make_act_map;
using ffn::make_weight_map_fp8;
using ffn::make_act_map_fp8;

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    dev = 0;
  }
  return dev < 0 ? 0 : (dev >= MAX_DEVICES ? MAX_DEVICES - 1 : dev);
}

int sm_count() {
  static std::atomic<int> cached[MAX_DEVICES];
  const int dev = current_device();
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = 148;
    }
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

// Experts holding few rows on average: 256-row CTA-pair tiles would be mostly padding (a Zipf-routed
// 128-expert layer has most experts below 128 rows), so GEMM-2 takes 128-row single-CTA tiles.  Decided from the
// shape alone (the routing-dependent counts never visit the host); flag bits 32 (MOE_FLAG_GEMM2_PAIR) and 64
// (MOE_FLAG_GEMM2_SINGLE) force one form.
static bool small_experts(const Shape& s) {
  if (s.flags & 32) return false;
  if (s.flags & 64) return true;
  return (long long)s.T * s.k < 512ll * s.E;
}

size_t fused_table_blocks(const Shape& s) { return ffn::fused_max_blocks(s.T, s.k, s.E); }
size_t fused_tracker_bytes(const Shape& s) { return ffn::fused_tracker_words(s.T, s.k, s.E) * sizeof(int32_t); }

// flag bit 8 (MOE_FLAG_FUSED_FFN): both GEMMs in one persistent kernel paced by the tile tracker
static cudaError_t launch_expert_ffn_fused(const Shape& s, const FfnArgs& a, cudaStream_t st) {
  CUtensorMap m_w1, m_w3, m_w2;
  if (!make_weight_map(&m_w1, a.w1, s.E, s.d, s.f) || !make_weight_map(&m_w3, a.w3, s.E, s.d, s.f) ||
      !make_weight_map(&m_w2, a.w2, s.E, s.f, s.d))
    return cudaErrorInvalidValue;
  ffn::FusedParams p{};
  p.x = a.a_src;
  p.x_ld = s.d;
  p.x_rows = a.a_rows;
  p.gather_idx = a.gather_idx;
  p.gather_div = a.gather_div;
  p.h = static_cast<__nv_bfloat16*>(a.h);
  p.o = static_cast<__nv_bfloat16*>(a.o);
  p.topk_w = a.topk_w;
  p.row_pair = a.row_pair;
  p.expert_offsets = a.expert_offsets;
  p.mt_prefix = a.mt_prefix;
  p.blk_start = a.blk_start;
  p.blk_info = static_cast<const int4*>(a.blk_info);
  p.n_blocks = a.n_blocks;
  p.tbl_stride = (int)fused_table_blocks(s) + 1;
  // flag bit 16 (MOE_FLAG_SM_PARTITION): two thirds of the SMs for GEMM-1 (it has two thirds of the flops)
  p.part_g1 = (s.flags & 16) ? (2 * sm_count() + 1) / 3 : 0;
  p.E = s.E;
  p.d = s.d;
  p.f = s.f;
  p.T = s.T;
  p.k = s.k;
  p.n1 = (s.f + 127) / 128;
  p.n2 = (s.d + 255) / 256;
  p.status = a.status;
  p.comb = a.comb;                                        // comb.y == NULL: no Combine tasks
  p.xs = a.track_dispatch ? static_cast<__nv_bfloat16*>(a.xs) : nullptr;   // NULL: no Dispatch tasks
  return ffn::launch_ffn_fused(p, a.expert_counts, a.blk_start, static_cast<int4*>(a.blk_info), a.n_blocks, a.tracker,
                               m_w1, m_w3, m_w2, st);
}

cudaError_t launch_expert_ffn(const Shape& s, const FfnArgs& a, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  if ((s.flags & 8) && a.y_acc == nullptr && a.blk_start != nullptr) return launch_expert_ffn_fused(s, a, st);
  const int P = s.T * s.k;
  CUtensorMap m_w1, m_w3, m_w2, m_h;
  if (!make_weight_map(&m_w1, a.w1, s.E, s.d, s.f) || !make_weight_map(&m_w3, a.w3, s.E, s.d, s.f) ||
      !make_weight_map(&m_w2, a.w2, s.E, s.f, s.d) || !make_act_map(&m_h, a.h, P, s.f))
    return cudaErrorInvalidValue;

  ffn::GemmParams g1{};
  g1.a_src = static_cast<const __nv_bfloat16*>(a.a_src);
  g1.a_ld = s.d;
  g1.a_rows = a.a_rows;
  g1.gather_idx = a.gather_idx;
  g1.gather_div = a.gather_div;
  g1.out = static_cast<__nv_bfloat16*>(a.h);
  g1.out_ld = s.f;
  g1.expert_offsets = a.expert_offsets;
  g1.tile_prefix = a.mt_prefix;
  g1.E = s.E;
  g1.K = s.d;
  g1.N = s.f;
  g1.n_tiles = (s.f + 127) / 128;
  g1.status = a.status;
  cudaError_t err;
  if (a.pair_gemm1 && a.xs != nullptr) {
    // Dispatch writes the per-expert layout tensors, GEMM-1 runs on CTA pairs (MOE_FLAG_GEMM1_PAIR, or the shape rule)
    CUtensorMap m_xs;
    if (!make_act_map(&m_xs, a.xs, P, s.d)) return cudaErrorInvalidValue;
    if ((err = launch_permute_rows(s, a.a_src, a.a_rows, a.gather_idx, a.gather_div, a.expert_offsets, a.xs, a.status,
                                   st)) != cudaSuccess)
      return err;
    g1.tile_prefix = a.mp_prefix;
    err = ffn::launch_gemm1_pair(g1, m_w1, m_w3, m_xs, st);
  } else {
    err = ffn::launch_gemm1(g1, m_w1, m_w3, false, st);
  }
  if (err != cudaSuccess) return err;

  ffn::GemmParams g2{};
  g2.out = static_cast<__nv_bfloat16*>(a.o);
  g2.out_ld = s.d;
  g2.topk_w = a.topk_w;
  g2.row_pair = a.row_pair;
  g2.expert_offsets = a.expert_offsets;
  g2.tile_prefix = a.mp_prefix;
  g2.E = s.E;
  g2.K = s.f;
  g2.N = s.d;
  g2.n_tiles = (s.d + 255) / 256;
  g2.status = a.status;
  g2.y_acc = a.y_acc;
  g2.y_div = s.k;
  if (small_experts(s) && a.y_acc == nullptr) {
    g2.a_src = a.h;
    g2.a_ld = s.f;
    g2.tile_prefix = a.mt_prefix;
    return ffn::launch_gemm2_single(g2, m_w2, false, st);
  }
  return ffn::launch_gemm2(g2, m_w2, m_h, false, st);
}

// FP8 form: GEMM-1 on E4M3 rows and weights -> h (bf16) -> per-row quantisation of h -> GEMM-2 on E4M3.
cudaError_t launch_expert_ffn_fp8(const Shape& s, const FfnArgs& a, const Fp8Args& q, cudaStream_t st) {
  if (s.T == 0) return cudaSuccess;
  const int P = s.T * s.k;
  CUtensorMap m_w1, m_w3, m_w2, m_h;
  if (!make_weight_map_fp8(&m_w1, a.w1, s.E, s.f, s.d) || !make_weight_map_fp8(&m_w3, a.w3, s.E, s.f, s.d) ||
      !make_weight_map_fp8(&m_w2, a.w2, s.E, s.d, s.f) || !make_act_map_fp8(&m_h, q.hq, P, s.f))
    return cudaErrorInvalidValue;

  ffn::GemmParams g1{};
  g1.a_src = a.a_src;
  g1.a_ld = s.d;
  g1.a_rows = a.a_rows;
  g1.gather_idx = a.gather_idx;
  g1.gather_div = a.gather_div;
  g1.out = static_cast<__nv_bfloat16*>(a.h);
  g1.out_ld = s.f;
  g1.expert_offsets = a.expert_offsets;
  g1.tile_prefix = a.mt_prefix;
  g1.E = s.E;
  g1.K = s.d;
  g1.N = s.f;
  g1.n_tiles = (s.f + 127) / 128;
  g1.status = a.status;
  g1.a_scale = q.sx;
  g1.b_scale = q.s1;
  g1.b_scale2 = q.s3;
  cudaError_t err = ffn::launch_gemm1(g1, m_w1, m_w3, true, st);
  if (err != cudaSuccess) return err;
  if ((err = launch_quantize_rows(a.h, P, s.f, q.hq, q.sh, st)) != cudaSuccess) return err;

  ffn::GemmParams g2{};
  g2.out = static_cast<__nv_bfloat16*>(a.o);
  g2.out_ld = s.d;
  g2.topk_w = a.topk_w;
  g2.row_pair = a.row_pair;
  g2.expert_offsets = a.expert_offsets;
  g2.tile_prefix = a.mp_prefix;
  g2.E = s.E;
  g2.K = s.f;
  g2.N = s.d;
  g2.n_tiles = (s.d + 255) / 256;
  g2.status = a.status;
  g2.y_acc = a.y_acc;
  g2.y_div = s.k;
  g2.a_scale = q.sh;
  g2.b_scale = q.s2;
  if (small_experts(s) && a.y_acc == nullptr) {
    g2.a_src = q.hq;
    g2.a_ld = s.f;
    g2.tile_prefix = a.mt_prefix;
    return ffn::launch_gemm2_single(g2, m_w2, true, st);
  }
  return ffn::launch_gemm2(g2, m_w2, m_h, true, st);
}

}  // namespace tcmoe
