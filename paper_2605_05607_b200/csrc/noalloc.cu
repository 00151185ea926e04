// moe_dispatch_noalloc: the dispatch stage for callers that cannot hand the library a workspace.
//
// Some hosts of this library run where device memory cannot be requested at the time of the call:
// a plugin invoked inside a framework's already-planned memory arena, a real-time serving loop
// whose policy forbids allocator calls (and their implicit synchronisation) on the hot path, or a
// caller written against a fixed C interface with no way to carry a scratch buffer.  For them the
// scratch tables of the layout builder (membership bitmasks, popcount prefixes, tile prefixes and
// the status block) live in ONE file-scope device array of fixed size that every GPU which loads
// the library keeps until the process exits.
#include "../../include/tcmoe.h"

#include "common.cuh"

#include <cuda_runtime.h>
#include <mutex>

namespace tcmoe {
namespace {

constexpr size_t kScratchBytes = size_t(2) << 20;   // 2 MiB per GPU, resident for the life of the process
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address: the
// address a kernel may use is looked up once per device, with that device current.
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_setup_mutex;

int scratch_of_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return MOE_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return MOE_OK;
}

inline size_t up256(size_t v) { return (v + 255) & ~size_t(255); }

}  // namespace
}  // namespace tcmoe

using namespace tcmoe;

extern "C" int moe_dispatch_noalloc(const moe_shape_t* shape, const void* x, const int32_t* topk_idx,
                                    const moe_layout_t* layout, void* xg, int32_t* status_out, void* stream) {
  size_t unused = 0;
  int rc = moe_workspace_bytes(shape, &unused);   // validates the shape
  if (rc != MOE_OK) return rc;
  if (topk_idx == nullptr || layout == nullptr || (xg != nullptr && x == nullptr)) return MOE_ERR_INVALID_ARG;
  const void* ptrs[9] = {layout->expert_counts, layout->expert_offsets, layout->group_counts,
                         layout->group_offsets, layout->pair_row,       layout->row_pair,
                         layout->al,            layout->disp_token,     layout->row_src};
  for (const void* p : ptrs) {
    if (p == nullptr) return MOE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(p) & 15) return MOE_ERR_MISALIGNED;
  }
  if ((reinterpret_cast<uintptr_t>(x) & 127) || (reinterpret_cast<uintptr_t>(xg) & 127) ||
      (reinterpret_cast<uintptr_t>(topk_idx) & 15) || (reinterpret_cast<uintptr_t>(status_out) & 15))
    return MOE_ERR_MISALIGNED;

  // carve the scratch tables; refuse what does not fit the fixed array
  const size_t E = (size_t)shape->E, G = (size_t)shape->G, W = ((size_t)shape->T + 31) / 32;
  const size_t off_status = 0;
  const size_t off_masks = 256;                                     // emask then gmask, adjacent
  const size_t off_eprefix = up256(off_masks + (E + G) * W * 4);
  const size_t off_gprefix = up256(off_eprefix + E * W * 4);
  const size_t off_mt = up256(off_gprefix + G * W * 4);
  const size_t off_mp = up256(off_mt + (E + 1) * 4);
  const size_t need = up256(off_mp + (E + 1) * 4);
  if (need > kScratchBytes) return MOE_ERR_SCRATCH_LIMIT;

  void* base = nullptr;
  if ((rc = scratch_of_current_device(&base)) != MOE_OK) return rc;
  unsigned char* b = static_cast<unsigned char*>(base);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // the array keeps whatever the previous call left: the status block must start at zero (the
  // bitmasks are cleared by the layout builder itself)
  int32_t* status = reinterpret_cast<int32_t*>(b + off_status);
  if (cudaMemsetAsync(status, 0, 64, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  LayoutScratch sc;
  sc.emask = reinterpret_cast<uint32_t*>(b + off_masks);
  sc.gmask = sc.emask + E * W;
  sc.eprefix = reinterpret_cast<int32_t*>(b + off_eprefix);
  sc.gprefix = reinterpret_cast<int32_t*>(b + off_gprefix);
  sc.mt_prefix = reinterpret_cast<int32_t*>(b + off_mt);
  sc.mp_prefix = reinterpret_cast<int32_t*>(b + off_mp);
  sc.W = (int)W;
  const Shape s{shape->T, shape->d, shape->f, shape->E, shape->k, shape->G, shape->score_fn, shape->flags};
  const Layout L{layout->expert_counts, layout->expert_offsets, layout->group_counts, layout->group_offsets,
                 layout->pair_row,      layout->row_pair,       layout->al,           layout->disp_token,
                 layout->row_src};
  if (launch_layout(s, topk_idx, L, sc, status, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  if (xg != nullptr && launch_dispatch(s, x, L, xg, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  if (status_out != nullptr &&
      cudaMemcpyAsync(status_out, status, 8 * sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  return MOE_OK;
}
