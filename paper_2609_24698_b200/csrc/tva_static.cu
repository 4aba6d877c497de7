// tree_verify_attn_static: tree_verify_attn for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving engine that
// hands out all device memory from its own pool at start-up, inside a plug-in that must not
// touch the allocator of its host process, or at a point of a request loop where an allocation
// would stall every stream of the device.  They still pass their inputs and outputs, but have
// nowhere to get the call's workspace from.  This entry point keeps that workspace in a
// file-scope device array instead, so the call itself allocates nothing.
#include <cuda_runtime.h>

#include <atomic>

#include "tsv.h"

// The workspace.  Every GPU whose context loads this library holds these bytes until exit.
static __device__ __align__(256) unsigned char g_static_workspace[TSV_STATIC_WORKSPACE_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::atomic<void*> g_ws_addr[kMaxDevices];   // device address of the array, per device; null = not looked up yet
                                             // (threads that look it up at the same time store the same value)

// `g_static_workspace` in host code is only a handle for the symbol, not a device address:
// the address a kernel can use has to be asked for, per device, with that device current.
// The first look-up on a device also makes the runtime load this library's device code there,
// which is when the device reserves the array's bytes: it can fail on a device whose memory is
// already exhausted, so the first call belongs at start-up.
int static_workspace(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return TSV_ERR_CUDA; }
  void* p = g_ws_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) {
      cudaGetLastError();                    // leave no stale error behind for the next call's launch checks
      return TSV_ERR_CUDA;
    }
    g_ws_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return TSV_OK;
}

}  // namespace

extern "C" int tree_verify_attn_static(const tsv_shape* shape, const tsv_cache* cache, const tsv_nodes* nodes,
                                       const tsv_scratch* scratch, void* out, int32_t* topk_idx, int32_t* status,
                                       void* stream) {
  if (!shape) return TSV_ERR_NULL;
  const size_t need = tsv_workspace_bytes(shape);
  if (need == 0) return TSV_ERR_SHAPE;
  if (need > (size_t)TSV_STATIC_WORKSPACE_BYTES) return TSV_ERR_LIMIT;
  void* ws = nullptr;
  const int r = static_workspace(&ws);
  if (r != TSV_OK) return r;
  return tree_verify_attn(shape, cache, nodes, scratch, out, topk_idx, ws, (size_t)TSV_STATIC_WORKSPACE_BYTES, status, stream);
}
