// tree_verify_attn_static: tree_verify_attn for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving engine that
// hands out all device memory from its own pool at start-up, inside a plug-in that must not
// touch the allocator of its host process, or at a point of a request loop where an allocation
// would stall every stream of the device.  They still pass their inputs and outputs, but have
// nowhere to get the call's workspace from.  This entry point keeps that workspace in a
// file-scope device array instead, so the call itself allocates nothing.
#include <cuda_runtime.h>

#include "tsv.h"

// The workspace.  Every GPU whose context loads this library holds these bytes until exit.
static __device__ __align__(256) unsigned char g_static_workspace[TSV_STATIC_WORKSPACE_BYTES];

namespace {

constexpr int kMaxDevices = 64;
void* g_ws_addr[kMaxDevices];          // device address of the array, per device; 0 = not looked up yet

// `g_static_workspace` in host code is only a handle for the symbol, not a device address:
// the address a kernel can use has to be asked for, per device, with that device current.
int static_workspace(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TSV_ERR_CUDA;
  if (!g_ws_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return TSV_ERR_CUDA;
    g_ws_addr[dev] = p;
  }
  *out = g_ws_addr[dev];
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
