// lightkv_compress_layer_builtin_ws: lightkv_compress_layer for callers that cannot hand over a
// scratch buffer because they are not allowed to allocate device memory (a plug-in running inside
// a serving engine that owns the whole memory pool, a step replayed under a "no allocation" rule,
// a runtime whose allocator is frozen after start-up).  The stage's scratch lives in a
// file-scope device array of fixed size that belongs to the library image: every GPU that loads
// the library holds those bytes until the process exits.
//
// The array's name is only a host-side handle in host code.  Its device address is looked up once
// per device with cudaGetSymbolAddress (that device being current) and that pointer is what the
// kernels receive.
#include <mutex>

#include "launch.h"

namespace lkv {

static __device__ __align__(256) unsigned char g_builtin_ws[LIGHTKV_BUILTIN_WS_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_mutex;
static void* g_ws_addr[kMaxDevices];          // device address of g_builtin_ws on each ordinal, once known

// Address of the built-in scratch on the current device; nullptr when the lookup fails.
static void* builtin_ws_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_ws_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_builtin_ws) != cudaSuccess) return nullptr;
    g_ws_addr[dev] = p;
  }
  return g_ws_addr[dev];
}

}  // namespace lkv

extern "C" int lightkv_compress_layer_builtin_ws(const lightkv_plan_t* plan, const lightkv_layer_args_t* args) {
  if (!plan || !args || args->struct_size != sizeof(lightkv_layer_args_t)) return LIGHTKV_ERR_INVALID_ARG;
  lightkv_stage_info_t info;
  const int rc = lightkv_plan_stage_info(plan, args->stage, &info);
  if (rc != LIGHTKV_OK) return rc;
  if (info.workspace_bytes > size_t(LIGHTKV_BUILTIN_WS_BYTES)) return LIGHTKV_ERR_WORKSPACE;
  void* ws = lkv::builtin_ws_for_current_device();
  if (!ws) return LIGHTKV_ERR_CUDA;
  lightkv_layer_args_t a = *args;              // the caller's workspace fields are ignored
  a.workspace = ws;
  a.workspace_bytes = size_t(LIGHTKV_BUILTIN_WS_BYTES);
  return lightkv_compress_layer(plan, &a);
}
