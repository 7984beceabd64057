// Host-side launch interface between the C ABI (lightkv_api.cu) and the kernel files.
#pragma once
#include <mutex>

#include "common.cuh"

namespace lkv {

// Launch with programmatic stream serialization (see grid_dependency_sync) and, for cluster > 1, a cluster
// of that many CTAs along x.
template <typename... P, typename... A>
inline cudaError_t launch_kernel(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 unsigned cluster, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

struct LayerLaunch {
  int batch, hidden, n_q_heads, n_kv_heads, head_dim;
  int dtype, xi_mode, divergence;
  double keep;
  int fd_tiles;                      // estimate of FdTiling::n_tiles per sample (launch shape of the tensor-core FD kernel)
  Geometry geo;
  Workspace ws;
  TextSet text;                      // prompt-token set J of this call
  const lightkv_layer_args_t* a;
  cudaStream_t stream;
};

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per (kernel, device) instead of before every launch.
struct SmemAttrEntry { const void* kernel; int dev; int bytes; };
inline cudaError_t ensure_dynamic_smem_ptr(const void* kernel, int bytes) {
  static std::mutex mu;
  static SmemAttrEntry table[64];
  static int used = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  SmemAttrEntry* e = nullptr;
  for (int i = 0; i < used; ++i)
    if (table[i].kernel == kernel && table[i].dev == dev) { e = &table[i]; break; }
  if (e && e->bytes >= bytes) return cudaSuccess;
  const cudaError_t rc = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (rc != cudaSuccess) return rc;
  if (!e && used < 64) e = &table[used++];
  if (e) { e->kernel = kernel; e->dev = dev; e->bytes = bytes; }
  return cudaSuccess;
}
template <typename... P>
inline cudaError_t ensure_dynamic_smem(void (*kernel)(P...), int bytes) {
  return ensure_dynamic_smem_ptr(reinterpret_cast<const void*>(kernel), bytes);
}

// window build (Step 1 and "Window partitioning")
cudaError_t launch_window_build(const LayerLaunch& L);
// FD + best partner per A node (Step 2), fp32 FMA path
cudaError_t launch_fd_simt(const LayerLaunch& L);
// xi per head (Eq. "attention-factor"), fp32 FMA path; handles ATTN_FULL and ATTN_LSE
cudaError_t launch_xi_simt(const LayerLaunch& L);
// head sum of xi, ranking, merge map, weights (Steps 2-5)
cudaError_t launch_select_map(const LayerLaunch& L);
// weighted merge of the hidden states (Eq. "message-passing")
cudaError_t launch_merge_rows(const LayerLaunch& L);

struct KvLaunch {
  int batch, n_kv_heads, head_dim, dtype, cap_in, cap_out;
  const lightkv_kv_args_t* a;
  cudaStream_t stream;
};
cudaError_t launch_kv_compact(const KvLaunch& K);

// tcgen05 paths (lightkv_tc.cu).  `supported` queries are host-only.
bool tc_fd_supported(int hidden);
bool tc_xi_supported(int head_dim);
cudaError_t launch_fd_tc(const LayerLaunch& L);
cudaError_t launch_xi_tc(const LayerLaunch& L);

}  // namespace lkv
