// liblightkv kernels, part 2: tcgen05 tensor-core contractions (placeholder until the kernels land).
#include "launch.h"

namespace lkv {
bool tc_fd_supported(int) { return false; }
bool tc_xi_supported(int) { return false; }
cudaError_t launch_fd_tc(const LayerLaunch&) { return cudaErrorNotSupported; }
cudaError_t launch_xi_tc(const LayerLaunch&) { return cudaErrorNotSupported; }
}  // namespace lkv
