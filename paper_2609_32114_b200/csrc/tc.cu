// Tensor-core (tcgen05) path: host side.  Placeholder until the kernels land.
#include "common.cuh"

namespace ha_la {
bool tc_supported(const Problem&) { return false; }
size_t tc_workspace_bytes(const Problem&) { return 0; }
int tc_num_launches(const Problem&) { return 0; }
cudaError_t launch_tc(const Problem&, const ha_la_prefill_args&, PlanView, void*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace ha_la
