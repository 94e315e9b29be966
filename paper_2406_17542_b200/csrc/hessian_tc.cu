// Placeholder until the tcgen05 kernel lands: reports "not supported" so that every shape
// takes the SIMT kernel.
#include "common.cuh"
namespace cdq {
bool hessian_tc_supported(long long, long long, long long, const void*) { return false; }
size_t hessian_tc_workspace(long long, long long) { return 0; }
cudaError_t launch_hessian_tc(const void*, long long, long long, long long, int, float*, void*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace cdq
