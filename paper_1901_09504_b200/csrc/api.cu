// Host-only entry points of the C ABI.
#include "common.cuh"

extern "C" const char* ocs_version(void) { return "ocs-b200 0.1 (sm_100a)"; }

extern "C" ocs_status ocs_poll_status(const int* dev_status, void* stream, int* host_out) {
  if (!dev_status || !host_out) return OCS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_out, dev_status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return OCS_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? OCS_OK : OCS_ERR_CUDA;
}
