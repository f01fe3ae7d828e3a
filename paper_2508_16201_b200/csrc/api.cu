// Library identification and status strings.
#include "../../include/specvlm.h"

#include <cuda_runtime.h>

#include "host_util.h"

extern "C" const char* specvlm_version(void) { return "specvlm-b200 0.1 (sm_100a)"; }

extern "C" const char* specvlm_status_string(int32_t status) {
  switch (status) {
    case SPECVLM_OK: return "ok";
    case SPECVLM_ERR_INVALID_ARG: return "invalid argument";
    case SPECVLM_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case SPECVLM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SPECVLM_ERR_CUDA: return "CUDA call failed";
    case SPECVLM_ERR_TIMEOUT: return "device-side wait timed out";
    case SPECVLM_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of a no-allocation call";
    default: return "unknown status";
  }
}

// Diagnostic: every CTA overwrites its whole dynamic shared memory with NaN bit patterns.
namespace {
__global__ void poison_shared_kernel(int n_words) {
  extern __shared__ uint32_t poison_sm[];
  volatile uint32_t* sm = poison_sm;
  for (int i = threadIdx.x; i < n_words; i += blockDim.x) sm[i] = 0xffffffffu;
}
}  // namespace

extern "C" int32_t specvlm_debug_poison_shared_memory(void* stream) {
  constexpr int kBytes = 227 * 1024;                     // the most one CTA can own
  if (cudaFuncSetAttribute(poison_shared_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBytes) != cudaSuccess)
    return SPECVLM_ERR_CUDA;
  // one CTA fills an SM; a few rounds, so that every SM is very likely visited
  poison_shared_kernel<<<4 * specvlm::sm_count(), 256, kBytes, static_cast<cudaStream_t>(stream)>>>(kBytes / 4);
  return cudaGetLastError() == cudaSuccess ? SPECVLM_OK : SPECVLM_ERR_CUDA;
}
