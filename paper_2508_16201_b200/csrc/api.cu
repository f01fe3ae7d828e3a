// Library identification and status strings.
#include "../../include/specvlm.h"

#include <cuda_runtime.h>

#include "common.cuh"
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

// Diagnostic: the bounded barrier wait every kernel of the library uses, on a barrier that nobody
// ever arrives at.  The wait gives up after limit_ns, raises the CTA's abort flag, and the kernel
// reports it the way the product kernels do; it then returns normally.
__global__ void wait_timeout_kernel(uint64_t limit_ns, int32_t* d_status, int32_t* d_flag_out) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    specvlm::mbar_init(specvlm::smem_u32(&bar), 1);
    abort_flag = 0;
    specvlm::mbar_fence_init();
  }
  __syncthreads();
  const bool ok = specvlm::mbar_wait_limit(specvlm::smem_u32(&bar), 0, &abort_flag, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0) {
    if (!ok && d_status) *d_status = SPECVLM_ERR_TIMEOUT;
    if (d_flag_out) *d_flag_out = abort_flag;
  }
}
}  // namespace

extern "C" int32_t specvlm_debug_wait_timeout(int32_t limit_ms, int32_t* d_status, int32_t* d_abort_flag_or_null,
                                              void* stream) {
  if (limit_ms < 1 || limit_ms > 1000 || !d_status) return SPECVLM_ERR_INVALID_ARG;
  wait_timeout_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>((uint64_t)limit_ms * 1000000ull, d_status,
                                                                       d_abort_flag_or_null);
  return cudaGetLastError() == cudaSuccess ? SPECVLM_OK : SPECVLM_ERR_CUDA;
}

extern "C" int32_t specvlm_debug_poison_shared_memory(void* stream) {
  constexpr int kBytes = 227 * 1024;                     // the most one CTA can own
  static std::atomic<uint64_t> attr_done{0};
  if (!specvlm::smem_attr_once(attr_done, reinterpret_cast<const void*>(poison_shared_kernel), kBytes))
    return SPECVLM_ERR_CUDA;
  // one CTA fills an SM; a few rounds, so that every SM is very likely visited
  poison_shared_kernel<<<4 * specvlm::sm_count(), 256, kBytes, static_cast<cudaStream_t>(stream)>>>(kBytes / 4);
  return cudaGetLastError() == cudaSuccess ? SPECVLM_OK : SPECVLM_ERR_CUDA;
}
