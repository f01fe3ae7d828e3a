// Host-side helpers: argument validation of specvlm_kv_t, tensor-map encoding, launch checks.
#pragma once
#include <atomic>

#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include "../../include/specvlm.h"

namespace specvlm {

// One NVTX range per entry point (named after it): shows the host side of every call on a profiler's
// timeline; without a profiler attached the two calls are empty stubs.
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Checks every documented requirement of a cache descriptor.  Returns SPECVLM_OK or an error.
inline int32_t validate_kv(const specvlm_kv_t* kv, int32_t batch, bool need_v) {
  if (!kv || !kv->k || (need_v && !kv->v) || !kv->seq_lens) return SPECVLM_ERR_INVALID_ARG;
  if (batch < 1 || kv->n_layers < 1 || kv->n_kv_heads < 1 || kv->block_tokens < 1 ||
      kv->n_blocks < 1 || kv->max_seq_len < 1)
    return SPECVLM_ERR_INVALID_ARG;
  if (kv->head_dim != 64 && kv->head_dim != 128) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(kv->k) || (need_v && !aligned16(kv->v))) return SPECVLM_ERR_INVALID_ARG;
  const int64_t strides[4] = {kv->stride_layer, kv->stride_block, kv->stride_head, kv->stride_token};
  for (int64_t s : strides)
    if (s < 0 || (s % 8) != 0) return SPECVLM_ERR_INVALID_ARG;
  if (kv->stride_token < kv->head_dim) return SPECVLM_ERR_INVALID_ARG;
  if (kv->block_table) {
    if (kv->block_tokens % 64 != 0) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
    if (kv->max_blocks < 1 ||
        (int64_t)kv->max_blocks * kv->block_tokens < (int64_t)kv->max_seq_len)
      return SPECVLM_ERR_INVALID_ARG;
  } else {
    if (kv->block_tokens < kv->max_seq_len || kv->n_blocks < batch) return SPECVLM_ERR_INVALID_ARG;
  }
  return SPECVLM_OK;
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                    const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                    const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline encode_tiled_fn get_encode_tiled() {
  // resolved once per process; a pure function pointer (threads that race here store the same value)
  static std::atomic<encode_tiled_fn> cached{nullptr};
  encode_tiled_fn fn = cached.load(std::memory_order_acquire);
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<encode_tiled_fn>(p);
    cached.store(fn, std::memory_order_release);
  }
  return fn;
}

// 5-D view (channel, token-in-block, head, block, layer) of one cache tensor with a
// (64 channels x box_tokens tokens) box and the 128-byte swizzle.
inline int32_t encode_kv_map(CUtensorMap* map, const specvlm_kv_t* kv, void* base, int box_tokens) {
  encode_tiled_fn enc = get_encode_tiled();
  if (!enc) return SPECVLM_ERR_CUDA;
  const cuuint64_t dims[5] = {(cuuint64_t)kv->head_dim, (cuuint64_t)kv->block_tokens,
                              (cuuint64_t)kv->n_kv_heads, (cuuint64_t)kv->n_blocks,
                              (cuuint64_t)kv->n_layers};
  // a dimension of extent 1 may carry any stride; give it a harmless non-zero one
  auto sb = [](int64_t s) { return (cuuint64_t)(s > 0 ? s : 8) * 2u; };
  const cuuint64_t strides[4] = {sb(kv->stride_token), sb(kv->stride_head), sb(kv->stride_block),
                                 sb(kv->stride_layer)};
  const cuuint32_t box[5] = {64u, (cuuint32_t)box_tokens, 1u, 1u, 1u};
  const cuuint32_t estr[5] = {1u, 1u, 1u, 1u, 1u};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPECVLM_OK : SPECVLM_ERR_CUDA;
}

inline int32_t launch_status() {
  return cudaGetLastError() == cudaSuccess ? SPECVLM_OK : SPECVLM_ERR_CUDA;
}

inline int sm_count() {
  // one process drives one GPU; the count of the first device seen is kept
  static std::atomic<int> cached{0};
  int n = cached.load(std::memory_order_relaxed);
  if (!n) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
    cached.store(n, std::memory_order_relaxed);
  }
  return n;
}

// The opt-in shared-memory size of a kernel is a per-device function attribute: it is set on a
// device's first launch of that kernel and remembered (one bit per device ordinal in `done`, a
// static of the launching function), so that later calls spend no host time on it.
inline bool smem_attr_once(std::atomic<uint64_t>& done, const void* kern, int bytes) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  const uint64_t bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_acquire) & bit) return true;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  done.fetch_or(bit, std::memory_order_release);
  return true;
}

}  // namespace specvlm
