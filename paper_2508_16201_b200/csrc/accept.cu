// Step 4c: greedy acceptance.  Kernel 1 streams the fp32 logits once (16-byte loads, all of a
// thread's loads in flight together) and leaves one (max, lowest index) candidate per (row, vocab
// chunk); kernel 2 finishes the argmax of the gamma+1 rows of a sequence and counts the leading
// draft tokens that equal it.  Kernel 2 is launched with programmatic stream serialization: its
// CTAs are scheduled while kernel 1 still runs and wait (griddepcontrol.wait) for kernel 1's
// results, so the second launch costs no gap on the stream.
#include <mutex>

#include "common.cuh"
#include "host_util.h"

namespace specvlm {

constexpr int kAcceptThreads = 256;
constexpr int kAcceptVec = 8;                                      // float4 loads per thread, all issued up front
constexpr int kAcceptChunk = kAcceptThreads * kAcceptVec * 4;      // 8192 logits per CTA in kernel 1

struct Cand {
  float v;
  int32_t i;
};

// a is replaced by b when b is larger, or equal with a lower index
__device__ __forceinline__ void take_better(float& av, int& ai, float bv, int bi) {
  if (bv > av || (bv == av && bi < ai)) {
    av = bv;
    ai = bi;
  }
}

__global__ void __launch_bounds__(kAcceptThreads)
accept_partial_kernel(const float* __restrict__ logits, int vocab, int n_chunks, Cand* __restrict__ part) {
  // the dependent kernel may be scheduled from now on; it waits for this grid's completion itself
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int row = blockIdx.y, chunk = blockIdx.x;
  const float* base = logits + (size_t)row * vocab;
  const int lo = chunk * kAcceptChunk;
  const int hi = lo + kAcceptChunk < vocab ? lo + kAcceptChunk : vocab;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  if (((reinterpret_cast<uintptr_t>(base + lo)) & 15u) == 0) {
    const int n4 = (hi - lo) >> 2;
    const float4* b4 = reinterpret_cast<const float4*>(base + lo);
    float4 x[kAcceptVec];
#pragma unroll
    for (int u = 0; u < kAcceptVec; ++u) {
      const int k = threadIdx.x + u * kAcceptThreads;
      x[u] = k < n4 ? __ldcs(b4 + k) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
#pragma unroll
    for (int u = 0; u < kAcceptVec; ++u) {
      const int i0 = lo + 4 * (threadIdx.x + u * kAcceptThreads);
      // ascending index with strict '>' keeps the lowest index among equals
      if (x[u].x > bv) { bv = x[u].x; bi = i0; }
      if (x[u].y > bv) { bv = x[u].y; bi = i0 + 1; }
      if (x[u].z > bv) { bv = x[u].z; bi = i0 + 2; }
      if (x[u].w > bv) { bv = x[u].w; bi = i0 + 3; }
    }
    for (int i = lo + 4 * n4 + threadIdx.x; i < hi; i += kAcceptThreads) take_better(bv, bi, base[i], i);
  } else {
    for (int i = lo + threadIdx.x; i < hi; i += kAcceptThreads) take_better(bv, bi, base[i], i);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
    take_better(bv, bi, ov, oi);
  }
  __shared__ float sv[kAcceptThreads / 32];
  __shared__ int si[kAcceptThreads / 32];
  if ((threadIdx.x & 31) == 0) {
    sv[threadIdx.x >> 5] = bv;
    si[threadIdx.x >> 5] = bi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kAcceptThreads / 32; ++w) take_better(bv, bi, sv[w], si[w]);
    part[(size_t)row * n_chunks + chunk] = Cand{bv, bi};
  }
}

// one warp per (sequence, t); one CTA of (gamma+1) warps per sequence
__global__ void accept_finish_kernel(const Cand* part, int n_chunks,
                                     const int32_t* __restrict__ draft, int gamma,
                                     int32_t* __restrict__ accept_len, int32_t* __restrict__ next_token,
                                     int32_t* __restrict__ g_out) {
  __shared__ int g_sm[16];
  const int b = blockIdx.x, t = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Cand* row = part + ((size_t)b * (gamma + 1) + t) * n_chunks;
  asm volatile("griddepcontrol.wait;" ::: "memory");         // kernel 1 has completed, its candidates are visible
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int c = lane; c < n_chunks; c += 32) {
    const int2 raw = __ldcg(reinterpret_cast<const int2*>(row + c));     // from L2: written by the grid before
    take_better(bv, bi, __int_as_float(raw.x), raw.y);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
    take_better(bv, bi, ov, oi);
  }
  if (lane == 0) {
    g_sm[t] = bi;
    if (g_out) g_out[(size_t)b * (gamma + 1) + t] = bi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = 0;
    while (n < gamma && draft[(size_t)b * gamma + n] == g_sm[n]) ++n;
    accept_len[b] = n;
    next_token[b] = g_sm[n];
  }
}

// Tree drafting: one warp per node finishes its arg-max, then one thread walks from the root to
// the child whose token is the target's choice at the current node, as long as there is one.
__global__ void accept_tree_finish_kernel(const Cand* part, int n_chunks,
                                          const int32_t* __restrict__ node_tokens,
                                          const int32_t* __restrict__ parents, int n_nodes,
                                          int32_t* __restrict__ accept_len, int32_t* __restrict__ next_token,
                                          int32_t* __restrict__ path, int32_t* __restrict__ g_out) {
  __shared__ int g_sm[64];
  const int b = blockIdx.x, lane = threadIdx.x & 31;
  asm volatile("griddepcontrol.wait;" ::: "memory");         // kernel 1 has completed, its candidates are visible
  // a warp per node; with more than 32 nodes the warps take a second one each
  for (int t = threadIdx.x >> 5; t < n_nodes; t += blockDim.x >> 5) {
    const Cand* row = part + ((size_t)b * n_nodes + t) * n_chunks;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = lane; c < n_chunks; c += 32) {
      const int2 raw = __ldcg(reinterpret_cast<const int2*>(row + c));
      take_better(bv, bi, __int_as_float(raw.x), raw.y);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
      take_better(bv, bi, ov, oi);
    }
    if (lane == 0) {
      g_sm[t] = bi;
      if (g_out) g_out[(size_t)b * n_nodes + t] = bi;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int32_t* tok = node_tokens + (size_t)b * n_nodes;
    const int32_t* par = parents + (size_t)b * n_nodes;
    int32_t* pth = path + (size_t)b * n_nodes;
    int cur = 0, n = 0;
    while (true) {
      int nxt = -1;
      for (int c = cur + 1; c < n_nodes; ++c)
        if (par[c] == cur && tok[c] == g_sm[cur]) {
          nxt = c;
          break;
        }
      if (nxt < 0) break;
      pth[n++] = nxt;
      cur = nxt;
    }
    for (int i = n; i < n_nodes; ++i) pth[i] = -1;
    accept_len[b] = n;
    next_token[b] = g_sm[cur];
  }
}

// Launches `kern` so that it may be scheduled while the kernel before it in the stream still runs
// (programmatic stream serialization); the kernel itself waits for that kernel's results.
template <typename... KArgs, typename... Args>
static int32_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...) != cudaSuccess) return SPECVLM_ERR_CUDA;
  return launch_status();
}

// Built-in scratch of specvlm_accept_noalloc: room for kStaticCands (row, vocab chunk) candidates.
// Every GPU that loads the library holds these 128 KB until the process exits.
constexpr int kStaticCands = 16384;
static __device__ __align__(256) Cand g_accept_scratch[kStaticCands];

}  // namespace specvlm

using namespace specvlm;

extern "C" size_t specvlm_accept_workspace_bytes(int32_t batch, int32_t gamma, int32_t vocab) {
  if (batch < 1 || gamma < 0 || vocab < 1) return 0;
  const size_t n_chunks = ((size_t)vocab + kAcceptChunk - 1) / kAcceptChunk;
  return round_up((size_t)batch * (gamma + 1) * n_chunks * sizeof(Cand), 256);
}

extern "C" int32_t specvlm_accept(const float* target_logits, const int32_t* draft_tokens,
                                  int32_t batch, int32_t gamma, int32_t vocab, int32_t* accept_len,
                                  int32_t* next_token, int32_t* target_argmax_or_null, void* ws,
                                  size_t ws_bytes, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!target_logits || !accept_len || !next_token || batch < 1 || gamma < 0 || vocab < 1 || !ws)
    return SPECVLM_ERR_INVALID_ARG;
  if (gamma > 0 && !draft_tokens) return SPECVLM_ERR_INVALID_ARG;
  if (gamma > 15) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if ((int64_t)batch * (gamma + 1) > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(target_logits) & 3u) || (reinterpret_cast<uintptr_t>(ws) & 7u))
    return SPECVLM_ERR_INVALID_ARG;
  if (ws_bytes < specvlm_accept_workspace_bytes(batch, gamma, vocab)) return SPECVLM_ERR_WORKSPACE_TOO_SMALL;
  const int n_chunks = (vocab + kAcceptChunk - 1) / kAcceptChunk;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Cand* part = static_cast<Cand*>(ws);
  accept_partial_kernel<<<dim3((unsigned)n_chunks, (unsigned)(batch * (gamma + 1))), kAcceptThreads, 0, st>>>(
      target_logits, vocab, n_chunks, part);
  int32_t rc = launch_status();
  if (rc != SPECVLM_OK) return rc;
  return launch_dependent(accept_finish_kernel, dim3((unsigned)batch), dim3(32u * (gamma + 1)), st,
                          static_cast<const Cand*>(part), n_chunks, draft_tokens, gamma, accept_len, next_token,
                          target_argmax_or_null);
}

extern "C" int32_t specvlm_accept_noalloc(const float* target_logits, const int32_t* draft_tokens,
                                          int32_t batch, int32_t gamma, int32_t vocab, int32_t* accept_len,
                                          int32_t* next_token, int32_t* target_argmax_or_null, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!target_logits || !accept_len || !next_token || batch < 1 || gamma < 0 || vocab < 1)
    return SPECVLM_ERR_INVALID_ARG;
  if (gamma > 0 && !draft_tokens) return SPECVLM_ERR_INVALID_ARG;
  if (gamma > 15) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if ((int64_t)batch * (gamma + 1) > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if (reinterpret_cast<uintptr_t>(target_logits) & 3u) return SPECVLM_ERR_INVALID_ARG;
  const int n_chunks = (vocab + kAcceptChunk - 1) / kAcceptChunk;
  if ((int64_t)batch * (gamma + 1) * n_chunks > kStaticCands) return SPECVLM_ERR_TOO_LARGE;

  // Set-up, once per device: in host code the array's name is only a handle, the kernels need
  // the device address of this device's copy.
  constexpr int kMaxDevices = 64;
  static Cand* scratch_of[kMaxDevices] = {};
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPECVLM_ERR_CUDA;
  Cand* part;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!scratch_of[dev]) {
      void* addr = nullptr;
      if (cudaGetSymbolAddress(&addr, g_accept_scratch) != cudaSuccess || !addr) return SPECVLM_ERR_CUDA;
      scratch_of[dev] = static_cast<Cand*>(addr);
    }
    part = scratch_of[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // every candidate slot that kernel 2 reads is written by kernel 1 of the same call first, so
  // nothing left over from an earlier call has to be cleared
  accept_partial_kernel<<<dim3((unsigned)n_chunks, (unsigned)(batch * (gamma + 1))), kAcceptThreads, 0, st>>>(
      target_logits, vocab, n_chunks, part);
  int32_t rc = launch_status();
  if (rc != SPECVLM_OK) return rc;
  return launch_dependent(accept_finish_kernel, dim3((unsigned)batch), dim3(32u * (gamma + 1)), st,
                          static_cast<const Cand*>(part), n_chunks, draft_tokens, gamma, accept_len, next_token,
                          target_argmax_or_null);
}

extern "C" int32_t specvlm_accept_tree(const float* target_logits, const int32_t* node_tokens,
                                       const int32_t* parents, int32_t batch, int32_t n_nodes, int32_t vocab,
                                       int32_t* accept_len, int32_t* next_token, int32_t* path,
                                       int32_t* target_argmax_or_null, void* ws, size_t ws_bytes, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!target_logits || !node_tokens || !parents || !accept_len || !next_token || !path || !ws || batch < 1 ||
      n_nodes < 1 || vocab < 1)
    return SPECVLM_ERR_INVALID_ARG;
  if (n_nodes > 64 || (int64_t)batch * n_nodes > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(target_logits) & 3u) || (reinterpret_cast<uintptr_t>(ws) & 7u))
    return SPECVLM_ERR_INVALID_ARG;
  if (ws_bytes < specvlm_accept_workspace_bytes(batch, n_nodes - 1, vocab)) return SPECVLM_ERR_WORKSPACE_TOO_SMALL;
  const int n_chunks = (vocab + kAcceptChunk - 1) / kAcceptChunk;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Cand* part = static_cast<Cand*>(ws);
  accept_partial_kernel<<<dim3((unsigned)n_chunks, (unsigned)(batch * n_nodes)), kAcceptThreads, 0, st>>>(
      target_logits, vocab, n_chunks, part);
  int32_t rc = launch_status();
  if (rc != SPECVLM_OK) return rc;
  return launch_dependent(accept_tree_finish_kernel, dim3((unsigned)batch), dim3(32u * (n_nodes < 32 ? n_nodes : 32)), st,
                          static_cast<const Cand*>(part), n_chunks, node_tokens, parents, n_nodes, accept_len,
                          next_token, path, target_argmax_or_null);
}
