// Cache maintenance around a speculative step: the K/V of the tokens a step feeds to a model are
// appended to that model's cache before its attention runs, and the rows of rejected drafts are
// dropped afterwards by shortening the sequence.  Pure byte movement and integer arithmetic.
//
// Sequence lengths, block tables and tree paths are device data: every value that becomes part
// of an address is range-checked in the kernels.  What fails a check is skipped (no access is
// made for it) and SPECVLM_ERR_INVALID_ARG is stored to d_status.
#include "common.cuh"
#include "host_util.h"

namespace specvlm {

struct AppendParams {
  const uint4* new_k;      // [L][B][n_new][Hkv][D] in 16-byte units
  const uint4* new_v;
  uint4* k;
  uint4* v;
  const int32_t* table;
  const int32_t* seq_lens; // lengths before the append
  int32_t* d_status;
  int64_t s_layer, s_block, s_head, s_token;   // cache strides in 16-byte units
  int32_t block_tokens, max_blocks, max_seq_len, n_blocks;
  int32_t n_layers, batch, n_new, n_kv_heads, chunks_per_row;
};

// one thread per 16-byte chunk of a new token row
__global__ void __launch_bounds__(256) append_kv_kernel(const __grid_constant__ AppendParams p) {
  const int64_t total = (int64_t)p.n_layers * p.batch * p.n_new * p.n_kv_heads * p.chunks_per_row;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t r = i;
    const int chunk = (int)(r % p.chunks_per_row); r /= p.chunks_per_row;
    const int head = (int)(r % p.n_kv_heads); r /= p.n_kv_heads;
    const int t = (int)(r % p.n_new); r /= p.n_new;
    const int b = (int)(r % p.batch);
    const int layer = (int)(r / p.batch);
    const int len = p.seq_lens[b];
    const int pos = len + t;
    if (len < 0 || len + p.n_new > p.max_seq_len) {
      // no room for all n_new rows (or a corrupt length): the sequence is left alone, every row of it
      if (p.d_status) *p.d_status = SPECVLM_ERR_INVALID_ARG;
      continue;
    }
    int blk = b, off = pos;
    if (p.table) {
      blk = __ldg(p.table + (size_t)b * p.max_blocks + pos / p.block_tokens);
      off = pos % p.block_tokens;
      if (blk < 0 || blk >= p.n_blocks) {
        if (p.d_status) *p.d_status = SPECVLM_ERR_INVALID_ARG;
        continue;
      }
    }
    const int64_t dst = layer * p.s_layer + blk * p.s_block + head * p.s_head + off * p.s_token + chunk;
    p.k[dst] = __ldcs(p.new_k + i);
    p.v[dst] = __ldcs(p.new_v + i);
  }
}

// seq_lens[b] += delta, or, with accept_len, seq_lens[b] -= gamma - accept_len[b]
__global__ void seq_len_update_kernel(int32_t* seq_lens, const int32_t* accept_len, int batch, int delta, int gamma,
                                      int max_seq_len, int32_t* d_status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  int n = seq_lens[b];
  if (accept_len) {
    const int a = accept_len[b];
    if (a < 0 || a > gamma || n < gamma + 1) {
      if (d_status) *d_status = SPECVLM_ERR_INVALID_ARG;
      return;
    }
    n -= gamma - a;
  } else {
    if (n < 0 || n + delta > max_seq_len) return;     // the append kernel has reported it
    n += delta;
  }
  seq_lens[b] = n;
}

struct CompactParams {
  uint4* k;
  uint4* v;
  const int32_t* table;
  const int32_t* seq_lens;   // lengths including the n_nodes window
  const int32_t* path;       // [B][n_nodes]: accepted nodes in order, then -1
  const int32_t* accept_len; // [B]
  int32_t* d_status;
  int64_t s_layer, s_block, s_head, s_token;
  int32_t block_tokens, max_blocks, n_blocks, max_seq_len, n_nodes, n_kv_heads, chunks_per_row;
};

// One CTA per (layer, KV head, sequence): the accepted nodes' rows move up behind the root.  A
// destination row can be a later move's source, so every row is read before any is written.
__global__ void __launch_bounds__(256) compact_tree_kernel(const __grid_constant__ CompactParams p) {
  const int b = blockIdx.y;
  const int layer = blockIdx.x / p.n_kv_heads, head = blockIdx.x - layer * p.n_kv_heads;
  const int n = min(max(p.accept_len[b], 0), p.n_nodes - 1);
  const int len = p.seq_lens[b];
  const int old = len - p.n_nodes;
  const int cpr = p.chunks_per_row;
  // address of (position, chunk), or -1 when the position's block-table entry is out of range
  auto addr = [&](int pos, int chunk) -> int64_t {
    int blk = b, off = pos;
    if (p.table) {
      blk = __ldg(p.table + (size_t)b * p.max_blocks + pos / p.block_tokens);
      off = pos % p.block_tokens;
      if (blk < 0 || blk >= p.n_blocks) return -1;
    }
    return layer * p.s_layer + blk * p.s_block + head * p.s_head + off * p.s_token + chunk;
  };
  constexpr int kMaxPerThread = 4;          // 63 rows x 16 chunks = 1008 chunks <= 4 x 256
  uint4 kk[kMaxPerThread], vv[kMaxPerThread];
  bool have[kMaxPerThread] = {false, false, false, false};
  if (old < 0 || len > p.max_seq_len) {     // tree_len_kernel reports the short sequence; a long one here
    if (len > p.max_seq_len && p.d_status && threadIdx.x == 0) *p.d_status = SPECVLM_ERR_INVALID_ARG;
    return;
  }
#pragma unroll
  for (int u = 0; u < kMaxPerThread; ++u) {
    const int idx = u * 256 + threadIdx.x;
    if (idx < n * cpr) {
      const int node = p.path[(size_t)b * p.n_nodes + idx / cpr];
      const int64_t a = node >= 1 && node < p.n_nodes ? addr(old + node, idx % cpr) : -1;
      if (a >= 0) {
        kk[u] = p.k[a];
        vv[u] = p.v[a];
        have[u] = true;
      } else if (p.d_status) {
        *p.d_status = SPECVLM_ERR_INVALID_ARG;
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int u = 0; u < kMaxPerThread; ++u) {
    const int idx = u * 256 + threadIdx.x;
    if (have[u]) {
      const int64_t a = addr(old + 1 + idx / cpr, idx % cpr);
      if (a >= 0) {
        p.k[a] = kk[u];
        p.v[a] = vv[u];
      } else if (p.d_status) {
        *p.d_status = SPECVLM_ERR_INVALID_ARG;
      }
    }
  }
}

// seq_lens[b] = seq_lens[b] - n_nodes + 1 + accept_len[b]
__global__ void tree_len_kernel(int32_t* seq_lens, const int32_t* accept_len, int batch, int n_nodes,
                                int32_t* d_status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int a = accept_len[b], n = seq_lens[b];
  if (a < 0 || a > n_nodes - 1 || n < n_nodes) {
    if (d_status) *d_status = SPECVLM_ERR_INVALID_ARG;
    return;
  }
  seq_lens[b] = n - n_nodes + 1 + a;
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int32_t specvlm_append_kv(const specvlm_kv_t* kv, const void* new_k, const void* new_v, int32_t batch,
                                     int32_t n_new, int32_t* seq_lens_inout, int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!kv || !new_k || !new_v || !seq_lens_inout || n_new < 1) return SPECVLM_ERR_INVALID_ARG;
  specvlm_kv_t c = *kv;
  c.seq_lens = seq_lens_inout;
  int32_t rc = validate_kv(&c, batch, true);
  if (rc != SPECVLM_OK) return rc;
  if (!aligned16(new_k) || !aligned16(new_v) || n_new > c.max_seq_len) return SPECVLM_ERR_INVALID_ARG;
  AppendParams p;
  p.new_k = static_cast<const uint4*>(new_k);
  p.new_v = static_cast<const uint4*>(new_v);
  p.k = static_cast<uint4*>(c.k);
  p.v = static_cast<uint4*>(c.v);
  p.table = c.block_table;
  p.seq_lens = seq_lens_inout;
  p.d_status = d_status;
  p.s_layer = c.stride_layer / 8; p.s_block = c.stride_block / 8; p.s_head = c.stride_head / 8;
  p.s_token = c.stride_token / 8;
  p.block_tokens = c.block_tokens; p.max_blocks = c.max_blocks; p.max_seq_len = c.max_seq_len;
  p.n_blocks = c.n_blocks;
  p.n_layers = c.n_layers; p.batch = batch; p.n_new = n_new; p.n_kv_heads = c.n_kv_heads;
  p.chunks_per_row = c.head_dim / 8;
  const int64_t total = (int64_t)p.n_layers * batch * n_new * p.n_kv_heads * p.chunks_per_row;
  int64_t blocks = (total + 255) / 256;
  const int64_t cap = (int64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  append_kv_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
  rc = launch_status();
  if (rc != SPECVLM_OK) return rc;
  // the lengths change only after every row has been placed by the kernel above
  seq_len_update_kernel<<<(unsigned)((batch + 127) / 128), 128, 0, st>>>(seq_lens_inout, nullptr, batch, n_new, 0,
                                                                         c.max_seq_len, d_status);
  return launch_status();
}

extern "C" int32_t specvlm_rollback_kv(int32_t* seq_lens_inout, const int32_t* accept_len, int32_t batch,
                                       int32_t gamma, int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!seq_lens_inout || !accept_len || batch < 1 || gamma < 0) return SPECVLM_ERR_INVALID_ARG;
  seq_len_update_kernel<<<(unsigned)((batch + 127) / 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      seq_lens_inout, accept_len, batch, 0, gamma, 0, d_status);
  return launch_status();
}

extern "C" int32_t specvlm_compact_tree_kv(const specvlm_kv_t* kv, const int32_t* path, const int32_t* accept_len,
                                           int32_t batch, int32_t n_nodes, int32_t* seq_lens_inout,
                                           int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!kv || !path || !accept_len || !seq_lens_inout || n_nodes < 1) return SPECVLM_ERR_INVALID_ARG;
  if (n_nodes > 64) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  specvlm_kv_t c = *kv;
  c.seq_lens = seq_lens_inout;
  int32_t rc = validate_kv(&c, batch, true);
  if (rc != SPECVLM_OK) return rc;
  if ((int64_t)c.n_layers * c.n_kv_heads > 0x7fffffff || batch > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  CompactParams p;
  p.k = static_cast<uint4*>(c.k);
  p.v = static_cast<uint4*>(c.v);
  p.table = c.block_table;
  p.seq_lens = seq_lens_inout;
  p.path = path;
  p.accept_len = accept_len;
  p.s_layer = c.stride_layer / 8; p.s_block = c.stride_block / 8; p.s_head = c.stride_head / 8;
  p.s_token = c.stride_token / 8;
  p.block_tokens = c.block_tokens; p.max_blocks = c.max_blocks; p.n_nodes = n_nodes;
  p.n_blocks = c.n_blocks; p.max_seq_len = c.max_seq_len; p.d_status = d_status;
  p.n_kv_heads = c.n_kv_heads; p.chunks_per_row = c.head_dim / 8;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  compact_tree_kernel<<<dim3((unsigned)(c.n_layers * c.n_kv_heads), (unsigned)batch), 256, 0, st>>>(p);
  rc = launch_status();
  if (rc != SPECVLM_OK) return rc;
  tree_len_kernel<<<(unsigned)((batch + 127) / 128), 128, 0, st>>>(seq_lens_inout, accept_len, batch, n_nodes,
                                                                   d_status);
  return launch_status();
}
