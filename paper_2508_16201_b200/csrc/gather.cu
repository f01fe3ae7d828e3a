// Step 3: compaction of the surviving video tokens' K/V rows (plus all text rows) into the
// draft cache.  Pure byte movement: 16-byte vector loads/stores, one (layer, KV head) slab per
// blockIdx.y, consecutive lanes on consecutive 16-byte chunks of a token row.
//
// The kept indices and the block tables are device data that the host cannot validate: every
// value that becomes part of an address is range-checked here.  A row whose index or block is out
// of range is skipped (nothing is read or written for it) and SPECVLM_ERR_INVALID_ARG is stored
// to d_status.
#include "common.cuh"
#include "host_util.h"

namespace specvlm {

constexpr int kGatherMaxBatch = 64;

struct GatherSeq {
  int32_t kept_off, kept_n, video_start, video_len, dst_len;
};

struct GatherParams {
  const uint4* src_k;
  const uint4* src_v;
  uint4* dst_k;
  uint4* dst_v;
  const int32_t* kept_idx;
  const int32_t* src_table;
  const int32_t* dst_table;
  int32_t* d_status;
  // strides in 16-byte units
  int64_t s_layer, s_block, s_head, s_token;
  int64_t d_layer, d_block, d_head, d_token;
  int32_t src_block_tokens, dst_block_tokens, src_max_blocks, dst_max_blocks, src_n_blocks, dst_n_blocks;
  int32_t n_kv_heads, chunks_per_row, batch0;
  GatherSeq seq[kGatherMaxBatch];
};

__global__ void __launch_bounds__(256) gather_kv_kernel(const __grid_constant__ GatherParams p) {
  const int bl = blockIdx.z;                 // sequence within this launch
  const GatherSeq sq = p.seq[bl];
  const int b = p.batch0 + bl;
  const int layer = blockIdx.y / p.n_kv_heads, head = blockIdx.y - layer * p.n_kv_heads;
  const int cpr = p.chunks_per_row;          // 8 (d = 64) or 16 (d = 128)
  const int rows_per_cta = 256 / cpr;
  const int chunk = threadIdx.x % cpr;
  for (int j = blockIdx.x * rows_per_cta + threadIdx.x / cpr; j < sq.dst_len;
       j += gridDim.x * rows_per_cta) {
    int sp;                                  // source token position
    bool ok = true;
    if (j < sq.video_start) {
      sp = j;
    } else if (j < sq.video_start + sq.kept_n) {
      const int kj = __ldg(p.kept_idx + sq.kept_off + (j - sq.video_start));
      ok = kj >= 0 && kj < sq.video_len;
      sp = sq.video_start + kj;
    } else {
      sp = j - sq.kept_n + sq.video_len;
    }
    int sblk = b, soff = sp;
    if (ok && p.src_table) {
      sblk = __ldg(p.src_table + (size_t)b * p.src_max_blocks + sp / p.src_block_tokens);
      soff = sp % p.src_block_tokens;
      ok = sblk >= 0 && sblk < p.src_n_blocks;
    }
    int dblk = b, doff = j;
    if (ok && p.dst_table) {
      dblk = __ldg(p.dst_table + (size_t)b * p.dst_max_blocks + j / p.dst_block_tokens);
      doff = j % p.dst_block_tokens;
      ok = dblk >= 0 && dblk < p.dst_n_blocks;
    }
    if (!ok) {
      if (p.d_status && chunk == 0) *p.d_status = SPECVLM_ERR_INVALID_ARG;
      continue;
    }
    const int64_t so = layer * p.s_layer + sblk * p.s_block + head * p.s_head + soff * p.s_token + chunk;
    const int64_t dof = layer * p.d_layer + dblk * p.d_block + head * p.d_head + doff * p.d_token + chunk;
    const uint4 kk = __ldcs(p.src_k + so);   // streamed: read once
    const uint4 vv = __ldcs(p.src_v + so);
    p.dst_k[dof] = kk;
    p.dst_v[dof] = vv;
  }
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int32_t specvlm_gather_kv(const specvlm_kv_t* src, const int32_t* kept_idx,
                                     const int32_t* kept_cu, const int32_t* video_start,
                                     const int32_t* video_len, const int32_t* src_len, int32_t batch,
                                     const specvlm_kv_t* dst, int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!src || !dst || !kept_idx || !kept_cu || !video_start || !video_len || !src_len || batch < 1)
    return SPECVLM_ERR_INVALID_ARG;
  // seq_lens are not read by this call; max_seq_len bounds the positions touched
  specvlm_kv_t s = *src, d = *dst;
  static const int32_t dummy = 0;
  if (!s.seq_lens) s.seq_lens = &dummy;
  if (!d.seq_lens) d.seq_lens = &dummy;
  int32_t rc = validate_kv(&s, batch, true);
  if (rc != SPECVLM_OK) return rc;
  rc = validate_kv(&d, batch, true);
  if (rc != SPECVLM_OK) return rc;
  if (s.n_layers != d.n_layers || s.n_kv_heads != d.n_kv_heads || s.head_dim != d.head_dim)
    return SPECVLM_ERR_INVALID_ARG;
  if ((int64_t)s.n_layers * s.n_kv_heads > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  int max_dst = 0;
  for (int b = 0; b < batch; ++b) {
    const int kn = kept_cu[b + 1] - kept_cu[b];
    if (kn < 0 || video_start[b] < 0 || video_len[b] < kn || src_len[b] < video_start[b] + video_len[b] ||
        src_len[b] > s.max_seq_len)
      return SPECVLM_ERR_INVALID_ARG;
    const int dl = src_len[b] - video_len[b] + kn;
    if (dl > d.max_seq_len) return SPECVLM_ERR_INVALID_ARG;
    if (dl > max_dst) max_dst = dl;
  }
  if (max_dst == 0) return SPECVLM_OK;

  GatherParams p;
  p.src_k = static_cast<const uint4*>(s.k);
  p.src_v = static_cast<const uint4*>(s.v);
  p.dst_k = static_cast<uint4*>(d.k);
  p.dst_v = static_cast<uint4*>(d.v);
  p.kept_idx = kept_idx;
  p.src_table = s.block_table;
  p.dst_table = d.block_table;
  p.s_layer = s.stride_layer / 8; p.s_block = s.stride_block / 8; p.s_head = s.stride_head / 8;
  p.s_token = s.stride_token / 8;
  p.d_layer = d.stride_layer / 8; p.d_block = d.stride_block / 8; p.d_head = d.stride_head / 8;
  p.d_token = d.stride_token / 8;
  p.src_block_tokens = s.block_tokens; p.dst_block_tokens = d.block_tokens;
  p.src_max_blocks = s.max_blocks; p.dst_max_blocks = d.max_blocks;
  p.src_n_blocks = s.n_blocks; p.dst_n_blocks = d.n_blocks;
  p.d_status = d_status;
  p.n_kv_heads = s.n_kv_heads;
  p.chunks_per_row = s.head_dim / 8;
  const int rows_per_cta = 256 / p.chunks_per_row;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  for (int b0 = 0; b0 < batch; b0 += kGatherMaxBatch) {
    const int nb = batch - b0 < kGatherMaxBatch ? batch - b0 : kGatherMaxBatch;
    int launch_max = 0;
    for (int i = 0; i < nb; ++i) {
      const int b = b0 + i;
      GatherSeq& q = p.seq[i];
      q.kept_off = kept_cu[b];
      q.kept_n = kept_cu[b + 1] - kept_cu[b];
      q.video_start = video_start[b];
      q.video_len = video_len[b];
      q.dst_len = src_len[b] - video_len[b] + q.kept_n;
      if (q.dst_len > launch_max) launch_max = q.dst_len;
    }
    p.batch0 = b0;
    int gx = (launch_max + rows_per_cta - 1) / rows_per_cta;
    if (gx > 64) gx = 64;                    // each CTA strides over the rest of its slab
    if (gx < 1) gx = 1;
    dim3 grid((unsigned)gx, (unsigned)(s.n_layers * s.n_kv_heads), (unsigned)nb);
    gather_kv_kernel<<<grid, 256, 0, st>>>(p);
    rc = launch_status();
    if (rc != SPECVLM_OK) return rc;
  }
  return SPECVLM_OK;
}
