// Parameters shared by the attention kernels and their launchers.
#pragma once
#include "common.cuh"

namespace specvlm {

struct AttnParams {
  const __nv_bfloat16* q;     // [L][B][n_q][Hq][D]
  __nv_bfloat16* out;         // same shape
  float* lse;                 // [L][B][n_q][Hq] or null
  float* ws_o;                // split partials: [item][split][rows][D], normalised
  float* ws_lse;              // [item][split][rows], log2 units
  int32_t* ws_cnt;            // [item] arrival counters of the splits, zero at launch
  const int32_t* block_table; // [B][max_blocks] or null
  const int32_t* seq_lens;    // [B]
  int32_t* d_status;
  int32_t batch, n_q, n_q_heads, n_kv_heads, group, rows;   // rows = group * n_q
  int32_t n_splits, max_blocks, block_tokens, max_seq_len;
  float scale_log2;           // sm_scale * log2(e)
};

// Tiles of kTileTokens owned by one split of a sequence of kv_len tokens.
__host__ __device__ inline void split_range(int kv_len, int n_splits, int split, int& tile_begin,
                                            int& tile_end) {
  const int n_tiles = (kv_len + kTileTokens - 1) / kTileTokens;
  const int per = (n_tiles + n_splits - 1) / n_splits;
  tile_begin = split * per;
  tile_end = tile_begin + per < n_tiles ? tile_begin + per : n_tiles;
  if (tile_begin > tile_end) tile_begin = tile_end;
}

}  // namespace specvlm
