// Step 1a: token rating from the verifier's language-to-video attention.
//
// The rating of video token j is the mean, over layers, query heads and language queries, of the
// causal softmax probability the query puts on j.  This is a dense contraction (every language
// query row against every key), so it runs on the tensor cores, in two passes over QK^T:
//   pass 1 (row-centric)   the log-sum-exp of every language query row over all its causal keys;
//   pass 2 (column-centric) P = 2^(s - lse) recomputed tile by tile and summed down the rows.
// The full attention matrix is never stored.  All reductions run in a fixed order: per-layer
// partial column sums, then one ordered sum over layers.
//
// Rows of a (layer, KV head) problem are the language queries times the group's heads, in the
// order r = i * group + head_in_group; a row tile holds QT = floor(128 / group) queries.
#include <type_traits>

#include "common.cuh"
#include "host_util.h"

namespace specvlm {

constexpr int kScoresMaxBatch = 64;
constexpr int kKeyTile = 128;          // keys per CTA tile (two cache pages)

struct ScoreSeq {
  int32_t text_off, n_text, text_start, video_start, n_video, score_off;
  int32_t tile_off;                    // first CTA index (pass 1: row tiles, pass 2: key blocks)
};

struct ScoreParams {
  const __nv_bfloat16* q;              // [L][sum_text][Hq][D]
  float* lse;                          // [L][sum_text][Hq]: natural-log sum-exp of the scaled logits
  float* partial;                      // [L][sum_video]
  const int32_t* block_table;
  int32_t* d_status;
  int32_t batch, n_layers, n_q_heads, n_kv_heads, group, qt, sum_text, sum_video;
  int32_t max_blocks, block_tokens;
  float scale_log2;
  ScoreSeq seq[kScoresMaxBatch];
};

__device__ __forceinline__ int find_seq(const ScoreParams& p, int cta) {
  int b = 0;
  while (b + 1 < p.batch && p.seq[b + 1].tile_off <= cta) ++b;
  return b;
}

// issue the TMA loads of one 128-key K tile (two 64-token pages, D/64 channel halves each)
template <int D>
__device__ __forceinline__ void load_key_tile(const CUtensorMap* tm_k, const ScoreParams& p, int b,
                                              int g, int layer, int key0, uint32_t dst, uint32_t bar,
                                              uint64_t policy) {
#pragma unroll
  for (int pg = 0; pg < 2; ++pg) {
    const int tok0 = key0 + pg * 64;
    int blk = b, tok = tok0;
    if (p.block_table) {
      const int lblk = tok0 / p.block_tokens;
      // past the sequence's last page: an out-of-range block coordinate reads zeros
      blk = lblk < p.max_blocks ? p.block_table[(size_t)b * p.max_blocks + lblk] : -1;
      tok = tok0 % p.block_tokens;
    }
#pragma unroll
    for (int h = 0; h < D / 64; ++h)
      tma_load_5d(dst + h * (kKeyTile * 128) + pg * (64 * 128), tm_k, bar, h * 64, tok, g, blk, layer,
                  policy);
  }
}

// Some of the exponentials are taken on the FMA pipe (f2_exp2_poly) instead of the special-function
// unit, which both rating passes nearly saturate.  The polynomial costs about as many FMA-pipe cycles
// per value as the unit it relieves (8) plus issue slots, so only a small share pays, and the best
// share is a measured one (80 layers of 6272 video tokens, same box within a row of figures).
// Pass 1: 3 of the 16 pairs of a 32-column chunk, pairs 3, 7 and 11 (2 / 4 / 6 / 8 of 16 in an
// earlier form: 1144 / 1106 / 1175 / 1224 us; then 3 / 4 / 5 / 6 of 16: 1108 / 1143 / 1135 / 1173 us).
// Which pairs matters to the compiler: under this kernel's 96-register cap pairs {3, 7, 11} compile
// without a spill, {3, 11} and {2, 7, 12} with 400-850 bytes of spills and run 2-4 times slower.
// Pass 2: 2 of the 16 pairs, pairs 0 and 8 (0 / 1 / 2 / 3 / 4 / 6 / 8 of 16: 1208 / 1152 / 1141-1156 /
// 1158 / 1188 / 1245 / 1286 us); the place matters here too: pairs {3, 11} or {5, 13} take 1254 us,
// {7, 15} 1166, {0, 2} 1174, {0, 14} 1125 against 1133-1137 for {0, 8} on the same box.
constexpr uint32_t kPolyMaskLse = 0x0888u;             // bit i: pair i of a chunk takes the polynomial
constexpr uint32_t kPolyMaskColsum = 0x0101u;          // bit i: pair i of a chunk takes the polynomial

// ---------------------------------------------------------------------------------------------
// Pass 2 on the 5th-generation tensor cores.  CTA = (block of 128 video keys, layer), looping over
// the layer's KV heads and, for each, over all row tiles of the sequence:
//   D[key][row] = K_block (A: 128 keys x d, K-major) * Q_tile^T (B: 128 rows x d, K-major)
// is one chain of tcgen05.mma instructions (M = N = 128, K = 16 each) issued by a single thread,
// with both operands read straight from the 128-byte-swizzled tiles the TMA wrote and the fp32
// accumulator in tensor memory (one 128-column buffer per epilogue group, so the MMAs of the next
// tiles overlap the epilogues of the current ones).  With the keys on the TMEM lanes, an epilogue
// thread owns one key: it reads its 128 row values with tcgen05.ld and adds up 2^(s - lse_row) in
// registers for the whole layer -- the column sum needs no cross-thread reduction inside a group;
// the groups' sums meet once, at the end, in a fixed order.
// Warps: 0 = TMA producer, 1 = TMEM allocation + MMA issue, then kColsumGroups epilogue groups of
// four warps (one TMEM lane quadrant per warp) that take the tiles round-robin, each on its own
// accumulator buffer: four warps per scheduler keep the special-function unit busy while others
// wait for a TMEM load, a barrier or the row statistics.
// ---------------------------------------------------------------------------------------------
constexpr int kColsumGroups = 4;
constexpr int kColsumThreads = 64 + 128 * kColsumGroups;

template <int D, int STAGES>
__global__ void __launch_bounds__(kColsumThreads, 1)
scores_colsum_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                        const __grid_constant__ ScoreParams p) {
  constexpr int TILE_BYTES = kKeyTile * D * 2;
  constexpr int KSTEPS = D / 16;
  constexpr int NG = kColsumGroups;
  constexpr uint32_t kTmemCols = 128 * NG;
  static_assert(kTmemCols == 256 || kTmemCols == 512, "tensor memory is allocated in powers of two");
  constexpr uint32_t kIdesc = umma_idesc_bf16(128, 128, false, false);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* const smem = smem_raw + (base - raw_addr);
  const uint32_t k_sm = base;                                    // 2 K-block buffers
  const uint32_t q_sm = base + 2 * TILE_BYTES;                   // Q ring
  constexpr int kTail = (2 + STAGES) * TILE_BYTES;
  const uint32_t bar_qfull = base + kTail;
  const uint32_t bar_qempty = bar_qfull + 8 * STAGES;
  const uint32_t bar_kfull = bar_qempty + 8 * STAGES;            // [2]
  const uint32_t bar_kempty = bar_kfull + 16;                    // [2]
  const uint32_t bar_tfull = bar_kempty + 16;                    // [NG]
  const uint32_t bar_tempty = bar_tfull + 8 * NG;                // [NG]
  uint8_t* const tail = smem + kTail + 16 * STAGES + 32 + 16 * NG;
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail + 8);
  float* const lse_sm = reinterpret_cast<float*>(tail + 16);     // [NG groups][2][128]: -lse in log2 units

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = find_seq(p, blockIdx.x);
  const ScoreSeq sq = p.seq[b];
  const int kblock = blockIdx.x - sq.tile_off;
  const int layer = blockIdx.y;
  const int key0 = (sq.video_start / 64) * 64 + kblock * kKeyTile;
  const int n_qt = (sq.n_text + p.qt - 1) / p.qt;
  const int n_units = p.n_kv_heads;
  const int n_tiles = n_units * n_qt;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_qfull + 8 * s, 1);
      mbar_init(bar_qempty + 8 * s, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_kfull + 8 * i, 1);
      mbar_init(bar_kempty + 8 * i, 1);
    }
    for (int i = 0; i < NG; ++i) {
      mbar_init(bar_tfull + 8 * i, 1);
      mbar_init(bar_tempty + 8 * i, 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  {
    // A row tile holds qt * group rows; the TMA box never writes the rows after them, and whatever
    // the shared memory held there would reach every key's sum through the product (a NaN times a
    // vanishing weight is still a NaN).  They are cleared once: row r of a tile is the 128 bytes at
    // r * 128 of each 64-channel block, whatever the swizzle does inside a row.
    const int rows_used = p.qt * p.group;
    const int n16 = (kKeyTile - rows_used) * 8;                    // 16-byte units per block
    for (int i = tid; i < STAGES * (D / 64) * n16; i += blockDim.x) {
      const int blk = i / n16, u = i - blk * n16;
      *reinterpret_cast<uint4*>(smem + 2 * TILE_BYTES + blk * (kKeyTile * 128) + rows_used * 128 + u * 16) =
          make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async();                                           // the MMAs read it through the async proxy
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_q);
      const uint64_t pol_k = l2_policy_evict_first();
      const uint64_t pol_q = l2_policy_evict_last();             // Q is re-read by every key block
      const uint32_t q_tx = (D / 64) * p.qt * p.group * 128;     // bytes of one Q box set
      bool ok = true;
      int qi = 0;
      for (int u = 0; u < n_units && ok; ++u) {
        const int kb = u & 1;
        if (u >= 2) ok = mbar_wait(bar_kempty + 8 * kb, ((u >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(bar_kfull + 8 * kb, TILE_BYTES);
        load_key_tile<D>(&tm_k, p, b, u, layer, key0, k_sm + kb * TILE_BYTES, bar_kfull + 8 * kb, pol_k);
        for (int t = 0; t < n_qt && ok; ++t, ++qi) {
          const int s = qi % STAGES;
          if (qi >= STAGES) ok = mbar_wait(bar_qempty + 8 * s, ((qi / STAGES) - 1) & 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(bar_qfull + 8 * s, q_tx);
#pragma unroll
          for (int h = 0; h < D / 64; ++h)
            tma_load_5d(q_sm + s * TILE_BYTES + h * (kKeyTile * 128), &tm_q, bar_qfull + 8 * s, h * 64, 0, u,
                        sq.text_off + t * p.qt, layer, pol_q);
        }
      }
      if (!ok) {
        if (p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
        const uint64_t t0 = global_timer_ns();
        for (int i = qi > STAGES ? qi - STAGES : 0; i < qi; ++i)
          while (!mbar_try_wait(bar_qfull + 8 * (i % STAGES), (i / STAGES) & 1) &&
                 global_timer_ns() - t0 < kWaitLimitNs) {
          }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issue (one thread)
    if (lane == 0) {
      bool ok = true;
      int it = 0;
      for (int u = 0; u < n_units && ok; ++u) {
        const int kb = u & 1;
        ok = mbar_wait(bar_kfull + 8 * kb, (u >> 1) & 1, abort_flag);
        for (int t = 0; t < n_qt && ok; ++t, ++it) {
          const int s = it % STAGES, buf = it % NG;
          ok = mbar_wait(bar_qfull + 8 * s, (it / STAGES) & 1, abort_flag);
          if (ok && it >= NG) ok = mbar_wait(bar_tempty + 8 * buf, ((it / NG) - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a0 = k_sm + kb * TILE_BYTES, b0 = q_sm + s * TILE_BYTES;
#pragma unroll
          for (int ks = 0; ks < KSTEPS; ++ks) {
            // 16 channels per step: 32 bytes along the swizzled 128-byte row; channels 64.. live
            // in the second half-tile
            const uint32_t off = (ks >> 2) * (kKeyTile * 128) + (ks & 3) * 32;
            umma_bf16_ss(tmem_base + buf * 128, umma_desc_sw128(a0 + off, 16, 1024),
                         umma_desc_sw128(b0 + off, 16, 1024), kIdesc, ks > 0 ? 1u : 0u);
          }
          umma_commit(bar_qempty + 8 * s);      // the Q stage is free once these MMAs have read it
          umma_commit(bar_tfull + 8 * buf);     // and the accumulator buffer is complete
        }
        if (ok) umma_commit(bar_kempty + 8 * kb);
      }
      if (!ok && p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
    }
  } else {
    // ---------------------------------------------------------------- epilogue: NG groups x 4 warps, 128 keys
    const int grp = (warp - 2) >> 2;            // tiles with index % NG == grp, accumulator buffer grp
    const int quad = warp & 3;                  // TMEM lanes [32 * quad, 32 * quad + 32)
    const int key_l = quad * 32 + lane;         // this thread's key inside the block
    const int et = ((warp - 2) & 3) * 32 + lane;   // 0..127 inside the group: used to stage the row LSEs
    float* const lse_g = lse_sm + grp * 256;    // this group's two staging buffers of 128 rows
    // -lse (log2 units) of row `et` of the tile (KV head fu, row tile ft); -inf for rows past the valid
    // ones, whose exponentials then vanish.  (fu, ft) walk this group's tiles ahead of the loop
    // below: no division per tile, and the address is two multiply-adds off a fixed base.
    const int il = et / p.group, hg = et - il * p.group;
    const float* const lse_row =
        p.lse + ((size_t)layer * p.sum_text + sq.text_off + il) * p.n_q_heads + hg;
    int fu = 0, ft = grp;                       // the tile the next lse_fetch() is for
    while (ft >= n_qt) {
      ft -= n_qt;
      ++fu;
    }
    auto lse_fetch = [&]() -> float {
      float v = 0.f;
      if (fu < n_units) {
        const int rows_valid = min(p.qt, sq.n_text - ft * p.qt) * p.group;
        v = et < rows_valid ? -__ldg(lse_row + (size_t)(ft * p.qt) * p.n_q_heads + fu * p.group) * kLog2e : -INFINITY;
      }
      ft += NG;                                 // this group's next tile
      while (ft >= n_qt) {
        ft -= n_qt;
        ++fu;
      }
      return v;
    };
    uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};   // four chains of pairs for instruction-level parallelism
    bool alive = true;
    float lv = lse_fetch();
    int n = 0;
    for (int it = grp; it < n_tiles; it += NG, ++n) {
      const int buf = grp;
      float* const ls = lse_g + (n & 1) * 128;
      ls[et] = lv;
      // one barrier per tile: the buffer written here was last read two tiles ago, before the
      // previous tile's barrier
      asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory");
      lv = lse_fetch();                         // the next tile's: in flight during this tile's exponentials
      if (alive && !mbar_wait(bar_tfull + 8 * buf, (it / NG) & 1, abort_flag)) alive = false;
      alive = __all_sync(0xffffffffu, alive);   // warp-uniform: the TMEM loads below are warp-collective
      if (!alive) continue;                     // keep taking part in the barrier above
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * 128;
      const uint64_t sc2 = f2_pack(p.scale_log2, p.scale_log2);
      uint32_t va[32], vb[32];                  // the load of chunk c + 1 flies while chunk c is summed
      tmem_ld_x32(taddr, va);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t(&v)[32] = (c & 1) ? vb : va;
        tmem_ld_wait();
        if (c < 3) {
          tmem_ld_x32(taddr + (c + 1) * 32, (c & 1) ? va : vb);
        } else {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);   // buffer free for the MMAs of tile it + NG
        }
#pragma unroll
        for (int q = 0; q < 16; q += 2) {
          const float4 l4 = *reinterpret_cast<const float4*>(ls + c * 32 + 2 * q);
          const uint64_t ta = f2_fma(f2_pack(__uint_as_float(v[2 * q]), __uint_as_float(v[2 * q + 1])), sc2,
                                     f2_pack(l4.x, l4.y));
          const uint64_t tb = f2_fma(f2_pack(__uint_as_float(v[2 * q + 2]), __uint_as_float(v[2 * q + 3])), sc2,
                                     f2_pack(l4.z, l4.w));
          acc2[q & 3] = f2_add(acc2[q & 3], ((kPolyMaskColsum >> q) & 1) ? f2_exp2_poly(ta) : f2_exp2_sfu(ta));
          acc2[(q + 1) & 3] = f2_add(acc2[(q + 1) & 3], ((kPolyMaskColsum >> (q + 1)) & 1) ? f2_exp2_poly(tb) : f2_exp2_sfu(tb));
        }
      }
    }
    float acc;
    {
      float s0, s1, s2, s3, s4, s5, s6, s7;
      f2_unpack(acc2[0], s0, s1);
      f2_unpack(acc2[1], s2, s3);
      f2_unpack(acc2[2], s4, s5);
      f2_unpack(acc2[3], s6, s7);
      acc = ((s0 + s1) + (s2 + s3)) + ((s4 + s5) + (s6 + s7));
    }
    // the key's column sum = the groups' sums added in group order (fixed)
    float* const acc_sm = lse_sm;               // [NG - 1][128]: the staging area is free after the last tile
    asm volatile("bar.sync %0, %1;" ::"r"(NG + 1), "r"(128 * NG) : "memory");
    if (grp > 0) acc_sm[(grp - 1) * 128 + key_l] = acc;
    asm volatile("bar.sync %0, %1;" ::"r"(NG + 1), "r"(128 * NG) : "memory");
    if (alive && !*abort_flag) {
      const int j = key0 + key_l - sq.video_start;           // video token index of this key
      if (grp == 0 && j >= 0 && j < sq.n_video) {
#pragma unroll
        for (int g = 1; g < NG; ++g) acc += acc_sm[(g - 1) * 128 + key_l];
        p.partial[(size_t)layer * p.sum_video + sq.score_off + j] = acc;
      }
    } else if (p.d_status && et == 0) {
      *p.d_status = SPECVLM_ERR_TIMEOUT;
    }
  }
  // every role ends here; the allocating warp returns the tensor memory
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Pass 1 on tcgen05.  CTA = (row tile, KV head, layer), two CTAs per SM.
//   S[row][key] = Q_tile (A: 128 rows x d, K-major) * K_tile^T (B: 128 keys x d, K-major)
// as a chain of tcgen05.mma (M = N = 128, K = 16 each) into one of two 128-column TMEM buffers.
// With the rows on the TMEM lanes an epilogue thread owns one row: it reads its 128 logits of a
// tile with tcgen05.ld and keeps the row's running (max, sum) in two registers -- the row
// reduction needs no cross-thread step.  The kernel is bound by the exponentials (one per logit),
// not by the tensor pipe; two epilogue groups per CTA (alternate tiles, one accumulator buffer
// each, their (max, sum) pairs merged at the end) and a second CTA on the SM keep the
// special-function units fed while other warps wait for their TMEM loads.
// Warps: 0 = TMA producer (Q tile once, K tiles through a ring), 1 = TMEM allocation + MMA issue,
// 2..5 and 6..9 = the epilogue groups (one TMEM lane quadrant per warp).
// ---------------------------------------------------------------------------------------------
template <int D, int STAGES>
__global__ void __launch_bounds__(320, 2)
scores_lse_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                     const __grid_constant__ ScoreParams p) {
  constexpr int TILE_BYTES = kKeyTile * D * 2;
  constexpr int KSTEPS = D / 16;
  constexpr uint32_t kTmemCols = 256;
  constexpr uint32_t kIdesc = umma_idesc_bf16(128, 128, false, false);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* const smem = smem_raw + (base - raw_addr);
  const uint32_t q_sm = base;                                    // the row tile
  const uint32_t k_sm = base + TILE_BYTES;                       // K ring
  constexpr int kTail = (1 + STAGES) * TILE_BYTES;
  const uint32_t bar_qfull = base + kTail;
  const uint32_t bar_kfull = bar_qfull + 8;                      // [STAGES]
  const uint32_t bar_kempty = bar_kfull + 8 * STAGES;            // [STAGES]
  const uint32_t bar_tfull = bar_kempty + 8 * STAGES;            // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                    // [2]
  uint8_t* const tail = smem + kTail + 16 * STAGES + 40;
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(tail);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(tail + 8);
  float2* const ml_sm = reinterpret_cast<float2*>(tail + 16);    // [128] group 1's (max, sum) per row

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = find_seq(p, blockIdx.x);
  const ScoreSeq sq = p.seq[b];
  const int qtile = blockIdx.x - sq.tile_off;
  const int g = blockIdx.y, layer = blockIdx.z;
  const int i_first = qtile * p.qt;
  const int n_i = min(p.qt, sq.n_text - i_first);               // queries in this tile
  const int rows_valid = n_i * p.group;
  const int key_end = sq.text_start + i_first + n_i;            // keys [0, key_end) are needed
  const int n_kt = (key_end + kKeyTile - 1) / kKeyTile;

  if (tid == 0) {
    mbar_init(bar_qfull, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_kfull + 8 * s, 1);
      mbar_init(bar_kempty + 8 * s, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_tfull + 8 * i, 1);
      mbar_init(bar_tempty + 8 * i, 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_q);
      const uint64_t pol = l2_policy_evict_last();               // K is re-read by the other row tiles
      mbar_arrive_expect_tx(bar_qfull, (D / 64) * p.qt * p.group * 128);
#pragma unroll
      for (int h = 0; h < D / 64; ++h)
        tma_load_5d(q_sm + h * (kKeyTile * 128), &tm_q, bar_qfull, h * 64, 0, g, sq.text_off + i_first, layer, pol);
      bool ok = true;
      int i = 0;
      for (; i < n_kt; ++i) {
        const int s = i % STAGES;
        if (i >= STAGES) ok = mbar_wait(bar_kempty + 8 * s, ((i / STAGES) - 1) & 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(bar_kfull + 8 * s, TILE_BYTES);
        load_key_tile<D>(&tm_k, p, b, g, layer, i * kKeyTile, k_sm + s * TILE_BYTES, bar_kfull + 8 * s, pol);
      }
      if (!ok) {
        if (p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
        const uint64_t t0 = global_timer_ns();
        for (int k = i > STAGES ? i - STAGES : 0; k < i; ++k)
          while (!mbar_try_wait(bar_kfull + 8 * (k % STAGES), (k / STAGES) & 1) &&
                 global_timer_ns() - t0 < kWaitLimitNs) {
          }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issue (one thread)
    if (lane == 0) {
      bool ok = mbar_wait(bar_qfull, 0, abort_flag);
      for (int i = 0; i < n_kt && ok; ++i) {
        const int s = i % STAGES, buf = i & 1;
        ok = mbar_wait(bar_kfull + 8 * s, (i / STAGES) & 1, abort_flag);
        if (ok && i >= 2) ok = mbar_wait(bar_tempty + 8 * buf, ((i >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t da = umma_desc_sw128(q_sm, 16, 1024), db = umma_desc_sw128(k_sm + s * TILE_BYTES, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          // 16 channels per step: 32 bytes along the swizzled 128-byte row; channels 64.. live in
          // the second half-tile
          const uint32_t off = (ks >> 2) * (kKeyTile * 128) + (ks & 3) * 32;
          umma_bf16_ss(tmem_base + buf * 128, umma_desc_advance(da, off), umma_desc_advance(db, off), kIdesc,
                       ks > 0 ? 1u : 0u);
        }
        umma_commit(bar_kempty + 8 * s);
        umma_commit(bar_tfull + 8 * buf);
      }
      if (!ok && p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
    }
  } else {
    // ---------------------------------------------------------------- epilogue: 2 groups x 4 warps, 128 rows
    const int grp = (warp - 2) >> 2;            // tiles with (index & 1) == grp, accumulator buffer grp
    const int quad = warp & 3;                  // TMEM lanes [32 * quad, 32 * quad + 32)
    const int r = quad * 32 + lane;             // this thread's row
    const int il = r / p.group, hg = r - il * p.group;
    const int lim = r < rows_valid ? sq.text_start + i_first + il + 1 : 0;   // keys [0, lim) are visible
    const int first_lim = sq.text_start + i_first + 1;
    float m = -INFINITY, l = 0.f;
    bool alive = true;
    // One tile; MASKED (a type, so that each loop below gets its own copy of the code) says whether
    // the tile reaches past the first row's limit.  The copy for the tiles before it -- all but the
    // last one or two -- has no mask logic and no branch in it: a single warp-uniform branch inside
    // this loop was measured to double the kernel's time.
    auto tile = [&](int i, auto masked_c) -> bool {
      constexpr bool need_mask = decltype(masked_c)::value;
      const int buf = grp;
      if (alive && !mbar_wait(bar_tfull + 8 * buf, (i >> 1) & 1, abort_flag)) alive = false;
      alive = __all_sync(0xffffffffu, alive);   // warp-uniform: the TMEM loads below are warp-collective
      if (!alive) return false;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * 128;
      const int key0 = i * kKeyTile;
      uint32_t va[32], vb[32];                    // the load of chunk c + 1 flies while chunk c is summed
      tmem_ld_x32(taddr, va);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t(&v)[32] = (c & 1) ? vb : va;
        tmem_ld_wait();
        if (c < 3) {
          tmem_ld_x32(taddr + (c + 1) * 32, (c & 1) ? va : vb);
        } else {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);   // buffer free for the MMAs of tile i + 2
        }
        if constexpr (need_mask) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (key0 + c * 32 + j >= lim) v[j] = 0xff800000u;   // -inf: hidden by the causal rule
        }
        // the scale is positive, so the maximum of the raw products gives the maximum logit
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 32; j += 2) mx[(j >> 1) & 3] = fmaxf(mx[(j >> 1) & 3], fmaxf(__uint_as_float(v[j]), __uint_as_float(v[j + 1])));
        const float mn = fmaxf(m, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.scale_log2);
        const float mu = mn == -INFINITY ? 0.f : mn;
        const uint64_t sc2 = f2_pack(p.scale_log2, p.scale_log2), nmu2 = f2_pack(-mu, -mu);
        uint64_t ps[2] = {0ull, 0ull};            // two chains of pairs
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          const uint64_t t2 = f2_fma(f2_pack(__uint_as_float(v[2 * q]), __uint_as_float(v[2 * q + 1])), sc2, nmu2);
          // the pairs of kPolyMaskLse take the polynomial, spread so that both kinds interleave
          const bool poly = (kPolyMaskLse >> q) & 1;
          ps[q & 1] = f2_add(ps[q & 1], poly ? f2_exp2_poly(t2) : f2_exp2_sfu(t2));
        }
        float s0, s1, s2, s3;
        f2_unpack(ps[0], s0, s1);
        f2_unpack(ps[1], s2, s3);
        l = l * fast_exp2(m - mu) + ((s0 + s1) + (s2 + s3));
        m = mn;
      }
      return true;
    };
    {
      int i = grp;
      for (; i < n_kt && (i + 1) * kKeyTile <= first_lim; i += 2)
        if (!tile(i, std::false_type{})) break;
      for (; alive && i < n_kt; i += 2)
        if (!tile(i, std::true_type{})) break;
    }
    // merge the two groups' running pairs (every wait above is bounded, so both get here)
    if (grp == 1) ml_sm[r] = make_float2(m, l);
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (alive && !*abort_flag) {
      if (grp == 0 && r < rows_valid) {
        const float2 o = ml_sm[r];
        const float mm = fmaxf(m, o.x);
        const float ll = (l > 0.f ? l * fast_exp2(m - mm) : 0.f) + (o.y > 0.f ? o.y * fast_exp2(o.x - mm) : 0.f);
        p.lse[((size_t)layer * p.sum_text + sq.text_off + i_first + il) * p.n_q_heads + g * p.group + hg] =
            (mm + log2f(ll)) * kLn2;
      }
    } else if (p.d_status && r == 0) {
      *p.d_status = SPECVLM_ERR_TIMEOUT;
    }
  }
  // every role ends here; the allocating warp returns the tensor memory
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// scores[j] = (sum over layers, in order, of partial[l][j]) / (L * Hq * n_text of j's sequence)
__global__ void scores_finish_kernel(const __grid_constant__ ScoreParams p, float* __restrict__ scores) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= p.sum_video) return;
  int b = 0;
  while (b + 1 < p.batch && p.seq[b + 1].score_off <= j) ++b;
  float acc = 0.f;
  for (int l = 0; l < p.n_layers; ++l) acc += p.partial[(size_t)l * p.sum_video + j];
  scores[j] = acc / ((float)p.n_layers * (float)p.n_q_heads * (float)p.seq[b].n_text);
}

static void ws_layout(int n_layers, int n_q_heads, int64_t sum_text, int64_t sum_video, size_t& lse_bytes,
                      size_t& partial_bytes) {
  lse_bytes = round_up((size_t)n_layers * sum_text * n_q_heads * sizeof(float), 256);
  partial_bytes = round_up((size_t)n_layers * sum_video * sizeof(float), 256);
}

struct ScoreSetup {
  int layer_begin = 0, layer_count = 0;   // the layers this call rates
  bool finish = true;                      // reduce the per-layer partial sums into the scores
  specvlm_kv_t kv;
  ScoreParams p1, p2;          // pass-1 (row tiles) and pass-2 (key blocks) CTA tables
  CUtensorMap tk, tq;
  int n_row_tiles, n_key_blocks;
};

// Validates the arguments common to both entry points and fills the launch tables.
static int32_t setup_scores(const specvlm_kv_t* target_kv, const void* q_text, const int32_t* text_cu,
                            const int32_t* text_start, const int32_t* video_start, const int32_t* video_len,
                            const int32_t* video_cu, int32_t batch, int32_t n_q_heads, float sm_scale,
                            int32_t* d_status, ScoreSetup& su, int32_t layer_begin = 0, int32_t layer_end = -1) {
  if (!target_kv) return SPECVLM_ERR_INVALID_ARG;
  su.kv = *target_kv;
  specvlm_kv_t& kv = su.kv;
  if (layer_end < 0) layer_end = kv.n_layers;
  if (layer_begin < 0 || layer_end > kv.n_layers || layer_begin > layer_end) return SPECVLM_ERR_INVALID_ARG;
  static const int32_t dummy = 0;
  if (!kv.seq_lens) kv.seq_lens = &dummy;             // lengths come from text_start / text_cu here
  int32_t rc = validate_kv(&kv, batch, false);
  if (rc != SPECVLM_OK) return rc;
  if (!q_text || !text_cu || !text_start || n_q_heads < 1 || !(sm_scale > 0.f) || !aligned16(q_text))
    return SPECVLM_ERR_INVALID_ARG;
  if (batch > kScoresMaxBatch) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if (n_q_heads % kv.n_kv_heads != 0) return SPECVLM_ERR_INVALID_ARG;
  const int group = n_q_heads / kv.n_kv_heads;
  if (group > 16) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if (kv.n_layers > 65535 || kv.n_kv_heads > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;

  ScoreParams& p = su.p1;
  p.qt = 128 / group;
  int64_t sum_video = 0;
  for (int b = 0; b < batch; ++b) {
    const int nt = text_cu[b + 1] - text_cu[b];
    if (nt < 1 || text_start[b] < 0 || text_start[b] + nt > kv.max_seq_len) return SPECVLM_ERR_INVALID_ARG;
    if (video_len) {
      if (!video_start || !video_cu || video_len[b] < 1 || video_start[b] < 0 ||
          video_start[b] + video_len[b] > text_start[b] || video_cu[b] != sum_video)
        return SPECVLM_ERR_INVALID_ARG;
      sum_video += video_len[b];
    }
  }
  if (video_len && video_cu[batch] != sum_video) return SPECVLM_ERR_INVALID_ARG;
  if (sum_video > 0x7fffffff) return SPECVLM_ERR_UNSUPPORTED_SHAPE;

  p.q = static_cast<const __nv_bfloat16*>(q_text);
  p.lse = nullptr;
  p.partial = nullptr;
  p.block_table = kv.block_table;
  p.d_status = d_status;
  p.batch = batch;
  p.n_layers = kv.n_layers;
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = kv.n_kv_heads;
  p.group = group;
  p.sum_text = text_cu[batch];
  p.sum_video = (int32_t)sum_video;
  p.max_blocks = kv.max_blocks;
  p.block_tokens = kv.block_tokens;
  p.scale_log2 = sm_scale * kLog2e;
  su.p2 = p;
  su.layer_begin = layer_begin;
  su.layer_count = layer_end - layer_begin;
  su.finish = true;
  su.n_row_tiles = su.n_key_blocks = 0;
  for (int b = 0; b < batch; ++b) {
    const int nt = text_cu[b + 1] - text_cu[b];
    ScoreSeq s;
    s.text_off = text_cu[b];
    s.n_text = nt;
    s.text_start = text_start[b];
    s.video_start = video_len ? video_start[b] : 0;
    s.n_video = video_len ? video_len[b] : 0;
    s.score_off = video_len ? video_cu[b] : 0;
    s.tile_off = su.n_row_tiles;
    su.p1.seq[b] = s;
    s.tile_off = su.n_key_blocks;
    su.p2.seq[b] = s;
    su.n_row_tiles += (nt + p.qt - 1) / p.qt;
    su.n_key_blocks += (s.video_start % 64 + s.n_video + kKeyTile - 1) / kKeyTile;
  }

  // The kernels count layers from 0 (one code for a range and for the whole problem): the K map, the
  // Q map and the query pointer start at the range's first layer; the callers offset the row
  // statistics and the partial sums the same way.
  specvlm_kv_t kv_range = kv;
  kv_range.n_layers = su.layer_count > 0 ? su.layer_count : 1;
  void* const k_range = static_cast<uint8_t*>(kv.k) + (size_t)layer_begin * kv.stride_layer * 2;
  rc = encode_kv_map(&su.tk, &kv_range, k_range, 64);
  if (rc != SPECVLM_OK) return rc;
  encode_tiled_fn enc = get_encode_tiled();
  if (!enc) return SPECVLM_ERR_CUDA;
  const int D = kv.head_dim;
  const cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)group, (cuuint64_t)kv.n_kv_heads,
                              (cuuint64_t)p.sum_text, (cuuint64_t)kv_range.n_layers};
  const cuuint64_t strides[4] = {(cuuint64_t)D * 2, (cuuint64_t)group * D * 2, (cuuint64_t)n_q_heads * D * 2,
                                 (cuuint64_t)p.sum_text * n_q_heads * D * 2};
  const cuuint32_t box[5] = {64u, (cuuint32_t)group, 1u, (cuuint32_t)p.qt, 1u};
  const cuuint32_t estr[5] = {1u, 1u, 1u, 1u, 1u};
  const __nv_bfloat16* const q_range =
      static_cast<const __nv_bfloat16*>(q_text) + (size_t)layer_begin * p.sum_text * n_q_heads * D;
  su.p1.q = su.p2.q = q_range;
  if (enc(&su.tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<__nv_bfloat16*>(q_range), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SPECVLM_ERR_CUDA;
  return SPECVLM_OK;
}

template <int D>
static int32_t launch_lse(ScoreSetup& su, cudaStream_t st) {
  const dim3 grid((unsigned)su.n_row_tiles, (unsigned)su.kv.n_kv_heads, (unsigned)su.layer_count);
  constexpr int STAGES = 2;                              // two CTAs per SM: 3 x 32 KB each at d = 128
  constexpr int SMEM = (1 + STAGES) * kKeyTile * D * 2 + 1024 + 16 * STAGES + 40 + 16 + 128 * 8;
  auto k = scores_lse_tc_kernel<D, STAGES>;
  static std::atomic<uint64_t> attr_done{0};
  if (!smem_attr_once(attr_done, reinterpret_cast<const void*>(k), SMEM)) return SPECVLM_ERR_CUDA;
  k<<<grid, 320, SMEM, st>>>(su.tk, su.tq, su.p1);
  return launch_status();
}

template <int D>
static int32_t launch_colsum(ScoreSetup& su, cudaStream_t st) {
  constexpr int STAGES = 4;
  constexpr int SMEM = (2 + STAGES) * kKeyTile * D * 2 + 1024 + 16 * STAGES + 32 + 16 * kColsumGroups + 16 +
                       kColsumGroups * 2 * 128 * 4;
  auto k = scores_colsum_tc_kernel<D, STAGES>;
  static std::atomic<uint64_t> attr_done{0};
  if (!smem_attr_once(attr_done, reinterpret_cast<const void*>(k), SMEM)) return SPECVLM_ERR_CUDA;
  k<<<dim3((unsigned)su.n_key_blocks, (unsigned)su.layer_count), kColsumThreads, SMEM, st>>>(su.tk, su.tq, su.p2);
  return launch_status();
}

}  // namespace specvlm

using namespace specvlm;

extern "C" size_t specvlm_stage1_scores_workspace_bytes(const specvlm_kv_t* target_kv,
                                                        const int32_t* text_cu, const int32_t* video_len,
                                                        int32_t batch, int32_t n_q_heads) {
  if (!target_kv || !text_cu || !video_len || batch < 1 || n_q_heads < 1) return 0;
  int64_t sum_video = 0;
  for (int b = 0; b < batch; ++b) sum_video += video_len[b];
  size_t a, c;
  ws_layout(target_kv->n_layers, n_q_heads, text_cu[batch], sum_video, a, c);
  return a + c;
}

extern "C" size_t specvlm_stage1_scores_layer_sums_offset(const specvlm_kv_t* target_kv, const int32_t* text_cu,
                                                          int32_t batch, int32_t n_q_heads) {
  if (!target_kv || !text_cu || batch < 1 || n_q_heads < 1) return 0;
  size_t a, c;
  ws_layout(target_kv->n_layers, n_q_heads, text_cu[batch], 0, a, c);
  return a;
}

extern "C" int32_t specvlm_stage1_row_lse(const specvlm_kv_t* target_kv, const void* q_text,
                                          const int32_t* text_cu, const int32_t* text_start, int32_t batch,
                                          int32_t n_q_heads, float sm_scale, float* row_lse,
                                          int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!row_lse) return SPECVLM_ERR_INVALID_ARG;
  ScoreSetup su;
  int32_t rc = setup_scores(target_kv, q_text, text_cu, text_start, nullptr, nullptr, nullptr, batch,
                            n_q_heads, sm_scale, d_status, su);
  if (rc != SPECVLM_OK) return rc;
  su.p1.lse = row_lse;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return su.kv.head_dim == 128 ? launch_lse<128>(su, st) : launch_lse<64>(su, st);
}

static int32_t stage1_scores_range(const specvlm_kv_t* target_kv, const void* q_text, const int32_t* text_cu,
                                   const int32_t* text_start, const int32_t* video_start,
                                   const int32_t* video_len, const int32_t* video_cu, int32_t batch,
                                   int32_t n_q_heads, float sm_scale, const float* row_lse_or_null, float* scores,
                                   void* ws, size_t ws_bytes, int32_t layer_begin, int32_t layer_end, bool finish,
                                   int32_t* d_status, void* stream) {
  if (!video_start || !video_len || !video_cu || !scores || !ws) return SPECVLM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return SPECVLM_ERR_INVALID_ARG;
  ScoreSetup su;
  int32_t rc = setup_scores(target_kv, q_text, text_cu, text_start, video_start, video_len, video_cu, batch,
                            n_q_heads, sm_scale, d_status, su, layer_begin, layer_end);
  if (rc != SPECVLM_OK) return rc;
  size_t lse_bytes, partial_bytes;
  ws_layout(su.kv.n_layers, n_q_heads, su.p1.sum_text, su.p1.sum_video, lse_bytes, partial_bytes);
  if (ws_bytes < lse_bytes + partial_bytes) return SPECVLM_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool d128 = su.kv.head_dim == 128;
  su.finish = false;                       // the reduction below runs over all layers, not the range
  float* const partial_all = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + lse_bytes);
  if (su.layer_count > 0) {
    // the range's slices of the row statistics and of the per-layer partial sums
    const size_t lse_off = (size_t)layer_begin * su.p1.sum_text * n_q_heads;
    if (row_lse_or_null) {
      su.p2.lse = const_cast<float*>(row_lse_or_null) + lse_off;
    } else {
      su.p1.lse = su.p2.lse = static_cast<float*>(ws) + lse_off;
      rc = d128 ? launch_lse<128>(su, st) : launch_lse<64>(su, st);
      if (rc != SPECVLM_OK) return rc;
    }
    su.p2.partial = partial_all + (size_t)layer_begin * su.p1.sum_video;
    rc = d128 ? launch_colsum<128>(su, st) : launch_colsum<64>(su, st);
    if (rc != SPECVLM_OK) return rc;
  }
  if (!finish) return SPECVLM_OK;
  ScoreParams pf = su.p2;                  // all layers' partial sums, in layer order
  pf.partial = partial_all;
  pf.n_layers = su.kv.n_layers;
  scores_finish_kernel<<<(unsigned)((pf.sum_video + 255) / 256), 256, 0, st>>>(pf, scores);
  return launch_status();
}

extern "C" int32_t specvlm_stage1_scores(const specvlm_kv_t* target_kv, const void* q_text,
                                         const int32_t* text_cu, const int32_t* text_start,
                                         const int32_t* video_start, const int32_t* video_len,
                                         const int32_t* video_cu, int32_t batch, int32_t n_q_heads,
                                         float sm_scale, const float* row_lse_or_null, float* scores,
                                         void* ws, size_t ws_bytes, int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!target_kv) return SPECVLM_ERR_INVALID_ARG;
  return stage1_scores_range(target_kv, q_text, text_cu, text_start, video_start, video_len, video_cu, batch,
                             n_q_heads, sm_scale, row_lse_or_null, scores, ws, ws_bytes, 0, target_kv->n_layers, true,
                             d_status, stream);
}

extern "C" int32_t specvlm_stage1_scores_layers(const specvlm_kv_t* target_kv, const void* q_text,
                                                const int32_t* text_cu, const int32_t* text_start,
                                                const int32_t* video_start, const int32_t* video_len,
                                                const int32_t* video_cu, int32_t batch, int32_t n_q_heads,
                                                float sm_scale, const float* row_lse_or_null, float* scores,
                                                void* ws, size_t ws_bytes, int32_t layer_begin, int32_t layer_end,
                                                int32_t finish, int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  return stage1_scores_range(target_kv, q_text, text_cu, text_start, video_start, video_len, video_cu, batch,
                             n_q_heads, sm_scale, row_lse_or_null, scores, ws, ws_bytes, layer_begin, layer_end,
                             finish != 0, d_status, stream);
}
