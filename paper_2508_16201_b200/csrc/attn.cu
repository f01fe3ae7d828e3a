// Streaming softmax attention over a bf16 K/V cache for sm_100a: draft decode attention and
// (gamma+1)-query verification attention.
//
// Data movement: one producer warp moves 64-token K and V tiles HBM -> shared memory with
// 128-byte-swizzled tensor-map bulk copies (cp.async.bulk.tensor) through a multi-stage
// mbarrier ring; the cache is read exactly once.  Arithmetic: the GQA group's query heads times
// the query tokens form the M rows of bf16 m16n8k16 tensor-core tiles (QK^T and PV), softmax in
// fp32 with base-2 exponentials.  Long sequences are split across CTAs; a second kernel merges
// the split partials by their log-sum-exp.
#include "attn.cuh"
#include "attn_sched.h"
#include "host_util.h"

namespace specvlm {

// Issues the bulk tensor copies of tile `tg` (64 tokens of K and of V) of sequence b into one
// pipeline stage; completion is counted on `full`.
template <int D>
__device__ __forceinline__ void issue_kv_tile(const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                                              const AttnParams& p, int b, int g, int layer, int tg,
                                              uint32_t dst, uint32_t full, uint64_t policy) {
  constexpr int TILE_BYTES = kTileTokens * D * 2;
  int blk, tok;
  if (p.block_table) {
    const int tiles_per_block = p.block_tokens / kTileTokens;
    blk = p.block_table[(size_t)b * p.max_blocks + tg / tiles_per_block];
    tok = (tg % tiles_per_block) * kTileTokens;
  } else {
    blk = b;
    tok = tg * kTileTokens;
  }
  mbar_arrive_expect_tx(full, 2 * TILE_BYTES);
#pragma unroll
  for (int h = 0; h < D / 64; ++h) {
    tma_load_5d(dst + h * (kTileTokens * 128), tm_k, full, h * 64, tok, g, blk, layer, policy);
    tma_load_5d(dst + TILE_BYTES + h * (kTileTokens * 128), tm_v, full, h * 64, tok, g, blk, layer, policy);
  }
}

// ---------------------------------------------------------------------------------------------
// Kernel A: up to 16 query rows per KV head (decode: the group's heads; small verify windows).
// 4 consumer warps each own 16 of a tile's 64 tokens and keep private running (max, sum, O);
// they are merged once at the end.  Warp 4 is the TMA producer.
// ---------------------------------------------------------------------------------------------
template <int D, int STAGES>
__global__ void __launch_bounds__(160)
attn_rows16_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const AttnParams p) {
  constexpr int TILE_BYTES = kTileTokens * D * 2;
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  constexpr int KSTEPS = D / 16;
  constexpr int NT_O = D / 8;
  constexpr int OPITCH = D + 8;            // fp32 pitch of the end-of-kernel merge buffer

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* const smem = smem_raw + (base - raw_addr);
  const uint32_t bar_full = base + STAGES * STAGE_BYTES;
  const uint32_t bar_empty = bar_full + 8 * STAGES;
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(smem + STAGES * STAGE_BYTES + 16 * STAGES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, g = blockIdx.y, lb = blockIdx.z;
  const int layer = lb / p.batch, b = lb - layer * p.batch;

  int kv_len = p.seq_lens[b];
  kv_len = kv_len < 0 ? 0 : (kv_len > p.max_seq_len ? p.max_seq_len : kv_len);
  int tile_begin, tile_end;
  split_range(kv_len, p.n_splits, split, tile_begin, tile_end);
  const int n_my = tile_end - tile_begin;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == 4) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && n_my > 0) {
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      const uint64_t policy = l2_policy_evict_first();
      const int tiles_per_block = p.block_tokens / kTileTokens;   // used only when paged
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < n_my && ok; ++i) {
        const int s = i % STAGES;
        if (i >= STAGES) ok = mbar_wait(bar_empty + 8 * s, ((i / STAGES) - 1) & 1, abort_flag);
        if (!ok) break;
        const int tg = tile_begin + i;
        int blk, tok;
        if (p.block_table) {
          blk = p.block_table[(size_t)b * p.max_blocks + tg / tiles_per_block];
          tok = (tg % tiles_per_block) * kTileTokens;
        } else {
          blk = b;
          tok = tg * kTileTokens;
        }
        const uint32_t full = bar_full + 8 * s;
        mbar_arrive_expect_tx(full, STAGE_BYTES);
        const uint32_t dst = base + s * STAGE_BYTES;
#pragma unroll
        for (int h = 0; h < D / 64; ++h) {
          tma_load_5d(dst + h * (kTileTokens * 128), &tm_k, full, h * 64, tok, g, blk, layer, policy);
          tma_load_5d(dst + TILE_BYTES + h * (kTileTokens * 128), &tm_v, full, h * 64, tok, g, blk,
                      layer, policy);
        }
        issued = i + 1;
      }
      if (!ok) {
        // a wait expired: report, then stay until this CTA's copies in flight have landed
        if (p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
        const int first = issued > STAGES ? issued - STAGES : 0;
        for (int i = first; i < issued; ++i) {
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(bar_full + 8 * (i % STAGES), (i / STAGES) & 1) &&
                 global_timer_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int row0 = lane >> 2, row1 = row0 + 8, col = (lane & 3) * 2;
  uint32_t qf[KSTEPS][4];
  int lim0 = 0, lim1 = 0;   // number of visible keys for the two rows this thread holds
  {
    const __nv_bfloat16* q0 = nullptr;
    const __nv_bfloat16* q1 = nullptr;
    if (row0 < p.rows) {
      const int t = row0 / p.group, h = g * p.group + (row0 - t * p.group);
      q0 = p.q + (((size_t)lb * p.n_q + t) * p.n_q_heads + h) * D;
      lim0 = kv_len - p.n_q + t + 1;
    }
    if (row1 < p.rows) {
      const int t = row1 / p.group, h = g * p.group + (row1 - t * p.group);
      q1 = p.q + (((size_t)lb * p.n_q + t) * p.n_q_heads + h) * D;
      lim1 = kv_len - p.n_q + t + 1;
    }
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      qf[ks][0] = q0 ? *reinterpret_cast<const uint32_t*>(q0 + ks * 16 + col) : 0u;
      qf[ks][1] = q1 ? *reinterpret_cast<const uint32_t*>(q1 + ks * 16 + col) : 0u;
      qf[ks][2] = q0 ? *reinterpret_cast<const uint32_t*>(q0 + ks * 16 + 8 + col) : 0u;
      qf[ks][3] = q1 ? *reinterpret_cast<const uint32_t*>(q1 + ks * 16 + 8 + col) : 0u;
    }
  }

  float o[NT_O][4];
#pragma unroll
  for (int nt = 0; nt < NT_O; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  // per-lane ldmatrix row/chunk selectors
  const int mi = lane >> 3, r8 = lane & 7;
  const int k_tok = warp * 16 + (mi >> 1) * 8 + r8, k_chunk = mi & 1;   // K: non-transposed
  const int v_tok = warp * 16 + (mi & 1) * 8 + r8, v_chunk = mi >> 1;   // V: transposed

  bool alive = true;
  for (int i = 0; i < n_my; ++i) {
    const int s = i % STAGES;
    if (!mbar_wait(bar_full + 8 * s, (i / STAGES) & 1, abort_flag)) {
      alive = false;
      break;
    }
    const uint32_t k_base = base + s * STAGE_BYTES;
    const uint32_t v_base = k_base + TILE_BYTES;
    const int tb = (tile_begin + i) * kTileTokens + warp * 16;   // first token of this warp's slice
    if (tb < kv_len) {
      if (tb + 16 > kv_len) {
        // rows past the end of the sequence hold whatever the page held: clear V there so that
        // a zero probability times a stale non-finite value cannot reach the accumulator
        uint8_t* vt = smem + s * STAGE_BYTES + TILE_BYTES;
        const int first = kv_len - (tile_begin + i) * kTileTokens;      // first invalid local row
        for (int t = first + (lane >> 3); t < warp * 16 + 16; t += 4) {
#pragma unroll
          for (int h = 0; h < D / 64; ++h)
            *reinterpret_cast<uint4*>(vt + h * (kTileTokens * 128) + t * 128 + (lane & 7) * 16) =
                make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
      }
      float sc[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(k_base + tile_offset<D>(k_tok, 2 * ks + k_chunk), b0, b1, b2, b3);
        mma_bf16_16816(sc[0], qf[ks], b0, b1);
        mma_bf16_16816(sc[1], qf[ks], b2, b3);
      }
      // scale, causal / length mask, running max
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int tok = tb + nt * 8 + col + (e & 1);
          const int lim = (e < 2) ? lim0 : lim1;
          const float v = tok < lim ? sc[nt][e] * p.scale_log2 : -INFINITY;
          sc[nt][e] = v;
          if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
      const float a0 = fast_exp2(m0 - mu0), a1 = fast_exp2(m1 - mu1);
      m0 = mn0;
      m1 = mn1;
      float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        sc[nt][0] = fast_exp2(sc[nt][0] - mu0);
        sc[nt][1] = fast_exp2(sc[nt][1] - mu0);
        sc[nt][2] = fast_exp2(sc[nt][2] - mu1);
        sc[nt][3] = fast_exp2(sc[nt][3] - mu1);
        ps0 += sc[nt][0] + sc[nt][1];
        ps1 += sc[nt][2] + sc[nt][3];
      }
      l0 = l0 * a0 + ps0;
      l1 = l1 * a1 + ps1;
      uint32_t pa[4];
      pa[0] = pack_bf16x2(sc[0][0], sc[0][1]);
      pa[1] = pack_bf16x2(sc[0][2], sc[0][3]);
      pa[2] = pack_bf16x2(sc[1][0], sc[1][1]);
      pa[3] = pack_bf16x2(sc[1][2], sc[1][3]);
#pragma unroll
      for (int nt = 0; nt < NT_O; ++nt) {
        o[nt][0] *= a0;
        o[nt][1] *= a0;
        o[nt][2] *= a1;
        o[nt][3] *= a1;
      }
#pragma unroll
      for (int j = 0; j < D / 16; ++j) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(v_base + tile_offset<D>(v_tok, 2 * j + v_chunk), b0, b1, b2, b3);
        mma_bf16_16816(o[2 * j], pa, b0, b1);
        mma_bf16_16816(o[2 * j + 1], pa, b2, b3);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty + 8 * s);
  }

  // ------------------------------------------------------------ merge the 4 warps' partials
  // (named barrier over the 128 consumer threads; the producer warp has no part in it)
  asm volatile("bar.sync 1, 128;" ::: "memory");
  if (!alive || *abort_flag) return;   // a wait expired somewhere in this CTA: leave outputs alone
  float* const o_sm = reinterpret_cast<float*>(smem);                  // [4][16][OPITCH]
  float* const m_sm = o_sm + 4 * 16 * OPITCH;                          // [4][16]
  float* const l_sm = m_sm + 64;                                       // [4][16]
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  {
    float* ow = o_sm + warp * 16 * OPITCH;
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt) {
      *reinterpret_cast<float2*>(ow + row0 * OPITCH + nt * 8 + col) = make_float2(o[nt][0], o[nt][1]);
      *reinterpret_cast<float2*>(ow + row1 * OPITCH + nt * 8 + col) = make_float2(o[nt][2], o[nt][3]);
    }
    if ((lane & 3) == 0) {
      m_sm[warp * 16 + row0] = m0;
      m_sm[warp * 16 + row1] = m1;
      l_sm[warp * 16 + row0] = l0;
      l_sm[warp * 16 + row1] = l1;
    }
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  const int item = lb * p.n_kv_heads + g;
  for (int idx = tid; idx < p.rows * D; idx += 128) {
    const int r = idx / D, c = idx - r * D;
    float M = fmaxf(fmaxf(m_sm[r], m_sm[16 + r]), fmaxf(m_sm[32 + r], m_sm[48 + r]));
    float num = 0.f, den = 0.f;
    if (M != -INFINITY) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float f = fast_exp2(m_sm[w * 16 + r] - M);
        den += l_sm[w * 16 + r] * f;
        num += o_sm[(w * 16 + r) * OPITCH + c] * f;
      }
    }
    const float val = den > 0.f ? num / den : 0.f;
    const float lse2 = den > 0.f ? M + log2f(den) : -INFINITY;
    if (p.n_splits == 1) {
      const int t = r / p.group, h = g * p.group + (r - t * p.group);
      const size_t orow = ((size_t)lb * p.n_q + t) * p.n_q_heads + h;
      p.out[orow * D + c] = __float2bfloat16_rn(val);
      if (p.lse && c == 0) p.lse[orow] = lse2 * kLn2;
    } else {
      const size_t prow = ((size_t)item * p.n_splits + split) * p.rows + r;
      p.ws_o[prow * D + c] = val;
      if (c == 0) p.ws_lse[prow] = lse2;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Kernel B: 17..96 query rows per KV head (verification windows).  NG groups of 4 warps; a group
// owns MT m-tiles of 16 rows.  Inside a group, QK^T is split by tokens (warp w scores tokens
// 16w..16w+15 of the tile for all the group's rows) and PV is split by channels (warp w
// accumulates channels [D/4 * w, D/4 * (w+1)) for all rows over the tile's 64 tokens); the bf16
// probabilities cross between the two through a swizzled shared-memory tile.  K and V are read
// from shared memory once per group.  The last warp is the TMA producer.
// ---------------------------------------------------------------------------------------------
template <int D, int MT, int NG, int STAGES, int MINB>
__global__ void __launch_bounds__(NG == 1 ? 128 : 32 * (4 * NG + 1), MINB)
attn_rowsN_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const AttnParams p) {
  constexpr int TILE_BYTES = kTileTokens * D * 2;
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  constexpr int KSTEPS = D / 16;
  constexpr int NT_W = D / 32;               // n-tiles of 8 channels per warp in PV
  constexpr int GROWS = MT * 16;             // rows per group
  constexpr int P_BYTES = GROWS * 128;       // one group's probability tile (64 tokens bf16 per row)

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* const smem = smem_raw + (base - raw_addr);
  const uint32_t p_sm0 = base + STAGES * STAGE_BYTES;                       // [NG][GROWS][128 B]
  uint8_t* const after_p = smem + STAGES * STAGE_BYTES + NG * P_BYTES;
  float* const red_all = reinterpret_cast<float*>(after_p);                 // [NG][4][GROWS]
  const uint32_t bar_full = base + STAGES * STAGE_BYTES + NG * P_BYTES + NG * 4 * GROWS * 4;
  const uint32_t bar_empty = bar_full + 8 * STAGES;
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(
      smem + STAGES * STAGE_BYTES + NG * P_BYTES + NG * 4 * GROWS * 4 + 16 * STAGES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, g = blockIdx.y, lb = blockIdx.z;
  const int layer = lb / p.batch, b = lb - layer * p.batch;

  int kv_len = p.seq_lens[b];
  kv_len = kv_len < 0 ? 0 : (kv_len > p.max_seq_len ? p.max_seq_len : kv_len);
  int tile_begin, tile_end;
  split_range(kv_len, p.n_splits, split, tile_begin, tile_end);
  const int n_my = tile_end - tile_begin;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 4 * NG);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  // NG == 1: no producer warp (4 warps per CTA keep the full register budget at 2 CTAs per SM);
  // thread 0 refills a stage right after the first group barrier of the next tile, by which
  // time every warp has finished reading it.  NG == 2: a dedicated producer warp and empty
  // barriers, because the two groups only synchronise within themselves.
  constexpr bool kInline = NG == 1;
  uint64_t policy = 0;
  if (kInline) {
    if (tid == 0 && n_my > 0) {
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      policy = l2_policy_evict_first();
      const int pre = n_my < STAGES ? n_my : STAGES;
      for (int i = 0; i < pre; ++i)
        issue_kv_tile<D>(&tm_k, &tm_v, p, b, g, layer, tile_begin + i, base + i * STAGE_BYTES,
                         bar_full + 8 * i, policy);
    }
  } else if (warp == 4 * NG) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && n_my > 0) {
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      policy = l2_policy_evict_first();
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < n_my && ok; ++i) {
        const int s = i % STAGES;
        if (i >= STAGES) ok = mbar_wait(bar_empty + 8 * s, ((i / STAGES) - 1) & 1, abort_flag);
        if (!ok) break;
        issue_kv_tile<D>(&tm_k, &tm_v, p, b, g, layer, tile_begin + i, base + s * STAGE_BYTES,
                         bar_full + 8 * s, policy);
        issued = i + 1;
      }
      if (!ok) {
        if (p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
        const int first = issued > STAGES ? issued - STAGES : 0;
        for (int i = first; i < issued; ++i) {
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(bar_full + 8 * (i % STAGES), (i / STAGES) & 1) &&
                 global_timer_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int gi = warp >> 2, cw = warp & 3;            // group, warp within group
  const int rb = gi * GROWS;                          // first row of this group
  const int col = (lane & 3) * 2;
  const uint32_t p_sm = p_sm0 + gi * P_BYTES;
  float* const red = red_all + gi * 4 * GROWS;        // [4 warps][GROWS]
  const int bar_id = 1 + gi;

  uint32_t qf[MT][KSTEPS][4];
  int lim[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int r = rb + mt * 16 + (lane >> 2) + hf * 8;
      const __nv_bfloat16* qp = nullptr;
      lim[mt][hf] = 0;
      if (r < p.rows) {
        const int t = r / p.group, h = g * p.group + (r - t * p.group);
        qp = p.q + (((size_t)lb * p.n_q + t) * p.n_q_heads + h) * D;
        lim[mt][hf] = kv_len - p.n_q + t + 1;
      }
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        qf[mt][ks][hf] = qp ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + col) : 0u;
        qf[mt][ks][2 + hf] = qp ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + col) : 0u;
      }
    }
  }
  float o[MT][NT_W][4];
  float m[MT][2], l[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    m[mt][0] = m[mt][1] = -INFINITY;
    l[mt][0] = l[mt][1] = 0.f;
#pragma unroll
    for (int nt = 0; nt < NT_W; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;
  }

  const int mi = lane >> 3, r8 = lane & 7;
  const int k_tok = cw * 16 + (mi >> 1) * 8 + r8, k_chunk = mi & 1;

  bool alive = true;
  for (int i = 0; i < n_my; ++i) {
    const int s = i % STAGES;
    // A warp whose wait expired keeps taking part in the group barriers below (its results are
    // discarded at the end), so the other warps of the group can never be left waiting for it.
    if (alive && !mbar_wait(bar_full + 8 * s, (i / STAGES) & 1, abort_flag)) alive = false;
    const uint32_t k_base = base + s * STAGE_BYTES;
    const uint32_t v_base = k_base + TILE_BYTES;
    const int tile_tok0 = (tile_begin + i) * kTileTokens;
    const int tb = tile_tok0 + cw * 16;
    if (alive && tile_tok0 + kTileTokens > kv_len) {
      // clear the V rows past the end of the sequence (see kernel A); this warp clears the rows of
      // its own 16-token slice, the group barrier below publishes them to the other warps
      uint8_t* vt = smem + s * STAGE_BYTES + TILE_BYTES;
      int first = kv_len - tile_tok0;
      if (first < cw * 16) first = cw * 16;
      for (int t = first + (lane >> 3); t < cw * 16 + 16; t += 4) {
#pragma unroll
        for (int h = 0; h < D / 64; ++h)
          *reinterpret_cast<uint4*>(vt + h * (kTileTokens * 128) + t * 128 + (lane & 7) * 16) =
              make_uint4(0, 0, 0, 0);
      }
    }
    float sc[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) sc[mt][nt][0] = sc[mt][nt][1] = sc[mt][nt][2] = sc[mt][nt][3] = 0.f;
    if (alive && tb < kv_len) {
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(k_base + tile_offset<D>(k_tok, 2 * ks + k_chunk), b0, b1, b2, b3);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_bf16_16816(sc[mt][0], qf[mt][ks], b0, b1);
          mma_bf16_16816(sc[mt][1], qf[mt][ks], b2, b3);
        }
      }
    }
    // scale + mask, this warp's row maxima over its 16 tokens
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int tok = tb + nt * 8 + col + e;
            const float v = tok < lim[mt][hf] ? sc[mt][nt][hf * 2 + e] * p.scale_log2 : -INFINITY;
            sc[mt][nt][hf * 2 + e] = v;
            mx = fmaxf(mx, v);
          }
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if ((lane & 3) == 0) red[cw * GROWS + mt * 16 + (lane >> 2) + hf * 8] = mx;
      }
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    if (kInline && tid == 0 && alive && i >= 1 && i - 1 + STAGES < n_my) {
      // every warp is past its last read of the previous tile's stage: refill it
      const int nxt = i - 1 + STAGES;
      issue_kv_tile<D>(&tm_k, &tm_v, p, b, g, layer, tile_begin + nxt, base + ((i - 1) % STAGES) * STAGE_BYTES,
                       bar_full + 8 * ((i - 1) % STAGES), policy);
    }
    // tile maxima, probabilities -> shared memory (bf16), rescale the accumulators
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int rl = mt * 16 + (lane >> 2) + hf * 8;
        const float mx = fmaxf(fmaxf(red[rl], red[GROWS + rl]), fmaxf(red[2 * GROWS + rl], red[3 * GROWS + rl]));
        const float mn = fmaxf(m[mt][hf], mx);
        const float mu = mn == -INFINITY ? 0.f : mn;
        const float alpha = fast_exp2(m[mt][hf] - mu);
        m[mt][hf] = mn;
        float ps = 0.f;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const float p0 = fast_exp2(sc[mt][nt][hf * 2] - mu);
          const float p1 = fast_exp2(sc[mt][nt][hf * 2 + 1] - mu);
          ps += p0 + p1;
          const int chunk = 2 * cw + nt;
          const uint32_t addr = p_sm + rl * 128 + ((chunk ^ (rl & 7)) << 4) + col * 2;
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(pack_bf16x2(p0, p1)) : "memory");
        }
        l[mt][hf] = l[mt][hf] * alpha + ps;
#pragma unroll
        for (int nt = 0; nt < NT_W; ++nt) {
          o[mt][nt][hf * 2] *= alpha;
          o[mt][nt][hf * 2 + 1] *= alpha;
        }
      }
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
    // PV over the tile's 64 tokens for this warp's channel slice
#pragma unroll
    for (int kt = 0; kt < 4; ++kt) {
      uint32_t vb[NT_W][2];
      const int v_tok = kt * 16 + (mi & 1) * 8 + r8;
#pragma unroll
      for (int j = 0; j < NT_W / 2; ++j)
        ldmatrix_x4_trans(v_base + tile_offset<D>(v_tok, cw * NT_W + 2 * j + (mi >> 1)), vb[2 * j][0],
                          vb[2 * j][1], vb[2 * j + 1][0], vb[2 * j + 1][1]);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        uint32_t a[4];
        const int pr = mt * 16 + (mi & 1) * 8 + r8;
        ldmatrix_x4(p_sm + pr * 128 + (((2 * kt + (mi >> 1)) ^ (pr & 7)) << 4), a[0], a[1], a[2], a[3]);
#pragma unroll
        for (int nt = 0; nt < NT_W; ++nt) mma_bf16_16816(o[mt][nt], a, vb[nt][0], vb[nt][1]);
      }
    }
    __syncwarp();
    if (!kInline && lane == 0 && alive) mbar_arrive(bar_empty + 8 * s);
  }

  // ------------------------------------------------------------ row sums across the group's warps
  asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      float v = l[mt][hf];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      if ((lane & 3) == 0) red[cw * GROWS + mt * 16 + (lane >> 2) + hf * 8] = v;
    }
  asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
  if (!alive || *abort_flag) {
    if (p.d_status && (tid & 127) == 0) *p.d_status = SPECVLM_ERR_TIMEOUT;
    if (kInline && tid == 0) {
      // stay until the copies this thread issued have landed (bounded)
      const uint64_t t0 = global_timer_ns();
      for (int i = n_my > STAGES ? n_my - STAGES : 0; i < n_my; ++i)
        while (!mbar_try_wait(bar_full + 8 * (i % STAGES), (i / STAGES) & 1) &&
               global_timer_ns() - t0 < kWaitLimitNs) {
        }
    }
    return;
  }
  const int item = lb * p.n_kv_heads + g;
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int rl = mt * 16 + (lane >> 2) + hf * 8;
      const int r = rb + rl;
      if (r >= p.rows) continue;
      const float lt = red[rl] + red[GROWS + rl] + red[2 * GROWS + rl] + red[3 * GROWS + rl];
      const float inv = lt > 0.f ? 1.f / lt : 0.f;
      const float lse2 = lt > 0.f ? m[mt][hf] + log2f(lt) : -INFINITY;
      if (p.n_splits == 1) {
        const int t = r / p.group, h = g * p.group + (r - t * p.group);
        const size_t orow = ((size_t)lb * p.n_q + t) * p.n_q_heads + h;
#pragma unroll
        for (int nt = 0; nt < NT_W; ++nt)
          *reinterpret_cast<uint32_t*>(p.out + orow * D + cw * (D / 4) + nt * 8 + col) =
              pack_bf16x2(o[mt][nt][hf * 2] * inv, o[mt][nt][hf * 2 + 1] * inv);
        if (p.lse && cw == 0 && (lane & 3) == 0) p.lse[orow] = lse2 * kLn2;
      } else {
        const size_t prow = ((size_t)item * p.n_splits + split) * p.rows + r;
#pragma unroll
        for (int nt = 0; nt < NT_W; ++nt)
          *reinterpret_cast<float2*>(p.ws_o + prow * D + cw * (D / 4) + nt * 8 + col) =
              make_float2(o[mt][nt][hf * 2] * inv, o[mt][nt][hf * 2 + 1] * inv);
        if (cw == 0 && (lane & 3) == 0) p.ws_lse[prow] = lse2;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Split merge: out = sum_s w_s o_s / sum_s w_s,  w_s = 2^(lse_s - max lse).  One CTA per
// (layer, sequence, KV head); the split order is fixed, so results are reproducible.
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128) attn_merge_kernel(const AttnParams p) {
  const int item = blockIdx.x;
  const int lb = item / p.n_kv_heads, g = item - lb * p.n_kv_heads;
  const float* lse_base = p.ws_lse + (size_t)item * p.n_splits * p.rows;
  const float* o_base = p.ws_o + (size_t)item * p.n_splits * p.rows * D;
  for (int idx = threadIdx.x; idx < p.rows * (D / 4); idx += 128) {
    const int r = idx / (D / 4), c4 = idx - r * (D / 4);
    float M = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) M = fmaxf(M, lse_base[s * p.rows + r]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (M != -INFINITY) {
      for (int s = 0; s < p.n_splits; ++s) {
        const float w = fast_exp2(lse_base[s * p.rows + r] - M);
        const float4 v = *reinterpret_cast<const float4*>(o_base + ((size_t)s * p.rows + r) * D + c4 * 4);
        acc.x += w * v.x;
        acc.y += w * v.y;
        acc.z += w * v.z;
        acc.w += w * v.w;
        den += w;
      }
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const int t = r / p.group, h = g * p.group + (r - t * p.group);
    const size_t orow = ((size_t)lb * p.n_q + t) * p.n_q_heads + h;
    uint2 packed;
    packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(p.out + orow * D + c4 * 4) = packed;
    if (p.lse && c4 == 0) p.lse[orow] = den > 0.f ? (M + log2f(den)) * kLn2 : -INFINITY;
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
static int env_int(const char* name, int dflt) {
  const char* s = getenv(name);
  return s && *s ? atoi(s) : dflt;
}

// How many CTAs share one (layer, sequence, KV head).  All CTAs of a launch stream the same number
// of tiles, so the launch takes ceil(CTAs / resident slots) rounds of (tiles per CTA + a fixed
// start-up/epilogue cost of about two tiles); pick the split count that minimises that product.
static int choose_splits(int max_seq_len, int64_t items, int rows) {
  const int n_tiles = (max_seq_len + kTileTokens - 1) / kTileTokens;
  const int forced = env_int("SPECVLM_ATTN_SPLITS", 0);
  int best = 1;
  if (forced > 0) {
    best = forced;
  } else {
    const int64_t slots = (int64_t)sm_count() * (rows > 48 ? 1 : 2);
    double best_cost = 1e300;
    for (int s = 1; s <= 64 && s <= n_tiles; ++s) {
      const int per = (n_tiles + s - 1) / s;
      if ((s - 1) * per >= n_tiles) continue;            // would leave an empty split
      const double rounds = (double)((items * s + slots - 1) / slots);
      const double cost = rounds * (per + 2.0) + (s > 1 ? 0.5 : 0.0);
      if (cost < best_cost - 1e-9) {
        best_cost = cost;
        best = s;
      }
    }
  }
  if (best > 64) best = 64;
  if (best > n_tiles) best = n_tiles;
  if (best < 1) best = 1;
  return best;
}

static size_t attn_ws_bytes(const specvlm_kv_t* kv, int32_t batch, int rows) {
  const int64_t items = (int64_t)kv->n_layers * batch * kv->n_kv_heads;
  const int splits = choose_splits(kv->max_seq_len, items, rows);
  if (splits == 1) return 256;
  const size_t o = round_up((size_t)items * splits * rows * kv->head_dim * sizeof(float), 256);
  const size_t l = round_up((size_t)items * splits * rows * sizeof(float), 256);
  return o + l;
}

template <int D>
static int32_t launch_rows16(const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                             dim3 grid, cudaStream_t st) {
  constexpr int STAGES = 3;
  constexpr int SMEM = STAGES * 2 * kTileTokens * D * 2 + 1024 + 16 * STAGES + 16;
  auto kern = attn_rows16_kernel<D, STAGES>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
    return SPECVLM_ERR_CUDA;
  kern<<<grid, 160, SMEM, st>>>(tk, tv, p);
  return launch_status();
}

template <int D, int MT, int NG>
static int32_t launch_rowsN(const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p, dim3 grid,
                            cudaStream_t st) {
  constexpr int STAGES = NG == 1 ? 3 : 5;
  constexpr int MINB = NG == 1 ? 2 : 1;
  constexpr int SMEM = STAGES * 2 * kTileTokens * D * 2 + NG * MT * 16 * 128 + NG * 4 * MT * 16 * 4 +
                       16 * STAGES + 16 + 1024;
  auto kern = attn_rowsN_kernel<D, MT, NG, STAGES, MINB>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
    return SPECVLM_ERR_CUDA;
  kern<<<grid, NG == 1 ? 128 : 32 * (4 * NG + 1), SMEM, st>>>(tk, tv, p);
  return launch_status();
}

template <int D>
static int32_t launch_any(const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p, dim3 grid,
                          cudaStream_t st) {
  if (p.rows <= 16) return launch_rows16<D>(tk, tv, p, grid, st);
  if (p.rows <= 32) return launch_rowsN<D, 2, 1>(tk, tv, p, grid, st);
  if (p.rows <= 48) return launch_rowsN<D, 3, 1>(tk, tv, p, grid, st);
  if (p.rows <= 64) return launch_rowsN<D, 2, 2>(tk, tv, p, grid, st);
  return launch_rowsN<D, 3, 2>(tk, tv, p, grid, st);
}

// tcgen05 path (attn_tc.cu)
size_t attn_tc_ws_bytes(const specvlm_kv_t* kv, int32_t batch, int rows);
int32_t attn_tc_launch(const specvlm_kv_t* kv, const void* q, int32_t batch, int32_t n_q_heads, int32_t n_q,
                       float sm_scale, void* out, float* lse, void* ws, size_t ws_bytes, int32_t* d_status,
                       cudaStream_t st);

static bool use_legacy_mma() {
  const char* s = getenv("SPECVLM_ATTN_IMPL");
  return s && s[0] == 'm';             // "mma": the mma.sync kernels
}

static int32_t attn_common(const specvlm_kv_t* kv, const void* q, int32_t batch, int32_t n_q_heads,
                           int32_t n_q, float sm_scale, void* out, float* lse, void* ws,
                           size_t ws_bytes, int32_t* d_status, void* stream) {
  int32_t rc = validate_kv(kv, batch, true);
  if (rc != SPECVLM_OK) return rc;
  if (!q || !out || n_q_heads < 1 || n_q < 1 || !(sm_scale > 0.f)) return SPECVLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return SPECVLM_ERR_INVALID_ARG;
  if (n_q_heads % kv->n_kv_heads != 0) return SPECVLM_ERR_INVALID_ARG;
  const int group = n_q_heads / kv->n_kv_heads;
  if (group > 16 || n_q > 9) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  const int rows = group * n_q;
  if (!use_legacy_mma())
    return attn_tc_launch(kv, q, batch, n_q_heads, n_q, sm_scale, out, lse, ws, ws_bytes, d_status,
                          static_cast<cudaStream_t>(stream));
  if (rows > 96) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  const int64_t lb64 = (int64_t)kv->n_layers * batch;
  if (lb64 > 65535 * 64 || kv->n_kv_heads > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;

  const int64_t items = lb64 * kv->n_kv_heads;
  const int splits = choose_splits(kv->max_seq_len, items, rows);
  const size_t need = attn_ws_bytes(kv, batch, rows);
  if (splits > 1) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return SPECVLM_ERR_INVALID_ARG;
    if (ws_bytes < need) return SPECVLM_ERR_WORKSPACE_TOO_SMALL;
  }

  CUtensorMap tk, tv;
  rc = encode_kv_map(&tk, kv, kv->k, kTileTokens);
  if (rc != SPECVLM_OK) return rc;
  rc = encode_kv_map(&tv, kv, kv->v, kTileTokens);
  if (rc != SPECVLM_OK) return rc;

  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  p.ws_o = nullptr;
  p.ws_lse = nullptr;
  if (splits > 1) {
    p.ws_o = static_cast<float*>(ws);
    p.ws_lse = reinterpret_cast<float*>(
        static_cast<uint8_t*>(ws) +
        round_up((size_t)items * splits * rows * kv->head_dim * sizeof(float), 256));
  }
  p.block_table = kv->block_table;
  p.seq_lens = kv->seq_lens;
  p.d_status = d_status;
  p.batch = batch;
  p.n_q = n_q;
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = kv->n_kv_heads;
  p.group = group;
  p.rows = rows;
  p.n_splits = splits;
  p.max_blocks = kv->max_blocks;
  p.block_tokens = kv->block_tokens;
  p.max_seq_len = kv->max_seq_len;
  p.scale_log2 = sm_scale * kLog2e;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (lb64 > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  dim3 grid((unsigned)splits, (unsigned)kv->n_kv_heads, (unsigned)lb64);
  rc = kv->head_dim == 128 ? launch_any<128>(tk, tv, p, grid, st) : launch_any<64>(tk, tv, p, grid, st);
  if (rc != SPECVLM_OK) return rc;
  if (splits > 1) {
    if (kv->head_dim == 128)
      attn_merge_kernel<128><<<(unsigned)items, 128, 0, st>>>(p);
    else
      attn_merge_kernel<64><<<(unsigned)items, 128, 0, st>>>(p);
    rc = launch_status();
  }
  return rc;
}

}  // namespace specvlm

using namespace specvlm;

extern "C" size_t specvlm_attn_workspace_bytes(const specvlm_kv_t* kv, int32_t batch,
                                               int32_t n_q_heads, int32_t gamma) {
  if (!kv || batch < 1 || n_q_heads < 1 || gamma < 0 || kv->n_kv_heads < 1 ||
      n_q_heads % kv->n_kv_heads != 0 || kv->n_layers < 1 || kv->max_seq_len < 1)
    return 0;
  const int rows = (n_q_heads / kv->n_kv_heads) * (gamma + 1);
  if (!use_legacy_mma()) return rows <= 128 && batch <= kSchedMaxBatch ? attn_tc_ws_bytes(kv, batch, rows) : 0;
  return attn_ws_bytes(kv, batch, rows);
}

extern "C" int32_t specvlm_draft_decode_attn(const specvlm_kv_t* kv, const void* q, int32_t batch,
                                             int32_t n_q_heads, float sm_scale, void* out,
                                             float* lse_or_null, void* ws, size_t ws_bytes,
                                             int32_t* d_status, void* stream) {
  return attn_common(kv, q, batch, n_q_heads, 1, sm_scale, out, lse_or_null, ws, ws_bytes, d_status,
                     stream);
}

extern "C" int32_t specvlm_verify_attn(const specvlm_kv_t* kv, const void* q, int32_t batch,
                                       int32_t n_q_heads, int32_t gamma, float sm_scale, void* out,
                                       float* lse_or_null, void* ws, size_t ws_bytes,
                                       int32_t* d_status, void* stream) {
  if (gamma < 0 || gamma > 8) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  return attn_common(kv, q, batch, n_q_heads, gamma + 1, sm_scale, out, lse_or_null, ws, ws_bytes,
                     d_status, stream);
}
