// Attention entry points (draft decode and verification) and the kernel for up to 16 query rows
// per KV head, i.e. draft decode: the GQA group's heads of one query token.
//
// With so few rows the step is a pure K/V stream (3.5 flop per cache byte at group 7): 64-token K
// and V tiles go HBM -> shared memory by 128-byte-swizzled tensor-map bulk copies
// (cp.async.bulk.tensor) through an mbarrier ring, four warps each score 16 tokens of a tile on
// m16n8k16 bf16 tiles with a private online softmax, and are merged once at the end.  Long
// sequences are split across CTAs; the CTA that finishes an item last merges the split partials
// by their log-sum-exp, in split order.  Windows of more than 16 rows (verification) run on the
// tcgen05 kernel of attn_tc.cu.
#include "attn.cuh"
#include "attn_sched.h"
#include "host_util.h"

namespace specvlm {

// ---------------------------------------------------------------------------------------------
// Kernel A: up to 16 query rows per KV head (decode: the group's heads; small verify windows).
// 4 consumer warps each own 16 of a tile's 64 tokens and keep private running (max, sum, O);
// they are merged once at the end.  Warp 4 is the TMA producer.
// ---------------------------------------------------------------------------------------------
// NG consumer groups of 4 warps take alternate tiles (NG = 2 where an SM holds a single CTA, so
// that eight warps hide each other's latencies as two resident CTAs would).
template <int D, int STAGES, int NG>
__global__ void __launch_bounds__(32 * (4 * NG + 1))
attn_rows16_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const AttnParams p) {
  constexpr int TILE_BYTES = kTileTokens * D * 2;
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  constexpr int KSTEPS = D / 16;
  constexpr int NT_O = D / 8;
  constexpr int OPITCH = D + 8;            // fp32 pitch of the end-of-kernel merge buffer
  // A consumer group must see every phase of the ring slots it waits on: with the groups on
  // alternate tiles that holds only when a slot always belongs to the same group.  (A wait on a
  // phase two behind the barrier returns at once, the group then releases a slot it never read,
  // and the surplus arrival on the barrier is undefined behaviour: it faulted the kernel.)
  static_assert(STAGES % NG == 0, "ring depth must be a multiple of the number of consumer groups");

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

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  // Programmatic dependent launch: the kernel is launched so that it may start while the kernel
  // before it in the stream is still running.  Everything above touches no global memory; the
  // wait below returns once that kernel's memory operations are complete and visible.  The kernel
  // after this one may be scheduled as soon as every CTA here has got this far.
  if (tid == 32 * 4 * NG) {              // the producer's lane: descriptors are kernel parameters
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  __syncthreads();                       // the barriers are initialised
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // The first tile of an unsplit, contiguous cache sits at a known place whatever the sequence's
  // length (rows past the cache's end are zero-filled by the copy): the producer asks for it
  // before the length has even been read, which takes a global-memory round trip off the start.
  const bool spec = p.n_splits == 1 && p.block_table == nullptr;
  if (spec && tid == 32 * 4 * NG) {
    const uint64_t policy = l2_policy_evict_first();
    mbar_arrive_expect_tx(bar_full, STAGE_BYTES);
#pragma unroll
    for (int h = 0; h < D / 64; ++h) {
      tma_load_5d(base + h * (kTileTokens * 128), &tm_k, bar_full, h * 64, 0, g, b, layer, policy);
      tma_load_5d(base + TILE_BYTES + h * (kTileTokens * 128), &tm_v, bar_full, h * 64, 0, g, b, layer, policy);
    }
  }

  int kv_len = p.seq_lens[b];
  kv_len = kv_len < 0 ? 0 : (kv_len > p.max_seq_len ? p.max_seq_len : kv_len);
  int tile_begin, tile_end;
  split_range(kv_len, p.n_splits, split, tile_begin, tile_end);
  const int n_my = tile_end - tile_begin;

  if (warp == 4 * NG) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && n_my == 0 && spec) {
      // an empty sequence: nobody will consume the tile asked for above; stay until it has landed
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(bar_full, 0) && global_timer_ns() - t0 < kWaitLimitNs) {
      }
    }
    if (lane == 0 && n_my > 0) {
      const uint64_t policy = l2_policy_evict_first();
      const int tiles_per_block = p.block_tokens / kTileTokens;   // used only when paged
      int issued = spec ? 1 : 0;
      bool ok = true;
      for (int i = issued; i < n_my && ok; ++i) {
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
  const int cw = warp & 3, grp = warp >> 2;                           // token slice, consumer group
  const int k_tok = cw * 16 + (mi >> 1) * 8 + r8, k_chunk = mi & 1;   // K: non-transposed
  const int v_tok = cw * 16 + (mi & 1) * 8 + r8, v_chunk = mi >> 1;   // V: transposed

  bool alive = true;
  for (int i = grp; i < n_my; i += NG) {
    const int s = i % STAGES;
    if (!mbar_wait(bar_full + 8 * s, (i / STAGES) & 1, abort_flag)) {
      alive = false;
      break;
    }
    const uint32_t k_base = base + s * STAGE_BYTES;
    const uint32_t v_base = k_base + TILE_BYTES;
    const int tb = (tile_begin + i) * kTileTokens + cw * 16;     // first token of this warp's slice
    if (tb < kv_len) {
      if (tb + 16 > kv_len) {
        // rows past the end of the sequence hold whatever the page held: clear V there so that
        // a zero probability times a stale non-finite value cannot reach the accumulator
        uint8_t* vt = smem + s * STAGE_BYTES + TILE_BYTES;
        const int first = kv_len - (tile_begin + i) * kTileTokens;      // first invalid local row
        for (int t = first + (lane >> 3); t < cw * 16 + 16; t += 4) {
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

  // ------------------------------------------------------------ merge the consumer warps' partials
  // (named barrier over the 128 consumer threads; the producer warp has no part in it)
  asm volatile("bar.sync 1, %0;" ::"n"(128 * NG) : "memory");
  if (!alive || *abort_flag) return;   // a wait expired somewhere in this CTA: leave outputs alone
  constexpr int NW = 4 * NG;                                           // consumer warps
  float* const o_sm = reinterpret_cast<float*>(smem);                  // [NW][16][OPITCH]
  float* const m_sm = o_sm + NW * 16 * OPITCH;                         // [NW][16]
  float* const l_sm = m_sm + NW * 16;                                  // [NW][16]
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  {
    float* ow = o_sm + warp * 16 * OPITCH;
    // only the rows in use (7 of the 16 for the 7-head group of a decode step)
    if (row0 < p.rows) {
#pragma unroll
      for (int nt = 0; nt < NT_O; ++nt)
        *reinterpret_cast<float2*>(ow + row0 * OPITCH + nt * 8 + col) = make_float2(o[nt][0], o[nt][1]);
    }
    if (row1 < p.rows) {
#pragma unroll
      for (int nt = 0; nt < NT_O; ++nt)
        *reinterpret_cast<float2*>(ow + row1 * OPITCH + nt * 8 + col) = make_float2(o[nt][2], o[nt][3]);
    }
    if ((lane & 3) == 0) {
      m_sm[warp * 16 + row0] = m0;
      m_sm[warp * 16 + row1] = m1;
      l_sm[warp * 16 + row0] = l0;
      l_sm[warp * 16 + row1] = l1;
    }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(128 * NG) : "memory");
  // Every thread of the final pass derives its row's weights 2^(m_w - M) / den itself (16 shared
  // loads and NW exponentials): cheaper than a separate weight phase behind two more barriers.
  const int item = lb * p.n_kv_heads + g;
  for (int idx = tid; idx < p.rows * (D / 4); idx += 128 * NG) {
    const int r = idx / (D / 4), c = (idx - r * (D / 4)) * 4;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) M = fmaxf(M, m_sm[w * 16 + r]);
    float den = 0.f;
    float wt[NW];
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      wt[w] = M != -INFINITY ? fast_exp2(m_sm[w * 16 + r] - M) : 0.f;
      den += l_sm[w * 16 + r] * wt[w];
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float f = wt[w] * inv;
      const float4 x = *reinterpret_cast<const float4*>(o_sm + (w * 16 + r) * OPITCH + c);
      acc.x += x.x * f;
      acc.y += x.y * f;
      acc.z += x.z * f;
      acc.w += x.w * f;
    }
    const float lse2 = den > 0.f ? M + log2f(den) : -INFINITY;
    if (p.n_splits == 1) {
      const int t = r / p.group, h = g * p.group + (r - t * p.group);
      const size_t orow = ((size_t)lb * p.n_q + t) * p.n_q_heads + h;
      uint2 packed;
      packed.x = pack_bf16x2(acc.x, acc.y);
      packed.y = pack_bf16x2(acc.z, acc.w);
      *reinterpret_cast<uint2*>(p.out + orow * D + c) = packed;
      if (p.lse && c == 0) p.lse[orow] = lse2 * kLn2;
    } else {
      const size_t prow = ((size_t)item * p.n_splits + split) * p.rows + r;
      *reinterpret_cast<float4*>(p.ws_o + prow * D + c) = acc;
      if (c == 0) p.ws_lse[prow] = lse2;
    }
  }
  if (p.n_splits == 1) return;

  // ------------------------------------------------------------ merge of the item's splits
  // The CTA that brings an item's last partial merges them all, in split order (so the result
  // does not depend on which CTA that is):  out = sum_s w_s o_s / sum_s w_s,  w_s = 2^(lse_s - max).
  int* const last_sm = reinterpret_cast<int*>(l_sm + NW * 16);
  __threadfence();
  asm volatile("bar.sync 1, %0;" ::"n"(128 * NG) : "memory");
  if (tid == 0) {
    const int old = atomicAdd(p.ws_cnt + item, 1);
    __threadfence();
    *last_sm = old == p.n_splits - 1;
  }
  asm volatile("bar.sync 1, %0;" ::"n"(128 * NG) : "memory");
  if (!*last_sm) return;
  const float* lse_base = p.ws_lse + (size_t)item * p.n_splits * p.rows;
  const float* o_base = p.ws_o + (size_t)item * p.n_splits * p.rows * D;
  for (int idx = tid; idx < p.rows * (D / 4); idx += 128 * NG) {
    const int r = idx / (D / 4), c4 = idx - r * (D / 4);
    float M = -INFINITY;
#pragma unroll 4
    for (int s = 0; s < p.n_splits; ++s) M = fmaxf(M, __ldcg(lse_base + s * p.rows + r));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (M != -INFINITY) {
#pragma unroll 4
      for (int s = 0; s < p.n_splits; ++s) {
        const float w = fast_exp2(__ldcg(lse_base + s * p.rows + r) - M);
        const float4 v = __ldcg(reinterpret_cast<const float4*>(o_base + ((size_t)s * p.rows + r) * D + c4 * 4));
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
// Test hook (specvlm_debug_set_attn_splits): > 0 forces the split count of the 16-row kernel so
// that tests reach every path; 0 leaves the choice to the cost model below.
static std::atomic<int> g_forced_splits{0};

constexpr int kRows16Max = 16;     // windows up to this many rows run on attn_rows16_kernel

// How many CTAs share one (layer, sequence, KV head): the split count with the lowest estimated
// launch time (a test hook can force it).
static int choose_splits(int max_seq_len, int64_t items) {
  const int n_tiles = (max_seq_len + kTileTokens - 1) / kTileTokens;
  const int forced = g_forced_splits.load(std::memory_order_relaxed);
  int best = 1;
  if (forced > 0) {
    best = forced;
  } else {
    // Unit: the time one group of four warps needs for a tile, about 0.5 us.  A launch whose CTAs
    // fit one per SM runs the two-group kernel (half that per tile); otherwise two CTAs share an
    // SM and the launch runs in rounds over the resident slots.  Every CTA adds a start-up /
    // epilogue cost of two to three tiles; splitting adds the counter reset before the launch and
    // the merge at its end (about eight tiles, measured); and no launch beats the time HBM needs
    // for the bytes (about 95 tiles of 32 KB per unit).  With these figures neither the 755-token
    // nor the 6400-token draft cache of the 28-layer draft is split, which is what measures best.
    const int64_t sms = sm_count(), slots = 2 * sms;
    const double hbm_floor = (double)items * n_tiles / 95.0;
    double best_cost = 1e300;
    for (int s = 1; s <= 64 && s <= n_tiles; ++s) {
      const int per = (n_tiles + s - 1) / s;
      if ((s - 1) * per >= n_tiles) continue;            // would leave an empty split
      const int64_t ctas = items * s;
      double cost = ctas <= sms ? 0.5 * per + 3.0 : (double)((ctas + slots - 1) / slots) * (per + 2.0);
      if (cost < hbm_floor) cost = hbm_floor;
      if (s > 1) cost += 8.0;
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

// scratch of the 16-row kernel: split partials [item][split][rows][D] fp32, their LSEs, and one
// arrival counter per item
static void rows16_ws_layout(const specvlm_kv_t* kv, int32_t batch, int rows, int splits, size_t& o_bytes,
                             size_t& lse_bytes, size_t& cnt_bytes) {
  const size_t items = (size_t)kv->n_layers * batch * kv->n_kv_heads;
  o_bytes = round_up(items * splits * rows * kv->head_dim * sizeof(float), 256);
  lse_bytes = round_up(items * splits * rows * sizeof(float), 256);
  cnt_bytes = round_up(items * sizeof(int32_t), 256);
}

static size_t rows16_ws_bytes(const specvlm_kv_t* kv, int32_t batch, int rows) {
  const int64_t items = (int64_t)kv->n_layers * batch * kv->n_kv_heads;
  const int splits = choose_splits(kv->max_seq_len, items);
  if (splits == 1) return 256;
  size_t a, b, c;
  rows16_ws_layout(kv, batch, rows, splits, a, b, c);
  return a + b + c;
}

// tcgen05 path (attn_tc.cu)
size_t attn_tc_ws_bytes(const specvlm_kv_t* kv, int32_t batch, int rows, int group);
size_t attn_tc_tree_extra_bytes(int32_t batch, int32_t n_nodes);
int32_t attn_tc_launch(const specvlm_kv_t* kv, const void* q, int32_t batch, int32_t n_q_heads, int32_t n_q,
                       float sm_scale, void* out, float* lse, void* ws, size_t ws_bytes, int32_t* d_status,
                       cudaStream_t st, const int32_t* tree_parents);

template <int D, int STAGES, int NG>
static int32_t launch_rows16_s(const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                               dim3 grid, cudaStream_t st) {
  constexpr int SMEM = STAGES * 2 * kTileTokens * D * 2 + 1024 + 16 * STAGES + 16;
  auto kern = attn_rows16_kernel<D, STAGES, NG>;
  static std::atomic<uint64_t> attr_done{0};
  if (!smem_attr_once(attr_done, reinterpret_cast<const void*>(kern), SMEM)) return SPECVLM_ERR_CUDA;
  // launched with programmatic stream serialization: see the kernel's griddepcontrol.wait
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(32 * (4 * NG + 1), 1, 1);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, tk, tv, p) != cudaSuccess) return SPECVLM_ERR_CUDA;
  return launch_status();
}

// Ring depth: 3 stages let two CTAs share an SM; a launch with no more CTAs than SMs would leave
// every SM with one CTA and 96 KB of copies in flight, too little to cover the HBM latency, so it
// takes 6 stages and two consumer groups instead.
template <int D>
static int32_t launch_rows16(const CUtensorMap& tk, const CUtensorMap& tv, const AttnParams& p,
                             dim3 grid, cudaStream_t st) {
  const int64_t ctas = (int64_t)grid.x * grid.y * grid.z;
  constexpr int kDeep = D == 128 ? 6 : 12;
  return ctas <= sm_count() ? launch_rows16_s<D, kDeep, 2>(tk, tv, p, grid, st)
                            : launch_rows16_s<D, 3, 1>(tk, tv, p, grid, st);
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
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (rows > kRows16Max)
    return attn_tc_launch(kv, q, batch, n_q_heads, n_q, sm_scale, out, lse, ws, ws_bytes, d_status, st, nullptr);

  const int64_t lb64 = (int64_t)kv->n_layers * batch;
  if (lb64 > 65535 || kv->n_kv_heads > 65535) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  const int64_t items = lb64 * kv->n_kv_heads;
  const int splits = choose_splits(kv->max_seq_len, items);
  size_t o_bytes = 0, lse_bytes = 0, cnt_bytes = 0;
  if (splits > 1) {
    rows16_ws_layout(kv, batch, rows, splits, o_bytes, lse_bytes, cnt_bytes);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return SPECVLM_ERR_INVALID_ARG;
    if (ws_bytes < o_bytes + lse_bytes + cnt_bytes) return SPECVLM_ERR_WORKSPACE_TOO_SMALL;
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
  p.ws_cnt = nullptr;
  if (splits > 1) {
    uint8_t* w = static_cast<uint8_t*>(ws);
    p.ws_o = reinterpret_cast<float*>(w);
    p.ws_lse = reinterpret_cast<float*>(w + o_bytes);
    p.ws_cnt = reinterpret_cast<int32_t*>(w + o_bytes + lse_bytes);
    if (cudaMemsetAsync(p.ws_cnt, 0, (size_t)items * sizeof(int32_t), st) != cudaSuccess) return SPECVLM_ERR_CUDA;
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

  dim3 grid((unsigned)splits, (unsigned)kv->n_kv_heads, (unsigned)lb64);
  return kv->head_dim == 128 ? launch_rows16<128>(tk, tv, p, grid, st) : launch_rows16<64>(tk, tv, p, grid, st);
}

}  // namespace specvlm

using namespace specvlm;

extern "C" void specvlm_debug_set_attn_splits(int32_t n_splits) {
  g_forced_splits.store(n_splits > 0 ? n_splits : 0, std::memory_order_relaxed);
}

extern "C" size_t specvlm_attn_workspace_bytes(const specvlm_kv_t* kv, int32_t batch,
                                               int32_t n_q_heads, int32_t gamma) {
  if (!kv || batch < 1 || n_q_heads < 1 || gamma < 0 || kv->n_kv_heads < 1 ||
      n_q_heads % kv->n_kv_heads != 0 || kv->n_layers < 1 || kv->max_seq_len < 1)
    return 0;
  const int rows = (n_q_heads / kv->n_kv_heads) * (gamma + 1);
  if (n_q_heads / kv->n_kv_heads > 16 || gamma > 8) return 0;
  if (rows > kRows16Max) return batch <= kSchedMaxBatch ? attn_tc_ws_bytes(kv, batch, rows, n_q_heads / kv->n_kv_heads) : 0;
  return rows16_ws_bytes(kv, batch, rows);
}

extern "C" int32_t specvlm_draft_decode_attn(const specvlm_kv_t* kv, const void* q, int32_t batch,
                                             int32_t n_q_heads, float sm_scale, void* out,
                                             float* lse_or_null, void* ws, size_t ws_bytes,
                                             int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  return attn_common(kv, q, batch, n_q_heads, 1, sm_scale, out, lse_or_null, ws, ws_bytes, d_status,
                     stream);
}

extern "C" int32_t specvlm_verify_attn(const specvlm_kv_t* kv, const void* q, int32_t batch,
                                       int32_t n_q_heads, int32_t gamma, float sm_scale, void* out,
                                       float* lse_or_null, void* ws, size_t ws_bytes,
                                       int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (gamma < 0 || gamma > 8) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  return attn_common(kv, q, batch, n_q_heads, gamma + 1, sm_scale, out, lse_or_null, ws, ws_bytes,
                     d_status, stream);
}

extern "C" size_t specvlm_verify_tree_workspace_bytes(const specvlm_kv_t* kv, int32_t batch, int32_t n_q_heads,
                                                      int32_t n_nodes) {
  if (!kv || batch < 1 || batch > kSchedMaxBatch || n_q_heads < 1 || n_nodes < 1 || n_nodes > 64 ||
      kv->n_kv_heads < 1 || n_q_heads % kv->n_kv_heads != 0 || kv->n_layers < 1 || kv->max_seq_len < 1)
    return 0;
  const int rows = (n_q_heads / kv->n_kv_heads) * n_nodes;
  if (n_q_heads / kv->n_kv_heads > 16) return 0;
  return attn_tc_ws_bytes(kv, batch, rows, n_q_heads / kv->n_kv_heads) + attn_tc_tree_extra_bytes(batch, n_nodes);
}

extern "C" int32_t specvlm_verify_tree_attn(const specvlm_kv_t* kv, const void* q, const int32_t* parents,
                                            int32_t batch, int32_t n_q_heads, int32_t n_nodes, float sm_scale,
                                            void* out, float* lse_or_null, void* ws, size_t ws_bytes,
                                            int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  int32_t rc = validate_kv(kv, batch, true);
  if (rc != SPECVLM_OK) return rc;
  if (!q || !out || !parents || n_q_heads < 1 || n_nodes < 1 || !(sm_scale > 0.f)) return SPECVLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || n_q_heads % kv->n_kv_heads != 0) return SPECVLM_ERR_INVALID_ARG;
  const int group = n_q_heads / kv->n_kv_heads;
  if (group > 16 || n_nodes > 64) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  return attn_tc_launch(kv, q, batch, n_q_heads, n_nodes, sm_scale, out, lse_or_null, ws, ws_bytes, d_status,
                        static_cast<cudaStream_t>(stream), parents);
}
