// Streaming softmax attention over a bf16 K/V cache on the 5th-generation tensor cores of sm_100a:
// (gamma+1)-query verification attention and tree verification, i.e. windows of 17 to 128 rows per
// KV head and set of CTAs (a wider window is cut into parts that share one launch; up to 16 rows run on the kernel of
// attn.cu).
//
// One persistent CTA per SM streams a contiguous slice of the flat (layer, sequence, KV head, tile)
// list (attn_sched.h), so the cache is read exactly once, every SM moves the same number of bytes
// and only two partial results per CTA ever touch scratch memory.  A tile is 128 tokens: two
// 64-token sub-tiles (one cache page each) as the TMA moves them.
//
// Roles inside a CTA (12 warps = 3 warpgroups; the first gives registers to the other two):
//   warp 0     TMA producer of the item's query rows and of the K tiles
//   warp 3     TMA producer of the V tiles.  K and V have rings of their own because a K tile is
//              free again as soon as S = Q K^T has been computed, long before its V tile; and
//              producers of their own because one thread cannot issue all copies of a tile
//              within the time HBM needs to deliver it.
//   warp 1     issues S = Q K^T (one thread, tcgen05.mma, accumulator in TMEM)
//   warp 2     issues O += P V (one thread)
//   warps 4-7  softmax group 0: the even tiles of the slice
//   warps 8-11 softmax group 1: the odd tiles.  Each group has its own S buffer, P buffer, running
//              (max, sum) and its own O accumulator; the two are merged once per item.
// 128-token tiles keep the two issuing threads, whose per-tile cost in barrier round trips is
// fixed, below the time HBM needs to deliver a tile.
// The GQA group's heads times the query tokens are the M rows of the tiles: M = 64 when they fit
// (row r lives in TMEM lane 32 (r / 16) + r % 16), else M = 128 (row r in lane r); a softmax warp
// owns the rows of its 32 TMEM lanes.
//
// The running maximum of a row is only raised when a tile's maximum exceeds it by more than 2^8; O
// is then rescaled in place in TMEM.  Probabilities stay below 2^8, well inside bf16 / fp32 range,
// and the common tile needs no pass over O at all.
#include "attn.cuh"
#include "attn_sched.h"
#include "host_util.h"

namespace specvlm {

struct AttnTcParams {
  __nv_bfloat16* out;         // [L][B][n_win][Hq][D]
  float* lse;                 // [L][B][n_win][Hq] or null
  float* ws_o;                // partial results: [2 * grid][rows][D], normalised
  float* ws_lse;              // [2 * grid][rows], log2 units
  int32_t* ws_cnt;            // [items] arrival counters, zero at launch
  const int32_t* block_table; // [B][max_blocks] or null
  const int32_t* seq_lens;    // [B]
  int32_t* d_status;
  const uint64_t* anc;        // [B][n_win] ancestor masks of a draft tree (<= 64 nodes), or null: the window is a chain
  int32_t batch, n_layers, n_q_heads, n_kv_heads, group;
  int32_t n_win;              // tokens of the whole window
  int32_t n_parts, q_per;     // the window is cut into n_parts parts of q_per tokens (the last may be shorter)
  int32_t rows;               // rows of a full part = q_per * group (<= 128): the row pitch of the scratch slots
  int32_t max_blocks, block_tokens, max_seq_len;
  float scale_log2;           // sm_scale * log2(e)
};

constexpr float kRescaleThreshold = 8.f;   // log2 units
constexpr int kMaxTreeNodes = 64;          // a window mask is one 64-bit word per node
constexpr int kBigTokens = 2 * kTileTokens;          // tokens per MMA tile
constexpr int kTcThreads = 384;
// setmaxnreg moves registers between the warps of a CTA inside the pool the CTA got at launch
// (threads x registers per thread as compiled: 384 x 168), and an increase blocks until the pool
// has them -- for ever, if the requests add up to more than the pool.  The launch code checks the
// sum against the compiled kernel's pool and refuses to launch otherwise.
constexpr int kRegsLight = 96, kRegsSoftmax = 200;
constexpr int kRegsNeeded = 128 * kRegsLight + 256 * kRegsSoftmax;

template <int N> __device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N> __device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}

// 16 TMEM lanes x 64 fp32 columns -> 32 registers per thread: registers 4j, 4j+1 hold lane
// (base + tid/4), columns 8j + 2(tid%4) + {0,1}; registers 4j+2, 4j+3 the same columns of lane
// (base + 8 + tid/4).
__device__ __forceinline__ void tmem_ld_16x256b_x8(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_16x256b_x8(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.16x256b.x8.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ldg_cg_f32(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float4 ldg_cg_f32x4(const float* p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ int clamp_len(int n, int max_len) { return n < 0 ? 0 : (n > max_len ? max_len : n); }

// Cold paths of the softmax loop, kept out of line: the loop's code has to stay small enough for
// the instruction cache (with the mask logic inline the 128-row variant ran 25 % slower, although
// only one or two tiles of an item ever need a mask).
//
// Tiles that overlap the window of new tokens: the invisible logits of this thread's two rows
// (a 16-lane half of S: rows lr and lr + 8, columns 8j + lc + {0, 1} of each 64-column block) are
// overwritten with -inf in tensor memory, so the loop itself knows no masks.  Visibility of key
// `tok` for the row of query token t: every key before the window, and inside the window the
// positions whose bit is set in the row's mask -- the token's ancestors and itself for a tree
// (a0, a1 = the rows' masks), positions up to t for a chain (a0, a1 = the rows' limits `lim`:
// key tok is visible when tok < lim).
template <bool TREE>
__device__ __noinline__ void mask_s_half(uint32_t saddr, int tile_tok0, int win0, int lc, uint64_t a0, uint64_t a1) {
  const uint64_t a[2] = {a0, a1};
#pragma unroll 1
  for (int c = 0; c < 2; ++c) {
    uint64_t mk[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      if constexpr (TREE) {
        // 128 visibility bits of the tile: the keys before the window, then the row's window mask
        // at the window's offset in the tile
        const int sh = win0 - tile_tok0;                       // tile column of window position 0
        unsigned __int128 full = 0;
        if (a[e]) {
          if (sh > 0) full = sh >= 128 ? ~(unsigned __int128)0 : (((unsigned __int128)1 << sh) - 1);
          const unsigned __int128 w = a[e];
          full |= sh >= 0 ? (sh < 128 ? w << sh : (unsigned __int128)0)
                          : (sh > -64 ? w >> (-sh) : (unsigned __int128)0);
        }
        mk[e] = (uint64_t)(full >> (64 * c)) >> lc;
      } else {
        const int n_vis = (int)a[e] - tile_tok0 - 64 * c;       // visible columns of the block
        mk[e] = (n_vis <= 0 ? 0ull : (n_vis >= 64 ? ~0ull : ((1ull << n_vis) - 1ull))) >> lc;
      }
    }
    uint32_t v[32];
    tmem_ld_16x256b_x8(saddr + 64 * c, v);
    tmem_ld_wait();
#pragma unroll
    for (int k = 0; k < 32; ++k)
      if (!((mk[(k >> 1) & 1] >> ((k >> 2) * 8 + (k & 1))) & 1ull)) v[k] = 0xff800000u;   // -inf
    tmem_st_16x256b_x8(saddr + 64 * c, v);
  }
  tmem_st_wait();
}

// A row maximum grew past the lazy-rescale threshold: the rows' O accumulators (16-lane half,
// d columns from oaddr on) are multiplied by f0 (row lr) and f1 (row lr + 8) in tensor memory.
template <int D>
__device__ __noinline__ void rescale_o_half(uint32_t oaddr, float f0, float f1) {
#pragma unroll 1
  for (int cc = 0; cc < D / 64; ++cc) {
    uint32_t o[32];
    tmem_ld_16x256b_x8(oaddr + cc * 64, o);
    tmem_ld_wait();
#pragma unroll
    for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * (((k >> 1) & 1) ? f1 : f0));
    tmem_st_16x256b_x8(oaddr + cc * 64, o);
  }
  tmem_st_wait();
}

// Shared-memory plan.  A small region (barriers, flags, per-sequence tile counts, the softmax
// groups' row statistics) sits at the start of the dynamic shared memory; the tile rings and the
// operand tiles follow at the next 1024-byte boundary.
template <int D, int M>
struct TcCfg {
  static constexpr int SUB_BYTES = kTileTokens * D * 2;         // one 64-token K (or V) sub-tile
  static constexpr int NKP = D == 128 ? 2 : 3;                  // K ring: pair slots (128 tokens)
  static constexpr int NVP = D == 128 ? (M == 64 ? 3 : 2) : 3;  // V ring: pair slots
  static constexpr int NQ = (D == 128 && M == 128) ? 1 : 2;     // query buffers
  static constexpr int Q_BYTES = M * D * 2;                     // A operand of S = Q K^T
  static constexpr int P_BYTES = M * kBigTokens * 2;            // A operand of O += P V
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = OFF_K + NKP * 2 * SUB_BYTES;
  static constexpr int OFF_Q = OFF_V + NVP * 2 * SUB_BYTES;
  static constexpr int OFF_P = OFF_Q + NQ * Q_BYTES;
  static constexpr int BIG = OFF_P + 2 * P_BYTES;
  static constexpr int N_BARS = 2 * NKP + 2 * NVP + 17;
  static constexpr int SM_BAR = 0;
  static constexpr int SM_MISC = SM_BAR + 8 * N_BARS;
  static constexpr int SM_PREFIX = SM_MISC + 32;
  static constexpr int SM_STATS = SM_PREFIX + (kSchedMaxBatch + 1) * 4;     // [2 groups][M rows] float2
  static constexpr int SMALL_USED = SM_STATS + 2 * M * 8;
  static constexpr int SMALL = (SMALL_USED + 1023) / 1024 * 1024;
  static constexpr int kMaxSmem = 232448;                       // 227 KB
  // a spare KB for a base that is not 1024-byte aligned, where there is room for it
  static constexpr int TOTAL = SMALL + BIG + (SMALL + BIG + 1024 <= kMaxSmem ? 1024 : 0);
  static constexpr uint32_t COL_S = 0, COL_O = 2 * kBigTokens;  // TMEM: S of group g at 128 g, O at 256 + D g
  static constexpr uint32_t TMEM_COLS = 512;
  static_assert(SMALL + BIG <= kMaxSmem, "shared-memory plan does not fit");
};

// TREE: the window's visibility comes from per-token ancestor masks instead of the chain rule.
// A template parameter, not a run-time branch: the chain kernel's code is untouched by the tree
// variant (the softmax loop's speed proved sensitive to what is compiled around it).
template <int D, int M, bool TREE>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ AttnTcParams p) {
  using C = TcCfg<D, M>;
  constexpr int SUB_BYTES = C::SUB_BYTES, NKP = C::NKP, NVP = C::NVP, NQ = C::NQ;
  constexpr int Q_BYTES = C::Q_BYTES, P_BYTES = C::P_BYTES;
  constexpr int NH = M / 64;                          // 16-lane halves a softmax warp may own
  constexpr uint32_t kIdescQK = umma_idesc_bf16(M, kBigTokens, false, false);
  constexpr uint32_t kIdescPV = umma_idesc_bf16(M, D, false, true);   // V tile: channels run along the row

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t big = (raw_addr + C::SMALL_USED + 1023u) & ~1023u;
  uint8_t* const big_ptr = smem_raw + (big - raw_addr);
  const uint32_t k_sm = big + C::OFF_K, v_sm = big + C::OFF_V, q_sm = big + C::OFF_Q, p_sm = big + C::OFF_P;
  const uint32_t bar0 = raw_addr + C::SM_BAR;
  const uint32_t bar_k_full = bar0, bar_k_empty = bar_k_full + 8 * NKP;
  const uint32_t bar_v_full = bar_k_empty + 8 * NKP, bar_v_empty = bar_v_full + 8 * NVP;
  const uint32_t bar_q_full = bar_v_empty + 8 * NVP;   // [2]
  const uint32_t bar_q_empty = bar_q_full + 16;        // [2]
  const uint32_t bar_s_full = bar_q_empty + 16;        // [2]: one per softmax group
  const uint32_t bar_s_empty = bar_s_full + 16;        // [2]
  const uint32_t bar_p_full = bar_s_empty + 16;        // [2]
  const uint32_t bar_p_empty = bar_p_full + 16;        // [2]
  const uint32_t bar_o_full = bar_p_empty + 16;
  const uint32_t bar_o_empty = bar_o_full + 8;
  const uint32_t bar_ep_stats = bar_o_empty + 8;       // both groups' row statistics are in shared memory
  const uint32_t bar_ep_done = bar_ep_stats + 8;       // a partial result has been written
  const uint32_t bar_ep_flag = bar_ep_done + 8;        // ... and the arrival counter has been read
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(smem_raw + C::SM_MISC);
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + C::SM_MISC + 8);
  volatile int* const last_flag = reinterpret_cast<volatile int*>(smem_raw + C::SM_MISC + 16);
  volatile int* const any_empty = reinterpret_cast<volatile int*>(smem_raw + C::SM_MISC + 20);
  int* const prefix = reinterpret_cast<int*>(smem_raw + C::SM_PREFIX);
  float2* const stats = reinterpret_cast<float2*>(smem_raw + C::SM_STATS);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // the plan needs the tiles inside the allocation (true whenever the base is 1024-byte aligned)
  if (big + C::BIG > raw_addr + C::TOTAL) {
    if (tid == 0 && p.d_status) *p.d_status = SPECVLM_ERR_CUDA;
    return;
  }

  // ------------------------------------------------------------------ set-up
  if (tid == 0) {
    for (int s = 0; s < NKP; ++s) {
      mbar_init(bar_k_full + 8 * s, 1);
      mbar_init(bar_k_empty + 8 * s, 1);
    }
    for (int s = 0; s < NVP; ++s) {
      mbar_init(bar_v_full + 8 * s, 1);
      mbar_init(bar_v_empty + 8 * s, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_q_full + 8 * i, 1);
      mbar_init(bar_q_empty + 8 * i, 1);
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_s_empty + 8 * i, 4);
      mbar_init(bar_p_full + 8 * i, 4);
      mbar_init(bar_p_empty + 8 * i, 1);
    }
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_empty, 8);
    mbar_init(bar_ep_stats, 8);
    mbar_init(bar_ep_done, 8);
    mbar_init(bar_ep_flag, 1);
    *abort_flag = 0;
    *any_empty = 0;
    prefix[0] = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
  // tiles per sequence, then their running sum
  for (int b = tid; b < p.batch; b += blockDim.x) {
    const int n = clamp_len(p.seq_lens[b], p.max_seq_len);
    prefix[b + 1] = (n + kBigTokens - 1) / kBigTokens;
    if (n == 0) *any_empty = 1;
  }
  // query rows that no item uses stay zero (the TMA only ever writes the first `rows` rows)
  for (int idx = tid; idx < NQ * Q_BYTES / 16; idx += blockDim.x)
    *reinterpret_cast<uint4*>(big_ptr + C::OFF_Q + idx * 16) = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    int carry = 0;
    for (int b0 = 0; b0 < p.batch; b0 += 32) {
      const int b = b0 + lane;
      int v = b < p.batch ? prefix[b + 1] : 0;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += o;
      }
      if (b < p.batch) prefix[b + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const int hkv = p.n_kv_heads;
  const int64_t total = (int64_t)p.n_layers * hkv * prefix[p.batch];
  // A window of more than 128 rows is cut into parts of q_per query tokens, the accumulators of one
  // part filling the tensor memory.  The parts run side by side in this one launch: the grid is
  // n_parts sets of CTAs, every set slices the same flat tile list in the same way, so CTA c of each
  // set streams the same K/V tiles at about the same time and all but the first to ask find them in
  // the L2 cache -- HBM delivers every tile once, not once per part.
  const int ctas_per_part = (int)gridDim.x / p.n_parts;
  const int part = blockIdx.x / ctas_per_part;          // >= n_parts: a spare CTA without work
  const int cta = blockIdx.x - part * ctas_per_part;    // index inside the part's set
  const int gcta = blockIdx.x;                          // index of this CTA's scratch slots
  const int q0 = part * p.q_per;                        // first window token of the part
  const int n_q_part = part < p.n_parts ? (p.n_win - q0 < p.q_per ? p.n_win - q0 : p.q_per) : 0;
  const int rows = n_q_part > 0 ? n_q_part * p.group : 0;   // rows in use (of the M rows of a tile)
  const int n_active = sched_active_ctas(total, ctas_per_part);
  const bool active = total > 0 && rows > 0 && cta < n_active;
  const int64_t T0 = active ? slice_begin(cta, n_active, total) : 0;
  const int64_t T1 = active ? slice_begin(cta + 1, n_active, total) : 0;
  const int n_items = p.n_layers * p.batch * hkv;
  const int n_my = (int)(T1 - T0);

  if (warp == 0 || warp == 3) {
    // ================================================================ TMA producers
    // warp 0: query rows + K tiles; warp 3: V tiles.  Both walk the same slice.
    setmaxnreg_dec<kRegsLight>();
    if (lane == 0 && active) {
      const bool is_k = warp == 0;
      const CUtensorMap* const tm = is_k ? &tm_k : &tm_v;
      tma_prefetch_desc(tm);
      if (is_k) tma_prefetch_desc(&tm_q);
      const uint64_t policy = l2_policy_evict_first();
      const uint64_t policy_q = l2_policy_evict_last();
      const int subs_per_block = p.block_table ? p.block_tokens / kTileTokens : 1;
      const int n_ring = is_k ? NKP : NVP;
      const uint32_t ring_sm = is_k ? k_sm : v_sm, bar_full = is_k ? bar_k_full : bar_v_full;
      const uint32_t bar_empty = is_k ? bar_k_empty : bar_v_empty;
      // K tile: [64-channel block][128 tokens][128 B], the two sub-tiles stacked inside each block;
      // V tile: two sub-tiles of [64-channel block][64 tokens][128 B] one after the other
      const uint32_t blk_stride = is_k ? kBigTokens * 128 : kTileTokens * 128;
      const uint32_t sub_stride = is_k ? kTileTokens * 128 : SUB_BYTES;
      SliceCursor c;
      c.start(T0, T1, prefix, p.batch, hkv);
      bool ok = true;
      int i = 0;
      while (!c.done() && ok) {
        const Segment sg = c.sg;
        if (is_k) {
          // the item's query rows: a box of (64 channels) x (group heads) x (n_q tokens) per 64-channel block
          const int qb = c.seg_idx % NQ;
          if (c.seg_idx >= NQ) ok = mbar_wait(bar_q_empty + 8 * qb, ((c.seg_idx / NQ) - 1) & 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(bar_q_full + 8 * qb, (uint32_t)p.rows * 128u * (D / 64));
#pragma unroll
          for (int h = 0; h < D / 64; ++h)
            tma_load_5d(q_sm + qb * Q_BYTES + h * (M * 128), &tm_q, bar_q_full + 8 * qb, h * 64, 0, q0, sg.g,
                        sg.layer * p.batch + sg.b, policy_q);
        }
        const int n_sub_seq = (clamp_len(p.seq_lens[sg.b], p.max_seq_len) + kTileTokens - 1) / kTileTokens;
        const int32_t* table = p.block_table ? p.block_table + (size_t)sg.b * p.max_blocks : nullptr;
        int blk[2], blk_next[2] = {sg.b, sg.b};
        if (table) {
          const int s0 = 2 * sg.tile0;
          blk_next[0] = __ldg(table + s0 / subs_per_block);
          blk_next[1] = s0 + 1 < n_sub_seq ? __ldg(table + (s0 + 1) / subs_per_block) : 0;
        }
        for (int j = 0; j < sg.n_tiles; ++j, ++i) {
          const int s0 = 2 * (sg.tile0 + j);                    // first sub-tile of this tile
          const int n_sub = n_sub_seq - s0 < 2 ? n_sub_seq - s0 : 2;
          blk[0] = blk_next[0];
          blk[1] = blk_next[1];
          if (table && j + 1 < sg.n_tiles) {                    // table entries of the next tile, one tile ahead
            blk_next[0] = __ldg(table + (s0 + 2) / subs_per_block);
            blk_next[1] = s0 + 3 < n_sub_seq ? __ldg(table + (s0 + 3) / subs_per_block) : 0;
          }
          const int slot = i % n_ring;
          if (i >= n_ring) ok = mbar_wait(bar_empty + 8 * slot, ((i / n_ring) - 1) & 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(bar_full + 8 * slot, n_sub * SUB_BYTES);
          for (int u = 0; u < n_sub; ++u) {
            const int tok = table ? ((s0 + u) % subs_per_block) * kTileTokens : (s0 + u) * kTileTokens;
#pragma unroll
            for (int h = 0; h < D / 64; ++h)
              tma_load_5d(ring_sm + slot * 2 * SUB_BYTES + h * blk_stride + u * sub_stride, tm, bar_full + 8 * slot,
                          h * 64, tok, sg.g, blk[u], sg.layer, policy);
          }
        }
        if (ok) c.next_segment(prefix, p.batch, hkv);
      }
      if (!ok) {
        // a wait expired: report, then stay until this thread's copies in flight have landed (bounded)
        if (p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
        const uint64_t t0 = global_timer_ns();
        for (int k = i > n_ring ? i - n_ring : 0; k < i; ++k)
          while (!mbar_test_wait(bar_full + 8 * (k % n_ring), (k / n_ring) & 1) && global_timer_ns() - t0 < kWaitLimitNs) {
          }
      }
    }
  } else if (warp == 1) {
    // ================================================================ S = Q K^T issuer
    setmaxnreg_dec<kRegsLight>();
    if (lane == 0 && active) {
      SliceCursor c;
      c.start(T0, T1, prefix, p.batch, hkv);
      const uint64_t dq0 = umma_desc_sw128(q_sm, 16, 1024), dk0 = umma_desc_sw128(k_sm, 16, 1024);
      bool ok = true;
      for (int i = 0; i < n_my; ++i) {
        const int g = i & 1, kp = i % NKP, qb = c.seg_idx % NQ;
        ok = mbar_wait(bar_k_full + 8 * kp, (i / NKP) & 1, abort_flag);
        if (ok && c.j == 0) ok = mbar_wait(bar_q_full + 8 * qb, (c.seg_idx / NQ) & 1, abort_flag);
        if (ok && i >= 2) ok = mbar_wait(bar_s_empty + 8 * g, ((i >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t da = umma_desc_advance(dq0, qb * Q_BYTES), db = umma_desc_advance(dk0, kp * 2 * SUB_BYTES);
        const uint32_t d_tmem = tmem_base + C::COL_S + g * kBigTokens;
#pragma unroll
        for (int s = 0; s < D / 16; ++s)
          // 16 channels per step = 32 bytes along the swizzled 128-byte row; channels 64.. are the
          // second 64-channel block of each operand
          umma_bf16_ss(d_tmem, umma_desc_advance(da, (s >> 2) * (M * 128) + (s & 3) * 32),
                       umma_desc_advance(db, (s >> 2) * (kBigTokens * 128) + (s & 3) * 32), kIdescQK, s > 0 ? 1u : 0u);
        umma_commit(bar_s_full + 8 * g);
        umma_commit(bar_k_empty + 8 * kp);
        if (c.last_of_segment()) umma_commit(bar_q_empty + 8 * qb);
        c.next_tile(prefix, p.batch, hkv);
      }
      if (!ok && p.d_status) *p.d_status = SPECVLM_ERR_TIMEOUT;
    }
  } else if (warp == 2) {
    // ================================================================ O += P V issuer
    // The whole warp walks the slice; lane 0 issues.  The other lanes are there for the one job
    // that needs hands: where a sequence ends inside a sub-tile, the V rows past its end hold
    // whatever the page held, and are cleared so that a zero probability times a stale non-finite
    // value cannot reach O.
    setmaxnreg_dec<kRegsLight>();
    if (active) {
      SliceCursor c;
      c.start(T0, T1, prefix, p.batch, hkv);
      const uint64_t dp0 = umma_desc_sw128(p_sm, 16, 1024);
      const uint64_t dv0 = umma_desc_sw128(v_sm, kTileTokens * 128, 1024);   // 64-channel blocks 8 KB apart
      bool ok = true;
      int n_sub_seq = 0, kv_len = 0;
#define PV_WAIT(bar, parity)                                                        \
  do {                                                                              \
    ok = __all_sync(0xffffffffu, mbar_wait((bar), (parity), abort_flag));           \
  } while (0)
      for (int i = 0; i < n_my; ++i) {
        const int g = i & 1, vp = i % NVP;
        if (c.j == 0) {
          kv_len = clamp_len(p.seq_lens[c.sg.b], p.max_seq_len);
          n_sub_seq = (kv_len + kTileTokens - 1) / kTileTokens;
        }
        const int s0 = 2 * (c.sg.tile0 + c.j);
        const int n_sub = n_sub_seq - s0 < 2 ? n_sub_seq - s0 : 2;
        PV_WAIT(bar_v_full + 8 * vp, (i / NVP) & 1);
        if (!ok) break;
        if (s0 + n_sub == n_sub_seq && (kv_len & (kTileTokens - 1)) != 0) {
          uint8_t* vt = big_ptr + C::OFF_V + vp * 2 * SUB_BYTES + (n_sub - 1) * SUB_BYTES;
          const int first = kv_len - (n_sub_seq - 1) * kTileTokens;
          for (int idx = lane; idx < (kTileTokens - first) * (D / 8); idx += 32) {
            const int t = first + idx / (D / 8), c16 = idx % (D / 8);
            *reinterpret_cast<uint4*>(vt + (c16 >> 3) * (kTileTokens * 128) + t * 128 + (c16 & 7) * 16) =
                make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async();
          __syncwarp();
        }
        // the first product of each group overwrites that group's O: the previous item must be out
        if (c.j < 2 && c.seg_idx >= 1) PV_WAIT(bar_o_empty, (c.seg_idx - 1) & 1);
        if (ok) PV_WAIT(bar_p_full + 8 * g, (i >> 1) & 1);
        if (!ok) break;
        if (lane == 0) {
          tc_fence_after_sync();
          const uint64_t da = umma_desc_advance(dp0, g * P_BYTES), db = umma_desc_advance(dv0, vp * 2 * SUB_BYTES);
          const uint32_t d_tmem = tmem_base + C::COL_O + g * D;
          const uint32_t acc0 = c.j >= 2 ? 1u : 0u;
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            if (u < n_sub) {
#pragma unroll
              for (int kt = 0; kt < kTileTokens / 16; ++kt)
                // 16 tokens per step: 32 bytes along P's row, 16 rows of 128 bytes down the V sub-tile
                umma_bf16_ss(d_tmem, umma_desc_advance(da, u * (M * 128) + kt * 32),
                             umma_desc_advance(db, u * SUB_BYTES + kt * 2048), kIdescPV, (u > 0 || kt > 0) ? 1u : acc0);
            }
          }
          umma_commit(bar_p_empty + 8 * g);
          umma_commit(bar_v_empty + 8 * vp);
          if (c.last_of_segment()) umma_commit(bar_o_full);
        }
        __syncwarp();
        c.next_tile(prefix, p.batch, hkv);
      }
#undef PV_WAIT
      if (!ok && p.d_status && lane == 0) *p.d_status = SPECVLM_ERR_TIMEOUT;
    }
  } else {
    // ================================================================ softmax / epilogue (warps 4..11)
    setmaxnreg_inc<kRegsSoftmax>();
    const int grp = (warp - 4) >> 2;              // tiles with (index & 1) == grp
    const int quarter = warp & 3;                 // TMEM lanes [32 * quarter, +32)
    const int gt = (warp & 3) * 32 + lane;        // 0..127 inside the group
    const int st = grp * 128 + gt;                // 0..255 over both groups
    const int lr = lane >> 2, lc = (lane & 3) * 2;   // row inside a 16-lane half (and +8), first column of a pair
    // rows of this warp: half h covers item rows row0(h) + [0, 16), held in TMEM lanes 32 * quarter + 16 h + [0, 16)
    auto row0 = [&](int h) { return M == 64 ? 16 * quarter : 32 * quarter + 16 * h; };
    const int nh = (rows > row0(0) ? 1 : 0) + (NH > 1 && rows > row0(1) ? 1 : 0);

    // sequences without any token: their outputs are zero, their LSE -inf
    if (*any_empty && rows > 0) {
      for (int item = cta; item < n_items; item += ctas_per_part) {
        const int lb = item / hkv, g = item - lb * hkv, b = lb % p.batch;
        if (prefix[b + 1] != prefix[b]) continue;
        for (int idx = st; idx < rows * (D / 8); idx += 256) {
          const int r = idx / (D / 8), c8 = idx - r * (D / 8);
          const int t = r / p.group, h = g * p.group + (r - t * p.group);
          const size_t orow = ((size_t)lb * p.n_win + q0 + t) * p.n_q_heads + h;
          *reinterpret_cast<uint4*>(p.out + orow * D + c8 * 8) = make_uint4(0, 0, 0, 0);
          if (p.lse && c8 == 0) p.lse[orow] = -INFINITY;
        }
      }
    }

    SliceCursor c;
    c.start(T0, T1, prefix, p.batch, hkv);
    bool ok = true;
    int i0 = 0;           // index (inside the slice) of the current segment's first tile
    int n_partial = 0;    // partial epilogues so far
#define SM_WAIT(bar, parity)                                                        \
  do {                                                                              \
    ok = __all_sync(0xffffffffu, mbar_wait((bar), (parity), abort_flag));           \
    if (!ok) goto softmax_done;                                                     \
  } while (0)

    while (!c.done()) {
      const Segment sg = c.sg;
      const int seg_idx = c.seg_idx;
      const int kv_len = clamp_len(p.seq_lens[sg.b], p.max_seq_len);
      // Visibility of key `tok` for a row of query token t: every key before the window of the n_q
      // new tokens, and inside the window the positions whose bit is set in the row's mask -- bits
      // 0..t for a chain, the token's ancestors and itself for a tree.  Rows no item uses see nothing.
      // (A used row always has its own bit set, so a zero mask also marks an unused row.)
      // The chain keeps the equivalent limit form: key tok is visible to token t when tok < lim.
      const int win0 = kv_len - p.n_win;
      float2* const seg_stats = stats;
      if constexpr (M == 128) {
        // ------------------------------------------------------------ 128-row windows: a thread owns a row
        // With M = 128 row r sits in TMEM lane r, so thread `lane` of the warp of quadrant q reads row
        // 32 q + lane whole (tcgen05.ld 32x32b): its maximum and sum need no shuffles, its 128
        // probabilities leave as sixteen 16-byte stores into the swizzled P tile, and the TMEM load of
        // the next 16 columns is in flight while the current 16 are worked on.
        const int my_row = 32 * quarter + lane;
        const bool warp_on = rows > 32 * quarter;         // warp-uniform: some row of this quadrant is in use
        uint64_t my_a;                                       // the row's window mask (tree) or key limit (chain)
        if constexpr (TREE) {
          my_a = my_row < rows ? __ldg(p.anc + (size_t)sg.b * p.n_win + q0 + my_row / p.group) : 0ull;
        } else {
          my_a = my_row < rows ? (uint64_t)(win0 + q0 + my_row / p.group + 1) : 0ull;
        }
        float m_row = -INFINITY, l_row = 0.f;
        const uint32_t prow = p_sm + grp * P_BYTES + my_row * 128;
        const uint32_t psw = (uint32_t)(my_row & 7);

        for (int j = (i0 + grp) & 1; j < sg.n_tiles; j += 2) {
          const int i = i0 + j;
          const int tile_tok0 = (sg.tile0 + j) * kBigTokens;
          const bool need_mask = tile_tok0 + kBigTokens > win0 + (TREE ? 0 : 1);
          SM_WAIT(bar_s_full + 8 * grp, (i >> 1) & 1);
          tc_fence_after_sync();
          if (!warp_on) {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_s_empty + 8 * grp);
            if (i >= 2) SM_WAIT(bar_p_empty + 8 * grp, ((i >> 1) - 1) & 1);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p_full + 8 * grp);
            continue;
          }
          const uint32_t saddr = tmem_base + ((uint32_t)(32 * quarter) << 16) + C::COL_S + grp * kBigTokens;
          if (__builtin_expect(need_mask, 0)) {
            // the out-of-line mask routine works on 16-lane halves with two rows per thread
#pragma unroll 1
            for (int h = 0; h < nh; ++h) {
              const uint64_t a0 = __shfl_sync(0xffffffffu, my_a, 16 * h + lr);
              const uint64_t a1 = __shfl_sync(0xffffffffu, my_a, 16 * h + lr + 8);
              mask_s_half<TREE>(saddr + ((uint32_t)(16 * h) << 16), tile_tok0, win0, lc, a0, a1);
            }
          }
          uint32_t va[16], vb[16];
          // the group's previous product has completed: P may be overwritten, O may be rescaled
          if (i >= 2) SM_WAIT(bar_p_empty + 8 * grp, ((i >> 1) - 1) & 1);
          if (j < 2) {
            // The group's first tile of the item (O is overwritten by its product): the row's reference
            // maximum is the tile's own, found by a pass of its own over the 128 logits (raw products:
            // the scale is positive).
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            tmem_ld_x16(saddr, va);
#pragma unroll 1
            for (int cc = 0; cc < 4; ++cc) {
              tmem_ld_wait();
              tmem_ld_x16(saddr + 32 * cc + 16, vb);
#pragma unroll
              for (int k = 0; k < 16; ++k) mx4[k & 3] = fmaxf(mx4[k & 3], __uint_as_float(va[k]));
              tmem_ld_wait();
              if (cc < 3) tmem_ld_x16(saddr + 32 * cc + 32, va);
#pragma unroll
              for (int k = 0; k < 16; ++k) mx4[k & 3] = fmaxf(mx4[k & 3], __uint_as_float(vb[k]));
            }
            m_row = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
          }
          // Every later tile takes ONE pass: p = 2^(s * scale - m) against the reference maximum the row
          // already has, the tile's own maximum being gathered on the way.  Only if that maximum turns
          // out more than the lazy-rescale threshold above the reference (a warp vote; rare after the
          // first tiles) is the reference raised, O rescaled in tensor memory and the pass repeated: S
          // stays in place until the decision is taken, and the probabilities of the abandoned pass are
          // simply overwritten (whatever they were, up to infinity, they never reach a product).
          // The pass is a rolled loop of four rounds of 32 logits, two TMEM loads of 16 columns each:
          // with 64 logits per round unrolled the code outgrew the instruction cache (the 9-token
          // window of 8 heads per KV head: 357 -> 336 us on 80 layers of 6400 tokens).
          float ps[2];
#pragma unroll 1
          for (int attempt = 0; attempt < 2; ++attempt) {
            const float nmu = m_row == -INFINITY ? 0.f : -m_row;   // a row that sees nothing yet stays at zero
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            ps[0] = ps[1] = 0.f;
            tmem_ld_x16(saddr, va);
#pragma unroll 1
            for (int cc = 0; cc < 4; ++cc) {     // 32 logits per round: four 16-byte chunks of the row
              const uint32_t pblk = prow + (cc >> 1) * (M * 128);
              const uint32_t ch0 = (uint32_t)(cc & 1) * 4;
              tmem_ld_wait();
              tmem_ld_x16(saddr + 32 * cc + 16, vb);
#pragma unroll
              for (int k4 = 0; k4 < 2; ++k4) {
                uint32_t w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const float s0 = __uint_as_float(va[8 * k4 + 2 * u]), s1 = __uint_as_float(va[8 * k4 + 2 * u + 1]);
                  mx4[u] = fmaxf(mx4[u], fmaxf(s0, s1));
                  const float p0 = fast_exp2(fmaf(s0, p.scale_log2, nmu));
                  const float p1 = fast_exp2(fmaf(s1, p.scale_log2, nmu));
                  ps[u & 1] += p0 + p1;
                  w[u] = pack_bf16x2(p0, p1);
                }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(pblk + (((ch0 + k4) ^ psw) << 4)),
                             "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
              }
              tmem_ld_wait();
              if (cc < 3) tmem_ld_x16(saddr + 32 * cc + 32, va);
#pragma unroll
              for (int k4 = 0; k4 < 2; ++k4) {
                uint32_t w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const float s0 = __uint_as_float(vb[8 * k4 + 2 * u]), s1 = __uint_as_float(vb[8 * k4 + 2 * u + 1]);
                  mx4[u] = fmaxf(mx4[u], fmaxf(s0, s1));
                  const float p0 = fast_exp2(fmaf(s0, p.scale_log2, nmu));
                  const float p1 = fast_exp2(fmaf(s1, p.scale_log2, nmu));
                  ps[u & 1] += p0 + p1;
                  w[u] = pack_bf16x2(p0, p1);
                }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(pblk + (((ch0 + 2 + k4) ^ psw) << 4)),
                             "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
              }
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
            const bool up = mx > m_row + kRescaleThreshold;
            if (__builtin_expect(__any_sync(0xffffffffu, up) == 0, 1)) break;
            // raise the reference maximum of those rows, rescale their sums and their O rows, go again
            const float a = up ? fast_exp2(m_row - mx) : 1.f;
            if (up) m_row = mx;
            l_row *= a;
            tc_fence_after_sync();
#pragma unroll 1
            for (int h = 0; h < nh; ++h) {
              const float f0 = __shfl_sync(0xffffffffu, a, 16 * h + lr);
              const float f1 = __shfl_sync(0xffffffffu, a, 16 * h + lr + 8);
              rescale_o_half<D>(tmem_base + ((uint32_t)(32 * quarter + 16 * h) << 16) + C::COL_O + grp * D, f0, f1);
            }
            tc_fence_before_sync();
          }
          tc_fence_before_sync();                // every read of the tile's logits is complete: S is free
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_s_empty + 8 * grp);
          l_row += ps[0] + ps[1];
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p_full + 8 * grp);
        }
        // publish this group's row statistics for the merge below
        if (seg_idx >= 1) SM_WAIT(bar_o_empty, (seg_idx - 1) & 1);
        if (warp_on) seg_stats[grp * M + my_row] = make_float2(m_row, l_row);
      } else {
      uint64_t vis[NH][2];
      int lim[NH][2];
      float m_used[NH][2], l_sum[NH][2];
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int r = row0(h) + lr + 8 * e;
          const int t = r / p.group;
          if constexpr (TREE) {
            vis[h][e] = r < rows ? __ldg(p.anc + (size_t)sg.b * p.n_win + q0 + t) : 0ull;
          } else {
            lim[h][e] = r < rows ? win0 + q0 + t + 1 : 0;
          }
          m_used[h][e] = -INFINITY;
          l_sum[h][e] = 0.f;
        }

      for (int j = (i0 + grp) & 1; j < sg.n_tiles; j += 2) {
        const int i = i0 + j;
        const int tile_tok0 = (sg.tile0 + j) * kBigTokens;
        const bool need_mask = tile_tok0 + kBigTokens > win0 + (TREE ? 0 : 1);
        SM_WAIT(bar_s_full + 8 * grp, (i >> 1) & 1);
        tc_fence_after_sync();
        if (nh == 0) {
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_s_empty + 8 * grp);
        }
        // One copy of the code serves both 16-row halves of a warp (the 128-row variant): the loop is
        // rolled, the current half's state sits at index 0 of its arrays, and the two halves' states
        // change places after each half -- twice per tile, so every tile finds them as it left them.
#pragma unroll 1
        for (int h = 0; h < nh; ++h) {
          // The half's 16 rows x 128 columns are read from TMEM twice, 64 columns at a time, by the
          // same (rolled) code: once for the row maxima, once for the probabilities.  That halves
          // the live registers and the code of the loop; a TMEM load costs far less than the spills.
          const uint32_t saddr = tmem_base + ((uint32_t)(32 * quarter + 16 * h) << 16) + C::COL_S + grp * kBigTokens;
          if (__builtin_expect(need_mask, 0)) {
            if constexpr (TREE) mask_s_half<true>(saddr, tile_tok0, win0, lc, vis[0][0], vis[0][1]);
            else mask_s_half<false>(saddr, tile_tok0, win0, lc, (uint64_t)lim[0][0], (uint64_t)lim[0][1]);
          }
          float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            uint32_t v[32];
            tmem_ld_16x256b_x8(saddr + 64 * c, v);
            tmem_ld_wait();
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int k = 0; k < 32; ++k) mx[k & 3] = fmaxf(mx[k & 3], __uint_as_float(v[k]));
            mx0 = fmaxf(mx0, fmaxf(mx[0], mx[1]));
            mx1 = fmaxf(mx1, fmaxf(mx[2], mx[3]));
          }
          mx0 *= p.scale_log2;                                     // the scale is positive
          mx1 *= p.scale_log2;
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
          // the group's previous product has completed: P may be overwritten, O may be rescaled
          if (h == 0 && i >= 2) SM_WAIT(bar_p_empty + 8 * grp, ((i >> 1) - 1) & 1);
          if (j < 2) {
            // the group's first tile of the item: O is overwritten by this tile's product
            m_used[0][0] = mx0;
            m_used[0][1] = mx1;
          } else {
            const bool up0 = mx0 > m_used[0][0] + kRescaleThreshold, up1 = mx1 > m_used[0][1] + kRescaleThreshold;
            if (__builtin_expect(__any_sync(0xffffffffu, up0 || up1) != 0, 0)) {
              // raise the reference maximum of those rows and rescale their O rows in TMEM
              const float a0 = up0 ? fast_exp2(m_used[0][0] - mx0) : 1.f;
              const float a1 = up1 ? fast_exp2(m_used[0][1] - mx1) : 1.f;
              if (up0) m_used[0][0] = mx0;
              if (up1) m_used[0][1] = mx1;
              l_sum[0][0] *= a0;
              l_sum[0][1] *= a1;
              tc_fence_after_sync();
              rescale_o_half<D>(tmem_base + ((uint32_t)(32 * quarter + 16 * h) << 16) + C::COL_O + grp * D, a0, a1);
              tc_fence_before_sync();
            }
          }
          // probabilities: p = 2^(s * scale - m), with a row that sees nothing yet kept at zero
          const float nmu0 = m_used[0][0] == -INFINITY ? 0.f : -m_used[0][0];
          const float nmu1 = m_used[0][1] == -INFINITY ? 0.f : -m_used[0][1];
          float ps[4] = {0.f, 0.f, 0.f, 0.f};
          // rows of the A operand of O += P V: the item's rows
          const int m0 = row0(h) + lr, m1 = m0 + 8;
          const uint32_t prow0 = p_sm + grp * P_BYTES + m0 * 128 + lc * 2;
          const uint32_t prow1 = p_sm + grp * P_BYTES + m1 * 128 + lc * 2;
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {                            // the tile's two 64-token blocks
            uint32_t v[32];
            tmem_ld_16x256b_x8(saddr + 64 * c, v);
            tmem_ld_wait();
            if (c == 1 && h == nh - 1) {
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive(bar_s_empty + 8 * grp);
            }
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
              const float p0 = fast_exp2(fmaf(__uint_as_float(v[4 * jj]), p.scale_log2, nmu0));
              const float p1 = fast_exp2(fmaf(__uint_as_float(v[4 * jj + 1]), p.scale_log2, nmu0));
              const float p2 = fast_exp2(fmaf(__uint_as_float(v[4 * jj + 2]), p.scale_log2, nmu1));
              const float p3 = fast_exp2(fmaf(__uint_as_float(v[4 * jj + 3]), p.scale_log2, nmu1));
              ps[jj & 1] += p0 + p1;
              ps[2 + (jj & 1)] += p2 + p3;
              asm volatile("st.shared.b32 [%0], %1;" ::"r"(prow0 + c * (M * 128) + ((jj ^ (m0 & 7)) << 4)),
                           "r"(pack_bf16x2(p0, p1)) : "memory");
              asm volatile("st.shared.b32 [%0], %1;" ::"r"(prow1 + c * (M * 128) + ((jj ^ (m1 & 7)) << 4)),
                           "r"(pack_bf16x2(p2, p3)) : "memory");
            }
          }
          l_sum[0][0] += ps[0] + ps[1];
          l_sum[0][1] += ps[2] + ps[3];
          if (NH == 2 && nh == 2) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const float tm = m_used[0][e], tl = l_sum[0][e];
              m_used[0][e] = m_used[NH - 1][e];
              m_used[NH - 1][e] = tm;
              l_sum[0][e] = l_sum[NH - 1][e];
              l_sum[NH - 1][e] = tl;
              if constexpr (TREE) {
                const uint64_t tv = vis[0][e];
                vis[0][e] = vis[NH - 1][e];
                vis[NH - 1][e] = tv;
              } else {
                const int tv = lim[0][e];
                lim[0][e] = lim[NH - 1][e];
                lim[NH - 1][e] = tv;
              }
            }
          }
        }
        if (nh == 0 && i >= 2) SM_WAIT(bar_p_empty + 8 * grp, ((i >> 1) - 1) & 1);
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_p_full + 8 * grp);
      }

        // publish this group's row statistics for the merge below.  A group may get here while the
        // other one still reads the previous segment's statistics: wait until both have left that
        // epilogue (the barrier the PV issuer waits on as well)
        if (seg_idx >= 1) SM_WAIT(bar_o_empty, (seg_idx - 1) & 1);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          if (h >= nh) break;
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            float lt = l_sum[h][e];
            lt += __shfl_xor_sync(0xffffffffu, lt, 1);
            lt += __shfl_xor_sync(0xffffffffu, lt, 2);
            if ((lane & 3) == 0) seg_stats[grp * M + row0(h) + lr + 8 * e] = make_float2(m_used[h][e], lt);
          }
        }
      }

      // ---------------------------------------------------------------- end of the item's segment
      // merge the two groups' accumulators:
      //   O = (w0 O0 + w1 O1) / (w0 l0 + w1 l1),  w_g = 2^(m_g - max(m0, m1))
      const bool complete = sg.tile0 == 0 && sg.n_tiles == sg.item_tiles;
      const int lb = sg.layer * p.batch + sg.b;
      const int slot = partial_slot(gcta, T0, sg.item_begin);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_ep_stats);
      SM_WAIT(bar_ep_stats, seg_idx & 1);
      SM_WAIT(bar_o_full, seg_idx & 1);
      tc_fence_after_sync();
      // a group without a tile in this segment (one-tile segments) has nothing in its accumulator
      const bool has0 = sg.n_tiles >= 2 || (i0 & 1) == 0, has1 = sg.n_tiles >= 2 || (i0 & 1) == 1;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        if (h >= nh) break;
        float w0[2], w1[2], lse2[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int ln = row0(h) + lr + 8 * e;
          const float2 s0 = seg_stats[ln], s1 = seg_stats[M + ln];
          const float l0 = has0 ? s0.y : 0.f, l1 = has1 ? s1.y : 0.f;
          const float ma = l0 > 0.f ? s0.x : -INFINITY, mb = l1 > 0.f ? s1.x : -INFINITY;
          const float mm = fmaxf(ma, mb);
          const float a = l0 > 0.f ? fast_exp2(ma - mm) : 0.f, b = l1 > 0.f ? fast_exp2(mb - mm) : 0.f;
          const float den = a * l0 + b * l1;
          const float inv = den > 0.f ? 1.f / den : 0.f;
          w0[e] = a * inv;
          w1[e] = b * inv;
          lse2[e] = den > 0.f ? mm + log2f(den) : -INFINITY;
        }
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) {
          if ((cc & 1) != (D == 128 ? grp : 0)) continue;       // the groups share the column chunks
          if (D == 64 && grp == 1) continue;
          uint32_t oa[32], ob[32];
          const uint32_t oaddr = tmem_base + ((uint32_t)(32 * quarter + 16 * h) << 16) + C::COL_O + cc * 64;
          if (has0) tmem_ld_16x256b_x8(oaddr, oa);
          if (has1) tmem_ld_16x256b_x8(oaddr + D, ob);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int r = row0(h) + lr + 8 * e;
            if (r >= rows) continue;
            float res[16];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj)
#pragma unroll
              for (int x = 0; x < 2; ++x) {
                const int k = 4 * jj + 2 * e + x;
                float acc = 0.f;
                if (has0) acc = __uint_as_float(oa[k]) * w0[e];
                if (has1) acc += __uint_as_float(ob[k]) * w1[e];
                res[2 * jj + x] = acc;
              }
            if (complete) {
              const int t = r / p.group, hq = sg.g * p.group + (r - t * p.group);
              const size_t orow = ((size_t)lb * p.n_win + q0 + t) * p.n_q_heads + hq;
              __nv_bfloat16* dst = p.out + orow * D + cc * 64 + lc;
#pragma unroll
              for (int jj = 0; jj < 8; ++jj)
                *reinterpret_cast<uint32_t*>(dst + jj * 8) = pack_bf16x2(res[2 * jj], res[2 * jj + 1]);
              if (p.lse && cc == 0 && (lane & 3) == 0) p.lse[orow] = lse2[e] * kLn2;
            } else {
              float* dst = p.ws_o + ((size_t)slot * p.rows + r) * D + cc * 64 + lc;
#pragma unroll
              for (int jj = 0; jj < 8; ++jj)
                *reinterpret_cast<float2*>(dst + jj * 8) = make_float2(res[2 * jj], res[2 * jj + 1]);
              if (cc == 0 && (lane & 3) == 0) p.ws_lse[(size_t)slot * p.rows + r] = lse2[e];
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_o_empty);

      if (!complete) {
        // the CTA that brings an item's last partial result merges all of them, in slice order
        __threadfence();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_ep_done);
        const int64_t item_end = sg.item_begin + sg.item_tiles;
        const int c_first = slice_owner(sg.item_begin, n_active, total);
        const int c_last = slice_owner(item_end - 1, n_active, total);
        if (st == 0) {
          if (mbar_wait(bar_ep_done, n_partial & 1, abort_flag)) {
            const int old = atomicAdd(p.ws_cnt + (size_t)part * n_items + sg.item, 1);
            __threadfence();
            *last_flag = (old == c_last - c_first) ? 1 : 0;
          } else {
            *last_flag = 0;
          }
          mbar_arrive(bar_ep_flag);
        }
        SM_WAIT(bar_ep_flag, n_partial & 1);
        ++n_partial;
        if (*last_flag) {
          __threadfence();
          // Two output positions per thread and pass, the parts in chunks of kMergeChunk: every
          // load of a chunk is issued before the first is used, so a pass costs one trip to the L2
          // instead of one per part and value.  Parts are folded in slice order (fixed).
          constexpr int kMergeChunk = 4;
          const int n_parts = c_last - c_first + 1;
          const int n_idx = rows * (D / 4);
          for (int idx0 = st; idx0 < n_idx; idx0 += 512) {
            int r[2], c4[2];
            bool on[2];
            float mm[2] = {-INFINITY, -INFINITY}, den[2] = {0.f, 0.f};
            float4 acc[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const int idx = idx0 + 256 * u;
              on[u] = idx < n_idx;
              r[u] = on[u] ? idx / (D / 4) : 0;
              c4[u] = on[u] ? idx - r[u] * (D / 4) : 0;
            }
            for (int pc = 0; pc < n_parts; pc += kMergeChunk) {
              float ls[2][kMergeChunk];
              float4 x[2][kMergeChunk];
#pragma unroll
              for (int q = 0; q < kMergeChunk; ++q) {
                const bool have = pc + q < n_parts;
                const int cpart = c_first + pc + q;
                const int sl = have ? partial_slot(part * ctas_per_part + cpart, slice_begin(cpart, n_active, total), sg.item_begin) : 0;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                  if (have && on[u]) {
                    ls[u][q] = ldg_cg_f32(p.ws_lse + (size_t)sl * p.rows + r[u]);
                    x[u][q] = ldg_cg_f32x4(p.ws_o + ((size_t)sl * p.rows + r[u]) * D + c4[u] * 4);
                  } else {
                    ls[u][q] = -INFINITY;
                    x[u][q] = make_float4(0.f, 0.f, 0.f, 0.f);
                  }
                }
              }
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                float m2 = mm[u];
#pragma unroll
                for (int q = 0; q < kMergeChunk; ++q) m2 = fmaxf(m2, ls[u][q]);
                if (m2 == -INFINITY) continue;
                const float sc = mm[u] == -INFINITY ? 0.f : fast_exp2(mm[u] - m2);
                acc[u].x *= sc;
                acc[u].y *= sc;
                acc[u].z *= sc;
                acc[u].w *= sc;
                den[u] *= sc;
#pragma unroll
                for (int q = 0; q < kMergeChunk; ++q) {
                  const float w = ls[u][q] == -INFINITY ? 0.f : fast_exp2(ls[u][q] - m2);
                  acc[u].x += w * x[u][q].x;
                  acc[u].y += w * x[u][q].y;
                  acc[u].z += w * x[u][q].z;
                  acc[u].w += w * x[u][q].w;
                  den[u] += w;
                }
                mm[u] = m2;
              }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              if (!on[u]) continue;
              const float invd = den[u] > 0.f ? 1.f / den[u] : 0.f;
              const int t = r[u] / p.group, hq = sg.g * p.group + (r[u] - t * p.group);
              const size_t orow = ((size_t)lb * p.n_win + q0 + t) * p.n_q_heads + hq;
              uint2 packed;
              packed.x = pack_bf16x2(acc[u].x * invd, acc[u].y * invd);
              packed.y = pack_bf16x2(acc[u].z * invd, acc[u].w * invd);
              *reinterpret_cast<uint2*>(p.out + orow * D + c4[u] * 4) = packed;
              if (p.lse && c4[u] == 0) p.lse[orow] = den[u] > 0.f ? (mm[u] + log2f(den[u])) * kLn2 : -INFINITY;
            }
          }
        }
      }
      i0 += sg.n_tiles;
      c.next_segment(prefix, p.batch, hkv);
    }
  softmax_done:
    if (!ok && p.d_status && gt == 0) *p.d_status = SPECVLM_ERR_TIMEOUT;
#undef SM_WAIT
  }

  // every role ends here; the allocating warp returns the tensor memory
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// How a window of `rows` rows is cut: n_parts parts of q_per query tokens (at most 128 rows each).
static void tc_parts(int rows, int group, int& n_parts, int& q_per) {
  const int n_q = rows / group;
  const int q_max = 128 / group;                       // whole query tokens that fit the 128 rows of a part
  n_parts = (n_q + q_max - 1) / q_max;
  q_per = (n_q + n_parts - 1) / n_parts;               // the parts are made as equal as the tokens allow
}

// One set of CTAs per part, every set as large as the SMs allow (and the tile count is worth).
static int tc_grid(const specvlm_kv_t* kv, int32_t batch, int n_parts) {
  const int64_t tiles_max = (int64_t)kv->n_layers * batch * kv->n_kv_heads *
                            ((kv->max_seq_len + kBigTokens - 1) / kBigTokens);
  int per_part = sm_count() / n_parts;
  if (per_part < 1) per_part = 1;
  return n_parts * sched_active_ctas(tiles_max, per_part);
}

// scratch: two partial results per CTA (rows of a full part each), their LSEs, one arrival counter
// per (part, item)
static void tc_ws_layout(const specvlm_kv_t* kv, int32_t batch, int rows, int group, size_t& o_bytes, size_t& lse_bytes,
                         size_t& cnt_bytes) {
  int n_parts, q_per;
  tc_parts(rows, group, n_parts, q_per);
  const int grid = tc_grid(kv, batch, n_parts);
  const size_t items = (size_t)kv->n_layers * batch * kv->n_kv_heads;
  const size_t rows_part = (size_t)q_per * group;
  o_bytes = round_up((size_t)2 * grid * rows_part * kv->head_dim * sizeof(float), 256);
  lse_bytes = round_up((size_t)2 * grid * rows_part * sizeof(float), 256);
  cnt_bytes = round_up(items * n_parts * sizeof(int32_t), 256);
}

size_t attn_tc_ws_bytes(const specvlm_kv_t* kv, int32_t batch, int rows, int group) {
  size_t a, b, c;
  tc_ws_layout(kv, batch, rows, group, a, b, c);
  return a + b + c;
}

// Queries as a 5-D tensor (channel, head in group, query token, KV head, layer * batch + sequence):
// the box (64 channels, group, n_q, 1, 1) at token q0 is one item's rows of a launch, r = t * group + head.
static int32_t encode_q_map(CUtensorMap* map, const void* q, int D, int group, int n_win, int n_q, int n_kv_heads,
                            int64_t lb) {
  encode_tiled_fn enc = get_encode_tiled();
  if (!enc) return SPECVLM_ERR_CUDA;
  const int hq = group * n_kv_heads;
  const cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)group, (cuuint64_t)n_win, (cuuint64_t)n_kv_heads, (cuuint64_t)lb};
  const cuuint64_t strides[4] = {(cuuint64_t)D * 2, (cuuint64_t)hq * D * 2, (cuuint64_t)group * D * 2,
                                 (cuuint64_t)n_win * hq * D * 2};
  const cuuint32_t box[5] = {64u, (cuuint32_t)group, (cuuint32_t)n_q, 1u, 1u};
  const cuuint32_t estr[5] = {1u, 1u, 1u, 1u, 1u};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(q), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPECVLM_OK : SPECVLM_ERR_CUDA;
}

template <int D, int M, bool TREE>
static int32_t launch_tc_t(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const AttnTcParams& p,
                         int grid, cudaStream_t st) {
  using C = TcCfg<D, M>;
  auto kern = attn_tc_kernel<D, M, TREE>;
  // once per device and kernel variant: the opt-in shared-memory size, and the check that the
  // compiled kernel's register pool can satisfy the setmaxnreg requests (it never changes)
  static std::atomic<uint64_t> attr_done{0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SPECVLM_ERR_CUDA;
  if (!(attr_done.load(std::memory_order_acquire) & (1ull << (dev & 63)))) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return SPECVLM_ERR_CUDA;
    if (fa.numRegs * kTcThreads < kRegsNeeded) return SPECVLM_ERR_CUDA;   // setmaxnreg could never be satisfied
    if (!smem_attr_once(attr_done, reinterpret_cast<const void*>(kern), C::TOTAL)) return SPECVLM_ERR_CUDA;
  }
  kern<<<grid, kTcThreads, C::TOTAL, st>>>(tk, tv, tq, p);
  return launch_status();
}

// Ancestor masks of a draft tree: bit w of anc[b][t] says that node t attends window position w
// (itself and the nodes on its path to a root).  parents[b][t] < t, -1 for a root.
__global__ void tree_ancestors_kernel(const int32_t* __restrict__ parents, int n, int n_nodes,
                                      uint64_t* __restrict__ anc, int32_t* d_status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int t = i % n_nodes;
  const int32_t* par = parents + (i - t);
  uint64_t a = 1ull << t;
  int cur = t;
  for (int step = 0; step < n_nodes; ++step) {
    const int pp = par[cur];
    if (pp < 0) break;
    if (pp >= cur) {                      // not a tree in topological order: the node sees itself only
      if (d_status) *d_status = SPECVLM_ERR_INVALID_ARG;
      a = 1ull << t;
      break;
    }
    a |= 1ull << pp;
    cur = pp;
  }
  anc[i] = a;
}

size_t attn_tc_tree_extra_bytes(int32_t batch, int32_t n_nodes) {
  return round_up((size_t)batch * n_nodes * sizeof(uint64_t), 256);
}

template <int D, int M>
static int32_t launch_tc(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const AttnTcParams& p,
                         int grid, cudaStream_t st) {
  return p.anc ? launch_tc_t<D, M, true>(tk, tv, tq, p, grid, st) : launch_tc_t<D, M, false>(tk, tv, tq, p, grid, st);
}

int32_t attn_tc_launch(const specvlm_kv_t* kv, const void* q, int32_t batch, int32_t n_q_heads, int32_t n_q,
                       float sm_scale, void* out, float* lse, void* ws, size_t ws_bytes, int32_t* d_status,
                       cudaStream_t st, const int32_t* tree_parents) {
  const int group = n_q_heads / kv->n_kv_heads;
  const int rows = group * n_q;
  if (group > 16 || batch > kSchedMaxBatch) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  const int64_t items = (int64_t)kv->n_layers * batch * kv->n_kv_heads;
  if (items > 0x3fffffff) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return SPECVLM_ERR_INVALID_ARG;
  size_t o_bytes, lse_bytes, cnt_bytes;
  tc_ws_layout(kv, batch, rows, group, o_bytes, lse_bytes, cnt_bytes);
  const size_t base_bytes = o_bytes + lse_bytes + cnt_bytes;
  if (ws_bytes < base_bytes + (tree_parents ? attn_tc_tree_extra_bytes(batch, n_q) : 0))
    return SPECVLM_ERR_WORKSPACE_TOO_SMALL;
  if (tree_parents && n_q > kMaxTreeNodes) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  // A window of more than 128 rows is cut into parts of equal numbers of query tokens (the
  // accumulators of one part fill the tensor memory); the parts share one launch (see the kernel).
  int n_parts, q_per;
  tc_parts(rows, group, n_parts, q_per);
  if (q_per * group > 128) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  const int grid = tc_grid(kv, batch, n_parts);

  CUtensorMap tk, tv;
  int32_t rc = encode_kv_map(&tk, kv, kv->k, kTileTokens);
  if (rc != SPECVLM_OK) return rc;
  rc = encode_kv_map(&tv, kv, kv->v, kTileTokens);
  if (rc != SPECVLM_OK) return rc;

  AttnTcParams p;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  uint8_t* w = static_cast<uint8_t*>(ws);
  p.ws_o = reinterpret_cast<float*>(w);
  p.ws_lse = reinterpret_cast<float*>(w + o_bytes);
  p.ws_cnt = reinterpret_cast<int32_t*>(w + o_bytes + lse_bytes);
  p.n_parts = n_parts;
  p.q_per = q_per;
  p.rows = q_per * group;
  p.block_table = kv->block_table;
  p.seq_lens = kv->seq_lens;
  p.d_status = d_status;
  p.batch = batch;
  p.n_layers = kv->n_layers;
  p.n_win = n_q;
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = kv->n_kv_heads;
  p.group = group;
  p.max_blocks = kv->max_blocks;
  p.block_tokens = kv->block_tokens;
  p.max_seq_len = kv->max_seq_len;
  p.scale_log2 = sm_scale * kLog2e;
  p.anc = nullptr;
  if (tree_parents) {
    uint64_t* anc = reinterpret_cast<uint64_t*>(static_cast<uint8_t*>(ws) + base_bytes);
    const int n = batch * n_q;
    tree_ancestors_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(tree_parents, n, n_q, anc, d_status);
    rc = launch_status();
    if (rc != SPECVLM_OK) return rc;
    p.anc = anc;
  }

  CUtensorMap tq;
  rc = encode_q_map(&tq, q, kv->head_dim, group, n_q, q_per, kv->n_kv_heads, (int64_t)kv->n_layers * batch);
  if (rc != SPECVLM_OK) return rc;
  if (cudaMemsetAsync(p.ws_cnt, 0, (size_t)items * n_parts * sizeof(int32_t), st) != cudaSuccess) return SPECVLM_ERR_CUDA;
  if (kv->head_dim == 128)
    rc = p.rows <= 64 ? launch_tc<128, 64>(tk, tv, tq, p, grid, st) : launch_tc<128, 128>(tk, tv, tq, p, grid, st);
  else
    rc = p.rows <= 64 ? launch_tc<64, 64>(tk, tv, tq, p, grid, st) : launch_tc<64, 128>(tk, tv, tq, p, grid, st);
  if (rc != SPECVLM_OK) return rc;
  return SPECVLM_OK;
}

}  // namespace specvlm

// Host-only: how a verification window of n_q query tokens at `group` heads per KV head is cut into
// parts (see tc_parts); lets a CPU test sweep the rule.
extern "C" int32_t specvlm_debug_window_parts(int32_t n_q, int32_t group, int32_t* n_parts, int32_t* q_per) {
  if (n_q < 1 || group < 1 || group > 16 || !n_parts || !q_per) return SPECVLM_ERR_INVALID_ARG;
  int a, b;
  specvlm::tc_parts(n_q * group, group, a, b);
  *n_parts = a;
  *q_per = b;
  return SPECVLM_OK;
}
