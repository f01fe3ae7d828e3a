// Steps 1b + 2: Stage I top-k retention and Stage II spatially uniform reduction, one CTA per
// sequence with the whole fp32 score vector resident in shared memory.
//   1. radix select (4 passes of 8 bits, most significant first) finds the k1-th largest key T
//      and how many keys equal to T belong to the top-k1;
//   2. ordered block scans give (a) the rank of each key equal to T among its equals, so ties go
//      to the lower index, (b) the rank of each unselected token among the unselected ones,
//      hence its rank inside its frame, (c) the output position of each kept token;
//   3. the Stage-II pick test is integer arithmetic per token.
// Everything is deterministic: no atomics decide an output.
//
// Top-P mode (Eq. 6): the Stage-I count is the shortest prefix of the ranking whose cumulative
// score reaches lambda_r of the total.  The same radix descent runs on score mass instead of
// counts.  Masses are the scores truncated to multiples of 2^-36 (capped at 1) and summed as
// 64-bit integers, lambda_r is in thousandths: integer sums do not depend on the order of the
// additions, so the count is a function of the scores alone.
#include "common.cuh"
#include "host_util.h"

namespace specvlm {

constexpr int kSelThreads = 1024;
constexpr int kSelMaxBatch = 64;
constexpr int kTopPFracBits = 36;

// score mass of a key (keys of non-negative floats are their bits with the top bit set)
__device__ __forceinline__ unsigned long long key_mass(uint32_t key) {
  const double a = (double)__uint_as_float(key & 0x7fffffffu) * (double)(1ull << kTopPFracBits);
  const unsigned long long one = 1ull << kTopPFracBits;
  return a >= (double)one ? one : (unsigned long long)a;
}

struct SelSeq {
  int32_t score_off, n_frames, k1, k_total, kept_off;
  int32_t lambda_pm;                   // >= 0: Top-P mode, k1 is computed; < 0: k1 as given
  int32_t seq_index;                   // position in the batch (random selector's counter word)
};

// Philox-4x32, 10 rounds (Salmon et al., SC'11), first output word: the counter-based generator
// of the random selector
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1) {
  uint32_t c2 = 0u, c3 = 0u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0;
}
struct SelParams {
  const float* scores;
  int32_t* kept_idx;
  int32_t* k1_out;                     // [batch] Stage-I counts or null
  int32_t tokens_per_frame;
  int32_t k1_out_base;                 // index of seq[0] in k1_out
  int32_t random_keys;                 // 1: rank Philox keys instead of scores
  uint32_t seed_lo, seed_hi;
  SelSeq seq[kSelMaxBatch];
};

// exclusive prefix sum over the block of one int per thread; returns the exclusive prefix and
// stores the block total in *total.  warp_sums: 32 ints of shared memory.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += n;
  }
  __syncthreads();                     // warp_sums may still be read from a previous scan
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int ws = warp_sums[lane];
    int wi = ws;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += n;
    }
    warp_sums[lane] = wi - ws;         // exclusive prefix of the warp totals
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  return warp_sums[warp] + incl - v;
}

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const __grid_constant__ SelParams p) {
  extern __shared__ uint32_t sel_smem[];
  const SelSeq sq = p.seq[blockIdx.x];
  const int T = p.tokens_per_frame, F = sq.n_frames, n_v = F * T;
  int k1 = sq.k1;
  const int k_total = sq.k_total;
  uint32_t* const key = sel_smem;                                  // [n_v] keys, later states
  int* const cf = reinterpret_cast<int*>(sel_smem + n_v);         // [F + 1] unselected before frame f
  int* const hist = cf + F + 1;                                    // [256]
  int* const warp_sums = hist + 256;                               // [32]
  int* const misc = warp_sums + 32;                                // [8]
  unsigned long long* const mass = reinterpret_cast<unsigned long long*>(                // [256 + 2]
      (reinterpret_cast<uintptr_t>(misc + 8) + 7) & ~static_cast<uintptr_t>(7));
  const int tid = threadIdx.x;

  // order-preserving map float -> uint32 (larger float <=> larger key)
  if (p.random_keys) {
    // random selector: the key of token j is the top 24 bits of a Philox word, as an fp32 value
    for (int j = tid; j < n_v; j += kSelThreads) {
      const float r = (float)(philox4x32_10_word0((uint32_t)j, (uint32_t)sq.seq_index, p.seed_lo, p.seed_hi) >> 8);
      key[j] = __float_as_uint(r) | 0x80000000u;
    }
  } else {
    const float* sc = p.scores + sq.score_off;
    for (int j = tid; j < n_v; j += kSelThreads) {
      const uint32_t u = __float_as_uint(sc[j]);
      key[j] = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
  }

  // ---- 0. Top-P: the Stage-I count from the score mass
  if (sq.lambda_pm >= 0) {
    __syncthreads();
    if (tid == 0) mass[256] = 0ull;
    __syncthreads();
    {
      unsigned long long part = 0ull;
      for (int j = tid; j < n_v; j += kSelThreads) part += key_mass(key[j]);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
      if ((tid & 31) == 0) atomicAdd(&mass[256], part);            // integer: order-independent
    }
    __syncthreads();
    const unsigned long long target = (unsigned long long)sq.lambda_pm * mass[256];   // vs 1000 * prefix mass
    int c = 0;
    if (target > 0ull) {
      uint32_t pfx = 0, pfx_mask = 0;
      unsigned long long above = 0ull;     // mass of the keys ranked before every key matching pfx
      int n_above = 0;
      for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += kSelThreads) {
          hist[i] = 0;
          mass[i] = 0ull;
        }
        __syncthreads();
        for (int j = tid; j < n_v; j += kSelThreads) {
          if ((key[j] & pfx_mask) == pfx) {
            const uint32_t digit = (key[j] >> shift) & 255u;
            atomicAdd(&hist[digit], 1);
            atomicAdd(&mass[digit], key_mass(key[j]));
          }
        }
        __syncthreads();
        // Scanning the digits from 255 down, the first one whose keys bring the mass up to the target
        // (digit 0 if none does).  Warp 0 does it: lane l owns digits 8l .. 8l+7, a shuffle scan
        // gives the mass and the count above each lane's digits, and the one lane whose digits
        // contain the crossing walks its eight.
        if (tid < 32) {
          unsigned long long hm[8], sm = 0ull;
          int hc[8], sc = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            hm[i] = mass[8 * tid + i];
            hc[i] = hist[8 * tid + i];
            sm += hm[i];
            sc += hc[i];
          }
          unsigned long long am = sm;
          int ac = sc;
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long vm = __shfl_down_sync(0xffffffffu, am, off);
            const int vc = __shfl_down_sync(0xffffffffu, ac, off);
            if (tid + off < 32) {
              am += vm;
              ac += vc;
            }
          }
          unsigned long long acc = above + (am - sm);      // mass of the live keys with larger digits
          int n = n_above + (ac - sc);
          const bool crosses = 1000ull * acc < target && 1000ull * (acc + sm) >= target;
          const unsigned any = __ballot_sync(0xffffffffu, crosses);
          if (crosses || (any == 0u && tid == 0)) {
            int d = 8 * tid + 7;
#pragma unroll
            for (int i = 7; i >= 0; --i, --d) {
              if (d == 0 || 1000ull * (acc + hm[i]) >= target) break;
              acc += hm[i];
              n += hc[i];
            }
            misc[0] = d;
            misc[1] = n;
            mass[257] = acc;
          }
        }
        __syncthreads();
        pfx |= static_cast<uint32_t>(misc[0]) << shift;
        pfx_mask |= 255u << shift;
        n_above = misc[1];
        above = mass[257];
        __syncthreads();
      }
      // every key equal to pfx carries the same mass: take as many as still needed
      const unsigned long long q = key_mass(pfx);
      const unsigned long long need = target - 1000ull * above;      // > 0: `above` alone does not reach
      const unsigned long long e = q > 0ull ? (need + 1000ull * q - 1ull) / (1000ull * q) : 0ull;
      c = n_above + (int)e;
    }
    k1 = c < k_total ? c : k_total;
    if (tid == 0 && p.k1_out) p.k1_out[blockIdx.x + p.k1_out_base] = k1;
  }

  // ---- 1. radix select of the k1-th largest key
  uint32_t prefix = 0, prefix_mask = 0;
  int k_rem = k1;                      // how many of the keys matching `prefix` are still wanted
  if (k1 > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = tid; i < 256; i += kSelThreads) hist[i] = 0;
      __syncthreads();
      for (int j0 = 0; j0 < n_v; j0 += kSelThreads) {
        const int j = j0 + tid;
        const bool live = j < n_v && (key[j] & prefix_mask) == prefix;
        const uint32_t digit = live ? (key[j] >> shift) & 255u : 256u;
        // one shared-memory atomic per distinct digit in the warp
        const uint32_t peers = __match_any_sync(0xffffffffu, digit);
        if (live && (tid & 31) == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
      }
      __syncthreads();
      // Scanning the digits from 255 down, the first one that brings the count up to k_rem (digit 0
      // if none does): warp 0, lane l owning digits 8l .. 8l+7, as in the Top-P descent above.
      if (tid < 32) {
        int hc[8], sc = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          hc[i] = hist[8 * tid + i];
          sc += hc[i];
        }
        int ac = sc;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int vc = __shfl_down_sync(0xffffffffu, ac, off);
          if (tid + off < 32) ac += vc;
        }
        int acc = ac - sc;             // live keys with larger digits
        const bool crosses = acc < k_rem && acc + sc >= k_rem;
        const unsigned any = __ballot_sync(0xffffffffu, crosses);
        if (crosses || (any == 0u && tid == 0)) {
          int d = 8 * tid + 7;
#pragma unroll
          for (int i = 7; i >= 0; --i, --d) {
            if (d == 0 || acc + hc[i] >= k_rem) break;
            acc += hc[i];
          }
          misc[0] = d;                 // digit of the k_rem-th largest live key
          misc[1] = k_rem - acc;       // wanted among the keys with that digit
        }
      }
      __syncthreads();
      prefix |= static_cast<uint32_t>(misc[0]) << shift;
      prefix_mask |= 255u << shift;
      k_rem = misc[1];
      __syncthreads();
    }
  }
  const uint32_t thr = prefix;         // key of the k1-th largest element (when k1 > 0)

  // ---- 2a. ties: keys equal to thr are taken in index order until k_rem are taken
  // each thread owns a contiguous run of tokens so that block scans are ordered by index
  int per = (n_v + kSelThreads - 1) / kSelThreads;
  per |= 1;                            // odd run length: conflict-free strided shared-memory access
  const int j_lo = min(tid * per, n_v), j_hi = min(j_lo + per, n_v);
  int n_eq = 0;
  if (k1 > 0)
    for (int j = j_lo; j < j_hi; ++j) n_eq += key[j] == thr;
  int eq_rank = block_exclusive_scan(n_eq, warp_sums, &misc[2]);
  // states: 0 = dropped so far, 1 = in V_R
  int n_unsel = 0;
  for (int j = j_lo; j < j_hi; ++j) {
    const uint32_t kj = key[j];
    bool sel = false;
    if (k1 > 0) {
      if (kj > thr) sel = true;
      else if (kj == thr) sel = eq_rank++ < k_rem;
    }
    key[j] = sel ? 1u : 0u;
    n_unsel += !sel;
  }
  // ---- 2b. rank among the unselected tokens; unselected count before each frame
  int m_total;
  int e = block_exclusive_scan(n_unsel, warp_sums, &misc[3]);
  m_total = misc[3];
  {
    int run = e;
    for (int j = j_lo; j < j_hi; ++j) {
      if (j % T == 0) cf[j / T] = run;
      run += key[j] == 0u;
    }
    if (tid == 0) cf[F] = m_total;
  }
  __syncthreads();
  // ---- 3. Stage II pick test, then compaction
  // All products below stay under 2^32: counts are at most n_v <= 57 344 tokens (the shared-memory
  // limit), so 32-bit unsigned division is exact here -- and keeps this kernel's code small.
  const uint32_t n_u = (uint32_t)(k_total - k1);
  int n_keep = 0;
  {
    int run = e;
    for (int j = j_lo; j < j_hi; ++j) {
      if (key[j] == 0u) {
        const int f = j / T;
        const uint32_t c0 = (uint32_t)cf[f], c1 = (uint32_t)cf[f + 1];
        const uint32_t c_f = c1 - c0;
        const uint32_t rank = (uint32_t)run - c0;
        const uint32_t n_f = (c1 * n_u) / (uint32_t)m_total - (c0 * n_u) / (uint32_t)m_total;
        if (n_f > 0u) {
          const uint32_t t = (rank * n_f + c_f - 1u) / c_f;
          if (t < n_f && (t * c_f) / n_f == rank) key[j] = 2u;
        }
        ++run;
      }
      n_keep += key[j] != 0u;
    }
  }
  int pos = block_exclusive_scan(n_keep, warp_sums, &misc[4]);
  int32_t* out = p.kept_idx + sq.kept_off;
  for (int j = j_lo; j < j_hi; ++j)
    if (key[j] != 0u) out[pos++] = j;
}

// window / frame selectors: closed-form index lists, one CTA per sequence
struct RangeParams {
  int32_t* kept_idx;
  int32_t* kept_n_out;
  int32_t mode, tokens_per_frame, batch0;
  int32_t n_frames[kSelMaxBatch], k_total[kSelMaxBatch], kept_off[kSelMaxBatch];
};

__global__ void baseline_ranges_kernel(const __grid_constant__ RangeParams p) {
  const int i = blockIdx.x;
  const int F = p.n_frames[i], T = p.tokens_per_frame, K = p.k_total[i], n_v = F * T;
  int32_t* out = p.kept_idx + p.kept_off[i];
  int n = K;
  if (p.mode == SPECVLM_SEL_FRAMES) {
    const int nf = K / T;                       // whole frames that fit the budget
    n = nf * T;
    for (int j = threadIdx.x; j < n; j += blockDim.x) {
      const int fi = j / T;
      out[j] = (int)(((long long)fi * F) / nf) * T + (j - fi * T);
    }
  } else {
    const int start = p.mode == SPECVLM_SEL_WINDOW_FRONT ? 0 : (p.mode == SPECVLM_SEL_WINDOW_END ? n_v - K : (n_v - K) / 2);
    for (int j = threadIdx.x; j < n; j += blockDim.x) out[j] = start + j;
  }
  if (threadIdx.x == 0 && p.kept_n_out) p.kept_n_out[p.batch0 + i] = n;
}

static int32_t select_common(const float* scores, const int32_t* video_cu, const int32_t* n_frames,
                             int32_t tokens_per_frame, const int32_t* k_stage1, const int32_t* lambda_permille,
                             const int32_t* k_total, const int32_t* kept_cu, int32_t batch, int32_t* kept_idx,
                             int32_t* k1_out, void* stream, bool random_keys = false, uint64_t seed = 0) {
  if ((!scores && !random_keys) || !video_cu || !n_frames || (!k_stage1 && !lambda_permille) || !k_total || !kept_cu || !kept_idx ||
      batch < 1 || tokens_per_frame < 1)
    return SPECVLM_ERR_INVALID_ARG;
  size_t max_smem = 0;
  for (int b = 0; b < batch; ++b) {
    const int64_t n_v = (int64_t)n_frames[b] * tokens_per_frame;
    if (n_frames[b] < 1 || n_frames[b] > 1024 || n_v > 57344) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
    if (k_total[b] < 0 || k_total[b] > n_v) return SPECVLM_ERR_INVALID_ARG;
    if (lambda_permille) {
      if (lambda_permille[b] < 0 || lambda_permille[b] > 1000) return SPECVLM_ERR_INVALID_ARG;
    } else if (k_stage1[b] < 0 || k_stage1[b] > k_total[b]) {
      return SPECVLM_ERR_INVALID_ARG;
    }
    if ((!random_keys && video_cu[b + 1] - video_cu[b] < n_v) || kept_cu[b + 1] - kept_cu[b] < k_total[b])
      return SPECVLM_ERR_INVALID_ARG;
    // keys, per-frame counts, histogram, scan scratch, flags, then the 64-bit mass bins (8-byte aligned)
    const size_t words = (size_t)n_v + n_frames[b] + 1 + 256 + 32 + 8;
    const size_t sm = (words + (words & 1)) * 4 + (256 + 2) * 8;
    if (sm > max_smem) max_smem = sm;
  }
  if (max_smem > 232448) return SPECVLM_ERR_UNSUPPORTED_SHAPE;
  // the kernel may use up to a whole SM's shared memory; how much a launch gets is the launch's own figure
  static std::atomic<uint64_t> attr_done{0};
  if (!smem_attr_once(attr_done, reinterpret_cast<const void*>(select_kernel), 232448)) return SPECVLM_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SelParams p;
  p.scores = scores;
  p.kept_idx = kept_idx;
  p.k1_out = k1_out;
  p.tokens_per_frame = tokens_per_frame;
  p.random_keys = random_keys ? 1 : 0;
  p.seed_lo = (uint32_t)(seed & 0xffffffffu);
  p.seed_hi = (uint32_t)(seed >> 32);
  for (int b0 = 0; b0 < batch; b0 += kSelMaxBatch) {
    const int nb = batch - b0 < kSelMaxBatch ? batch - b0 : kSelMaxBatch;
    p.k1_out_base = b0;
    for (int i = 0; i < nb; ++i) {
      const int b = b0 + i;
      p.seq[i] = SelSeq{video_cu[b], n_frames[b], lambda_permille ? 0 : k_stage1[b], k_total[b], kept_cu[b],
                        lambda_permille ? lambda_permille[b] : -1, b};
    }
    select_kernel<<<(unsigned)nb, kSelThreads, max_smem, st>>>(p);
    const int32_t rc = launch_status();
    if (rc != SPECVLM_OK) return rc;
  }
  return SPECVLM_OK;
}

}  // namespace specvlm

using namespace specvlm;

extern "C" int32_t specvlm_select(const float* scores, const int32_t* video_cu, const int32_t* n_frames,
                                  int32_t tokens_per_frame, const int32_t* k_stage1,
                                  const int32_t* k_total, const int32_t* kept_cu, int32_t batch,
                                  int32_t* kept_idx, int32_t* d_status, void* stream) {
  NvtxRange nvtx_range(__func__);
  (void)d_status;
  if (!k_stage1) return SPECVLM_ERR_INVALID_ARG;
  return select_common(scores, video_cu, n_frames, tokens_per_frame, k_stage1, nullptr, k_total, kept_cu, batch,
                       kept_idx, nullptr, stream);
}

extern "C" int32_t specvlm_select_top_p(const float* scores, const int32_t* video_cu, const int32_t* n_frames,
                                        int32_t tokens_per_frame, const int32_t* lambda_permille,
                                        const int32_t* k_total, const int32_t* kept_cu, int32_t batch,
                                        int32_t* kept_idx, int32_t* k_stage1_out_or_null, int32_t* d_status,
                                        void* stream) {
  NvtxRange nvtx_range(__func__);
  (void)d_status;
  if (!lambda_permille) return SPECVLM_ERR_INVALID_ARG;
  return select_common(scores, video_cu, n_frames, tokens_per_frame, nullptr, lambda_permille, k_total, kept_cu,
                       batch, kept_idx, k_stage1_out_or_null, stream);
}

extern "C" int32_t specvlm_select_baseline(int32_t mode, uint64_t seed, const int32_t* n_frames,
                                           int32_t tokens_per_frame, const int32_t* k_total,
                                           const int32_t* kept_cu, int32_t batch, int32_t* kept_idx,
                                           int32_t* kept_n_out_or_null, void* stream) {
  NvtxRange nvtx_range(__func__);
  if (!n_frames || !k_total || !kept_cu || !kept_idx || batch < 1 || tokens_per_frame < 1)
    return SPECVLM_ERR_INVALID_ARG;
  if (mode < SPECVLM_SEL_WINDOW_FRONT || mode > SPECVLM_SEL_RANDOM) return SPECVLM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (mode == SPECVLM_SEL_RANDOM) {
    // the k_total largest Philox keys: the selection kernel with keys in place of scores and
    // Stage I taking the whole budget
    int32_t rc = select_common(nullptr, kept_cu /*unused*/, n_frames, tokens_per_frame, k_total, nullptr, k_total,
                               kept_cu, batch, kept_idx, nullptr, stream, true, seed);
    if (rc != SPECVLM_OK || !kept_n_out_or_null) return rc;
    return cudaMemcpyAsync(kept_n_out_or_null, k_total, (size_t)batch * sizeof(int32_t), cudaMemcpyHostToDevice, st) ==
                   cudaSuccess
               ? SPECVLM_OK
               : SPECVLM_ERR_CUDA;
  }
  RangeParams p;
  p.kept_idx = kept_idx;
  p.kept_n_out = kept_n_out_or_null;
  p.mode = mode;
  p.tokens_per_frame = tokens_per_frame;
  for (int b0 = 0; b0 < batch; b0 += kSelMaxBatch) {
    const int nb = batch - b0 < kSelMaxBatch ? batch - b0 : kSelMaxBatch;
    p.batch0 = b0;
    for (int i = 0; i < nb; ++i) {
      const int b = b0 + i;
      const int64_t n_v = (int64_t)n_frames[b] * tokens_per_frame;
      if (n_frames[b] < 1 || n_v > 0x7fffffff || k_total[b] < 0 || k_total[b] > n_v ||
          kept_cu[b + 1] - kept_cu[b] < k_total[b])
        return SPECVLM_ERR_INVALID_ARG;
      p.n_frames[i] = n_frames[b];
      p.k_total[i] = k_total[b];
      p.kept_off[i] = kept_cu[b];
    }
    baseline_ranges_kernel<<<(unsigned)nb, 256, 0, st>>>(p);
    const int32_t rc = launch_status();
    if (rc != SPECVLM_OK) return rc;
  }
  return SPECVLM_OK;
}
