/*
 * CPU oracle for the SpecVLM pruned-draft speculative-decoding hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what the
 * CUDA library must compute.  It shares no code, header, table or constant with the CUDA
 * path and must never be called from it; only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs execute it.
 *
 * Inputs are bf16 bit patterns (uint16_t); every value is widened exactly to double and
 * all arithmetic is fp64.  Layouts are plain contiguous arrays (the Python wrapper
 * de-pages paged caches before calling).
 *
 * Parity status of the readings taken where the paper is silent:
 *   - softmax domain of the guidance matrix G (Eq. 4): G is the language-row / video-column
 *     block of the FULL causal softmax matrix M.  parity unpinned against the authors' code
 *     (a switch computes the video-only renormalised variant for reporting).
 *   - everything else in this file (softmax attention rows) has textbook definitions and is
 *     pinned by closed forms and by a library fp64 attention in the tests.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_double(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* dot product of two bf16 rows of length d, in fp64, index order 0..d-1 */
static double dot_bf16(const uint16_t* a, const uint16_t* b, int d) {
  double s = 0.0;
  for (int c = 0; c < d; ++c) s += bf16_bits_to_double(a[c]) * bf16_bits_to_double(b[c]);
  return s;
}

/*
 * Token rating A = {a_j} (Eq. 4-5, Section 4.1).
 *
 * For every layer l, query head h (KV head g = h / (Hq/Hkv)) and language query i at absolute
 * position p_i = text_start + i, the attention row over the causal keys 0..p_i is
 *   M_{i,k} = exp(s_k - m) / sum_k' exp(s_k' - m),   s_k = sm_scale * <q_i, K_k>.
 * G_{i,j} = M_{i, video_start + j} for the video tokens j (Eq. 4); Eq. 5 averages G over the
 * language queries, and the sentence after Eq. 5 averages over all layers and heads:
 *   a_j = 1 / (n_layers * Hq * n_text) * sum_{l,h,i} G^{(l,h)}_{i,j}.
 *
 * video_only != 0 selects the alternative reading in which the softmax is taken over the
 * video keys alone (reported, never used for parity).
 *
 * q_text: [n_layers][n_text][Hq][d]     k: [n_layers][Hkv][n_tokens][d]
 * a: [n_video] fp64 out.  row_mass (optional): [n_layers][Hq][n_text] = sum_j G_{i,j}.
 * row_lse (optional): [n_layers][Hq][n_text] = m + log(sum exp(s - m)) of the full causal row.
 */
int oracle_stage1_scores(const uint16_t* q_text, const uint16_t* k, int n_layers, int Hq, int Hkv,
                         int d, int n_tokens, int video_start, int n_video, int text_start,
                         int n_text, double sm_scale, int video_only, double* a, double* row_mass,
                         double* row_lse) {
  if (Hq % Hkv != 0 || video_start < 0 || video_start + n_video > text_start ||
      text_start + n_text > n_tokens)
    return -1;
  const int group = Hq / Hkv;
  const long n_rows_lh = (long)n_layers * Hq;
  /* one accumulator per (layer, head) so the final reduction order is fixed */
  double* acc = (double*)calloc((size_t)n_rows_lh * (size_t)n_video, sizeof(double));
  if (!acc) return -2;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)n_tokens);
#pragma omp for schedule(dynamic, 1)
    for (long lh = 0; lh < n_rows_lh; ++lh) {
      const int l = (int)(lh / Hq), h = (int)(lh % Hq), g = h / group;
      const uint16_t* kbase = k + ((size_t)l * Hkv + g) * (size_t)n_tokens * d;
      double* accj = acc + (size_t)lh * n_video;
      for (int i = 0; i < n_text; ++i) {
        const uint16_t* qi = q_text + (((size_t)l * n_text + i) * Hq + h) * (size_t)d;
        const int p = text_start + i;         /* absolute position of the query */
        int k_lo = 0, k_hi = p;               /* causal key range [k_lo, k_hi]  */
        if (video_only) { k_lo = video_start; k_hi = video_start + n_video - 1; }
        double m = -INFINITY;
        for (int kk = k_lo; kk <= k_hi; ++kk) {
          s[kk] = sm_scale * dot_bf16(qi, kbase + (size_t)kk * d, d);
          if (s[kk] > m) m = s[kk];
        }
        double Z = 0.0;
        for (int kk = k_lo; kk <= k_hi; ++kk) Z += exp(s[kk] - m);
        double mass = 0.0;
        for (int j = 0; j < n_video; ++j) {
          const double g_ij = exp(s[video_start + j] - m) / Z;   /* G_{i,j}, Eq. 4 */
          accj[j] += g_ij;
          mass += g_ij;
        }
        if (row_mass) row_mass[(size_t)lh * n_text + i] = mass;
        if (row_lse) row_lse[(size_t)lh * n_text + i] = m + log(Z);
      }
    }
    free(s);
  }
  const double denom = (double)n_layers * (double)Hq * (double)n_text;
  for (int j = 0; j < n_video; ++j) {
    double t = 0.0;
    for (long lh = 0; lh < n_rows_lh; ++lh) t += acc[(size_t)lh * n_video + j];
    a[j] = t / denom;                                            /* Eq. 5 + layer/head mean */
  }
  free(acc);
  return 0;
}

/*
 * Softmax attention of n_q query tokens over one sequence's cache (Section 3.1: the draft's
 * decode step streams its whole KV cache; the target verifies gamma drafts in one pass).
 *
 *   o_{t,h} = sum_k softmax_k( sm_scale * <q_{t,h}, K_{g(h),k}> ) * V_{g(h),k}
 *
 * The cache already holds the keys/values of the n_q new tokens at its end.  Query t
 * (0-based) sees keys [0, kv_len - n_q + t]; with n_q == 1 this is plain decode attention
 * over all kv_len keys.  Two-pass softmax (max, then sum) in fp64.
 *
 * q: [n_q][Hq][d]   k, v: [Hkv][kv_stride][d] (kv_stride >= kv_len tokens per head)
 * out: [n_q][Hq][d] fp64   lse: [n_q][Hq] fp64 (optional)
 */
int oracle_attention(const uint16_t* q, const uint16_t* k, const uint16_t* v, int n_q, int Hq,
                     int Hkv, int d, int kv_len, int kv_stride, double sm_scale, double* out,
                     double* lse) {
  if (Hq % Hkv != 0 || n_q < 1 || kv_len < n_q || kv_stride < kv_len) return -1;
  const int group = Hq / Hkv;
#pragma omp parallel
  {
    double* p = (double*)malloc(sizeof(double) * (size_t)kv_len);
#pragma omp for schedule(dynamic, 1) collapse(2)
    for (int t = 0; t < n_q; ++t) {
      for (int h = 0; h < Hq; ++h) {
        const int g = h / group;
        const int n_keys = kv_len - n_q + t + 1;
        const uint16_t* qt = q + ((size_t)t * Hq + h) * (size_t)d;
        const uint16_t* kb = k + (size_t)g * kv_stride * d;
        const uint16_t* vb = v + (size_t)g * kv_stride * d;
        double m = -INFINITY;
        for (int kk = 0; kk < n_keys; ++kk) {
          p[kk] = sm_scale * dot_bf16(qt, kb + (size_t)kk * d, d);
          if (p[kk] > m) m = p[kk];
        }
        double Z = 0.0;
        for (int kk = 0; kk < n_keys; ++kk) { p[kk] = exp(p[kk] - m); Z += p[kk]; }
        double* o = out + ((size_t)t * Hq + h) * (size_t)d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int kk = 0; kk < n_keys; ++kk) {
          const double w = p[kk] / Z;
          const uint16_t* vr = vb + (size_t)kk * d;
          for (int c = 0; c < d; ++c) o[c] += w * bf16_bits_to_double(vr[c]);
        }
        if (lse) lse[(size_t)t * Hq + h] = m + log(Z);
      }
    }
    free(p);
  }
  return 0;
}

/* the softmax probabilities of one row, for tests of the "rows sum to 1" invariant */
int oracle_attention_probs(const uint16_t* q_row, const uint16_t* k_head, int d, int n_keys,
                           double sm_scale, double* probs) {
  double m = -INFINITY;
  for (int kk = 0; kk < n_keys; ++kk) {
    probs[kk] = sm_scale * dot_bf16(q_row, k_head + (size_t)kk * d, d);
    if (probs[kk] > m) m = probs[kk];
  }
  double Z = 0.0;
  for (int kk = 0; kk < n_keys; ++kk) { probs[kk] = exp(probs[kk] - m); Z += probs[kk]; }
  for (int kk = 0; kk < n_keys; ++kk) probs[kk] /= Z;
  return 0;
}

int oracle_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp master
    n = omp_get_num_threads();
  }
#endif
  return n;
}
