// Work partition of the persistent attention kernel.  Plain C++ (no CUDA types) so that the same
// functions run on the device and in a host unit test.
//
// An "item" is one (layer, sequence, KV head); it owns ceil(seq_len / 64) K/V tiles.  All tiles of
// all items form one flat list ordered by (layer, sequence, KV head, tile).  CTA c of n streams the
// contiguous slice [slice_begin(c), slice_begin(c + 1)) of that list, so every CTA moves the same
// number of tiles (+-1) and an item is cut only where a slice boundary falls inside it.  A CTA's
// slice is a sequence of "segments" (maximal runs inside one item); only its first and its last
// segment can be partial, which bounds the scratch memory to two partial results per CTA.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SPECVLM_HD __host__ __device__ __forceinline__
#else
#define SPECVLM_HD inline
#endif

namespace specvlm {

constexpr int kSchedMaxBatch = 127;     // sequences per call (their tile counts live in shared memory)
constexpr int kSchedMinTilesPerCta = 4;   // below this a slice is not worth a CTA of its own

// Number of CTAs that get a non-empty slice.
SPECVLM_HD int sched_active_ctas(int64_t total_tiles, int grid) {
  int64_t n = (total_tiles + kSchedMinTilesPerCta - 1) / kSchedMinTilesPerCta;
  if (n > grid) n = grid;
  if (n < 1) n = 1;
  return (int)n;
}

SPECVLM_HD int64_t slice_begin(int c, int n_active, int64_t total_tiles) {
  return (int64_t)c * total_tiles / n_active;
}

// The CTA whose slice holds flat tile f (0 <= f < total_tiles).
SPECVLM_HD int slice_owner(int64_t f, int n_active, int64_t total_tiles) {
  return (int)(((f + 1) * n_active - 1) / total_tiles);
}

struct Segment {
  int layer, b, g;        // the item
  int item;               // (layer * batch + b) * n_kv_heads + g
  int tile0;              // first tile of the segment inside the item
  int n_tiles;            // tiles of the segment
  int item_tiles;         // tiles of the whole item
  int64_t item_begin;     // flat index of the item's first tile
};

// Locates flat tile f and cuts the segment at `slice_end`.  prefix[b] = tiles of sequences < b
// (prefix[batch] = tiles of one KV head of one layer); every sequence holding f has >= 1 tile.
SPECVLM_HD Segment segment_at(int64_t f, int64_t slice_end, const int* prefix, int batch, int n_kv_heads) {
  Segment s;
  const int64_t per_layer = (int64_t)n_kv_heads * prefix[batch];
  s.layer = (int)(f / per_layer);
  const int64_t rem = f - (int64_t)s.layer * per_layer;
  int lo = 0, hi = batch - 1;             // last b with n_kv_heads * prefix[b] <= rem
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((int64_t)n_kv_heads * prefix[mid] <= rem) lo = mid; else hi = mid - 1;
  }
  s.b = lo;
  s.item_tiles = prefix[lo + 1] - prefix[lo];
  const int64_t rem2 = rem - (int64_t)n_kv_heads * prefix[lo];
  s.g = (int)(rem2 / s.item_tiles);
  s.tile0 = (int)(rem2 - (int64_t)s.g * s.item_tiles);
  s.item = (s.layer * batch + s.b) * n_kv_heads + s.g;
  s.item_begin = f - s.tile0;
  int64_t n = s.item_tiles - s.tile0;
  if (n > slice_end - f) n = slice_end - f;
  s.n_tiles = (int)n;
  return s;
}

// Scratch slot of the partial result that CTA c holds for the item starting at flat tile item_begin:
// slot 2c when the item is the first segment of c's slice, 2c + 1 otherwise (then it is the last).
SPECVLM_HD int partial_slot(int c, int64_t cta_slice_begin, int64_t item_begin) {
  return cta_slice_begin >= item_begin ? 2 * c : 2 * c + 1;
}

// Walks a CTA's slice segment by segment, in flat order.  (Taking the item that the slice end cuts
// first, so that the merges of cut items happen early, was measured slower: the partial results'
// stores and fences then wait behind the full-rate K/V streams of the other CTAs.)
struct SliceCursor {
  int64_t f, end;
  Segment sg;
  int j;          // tile inside the current segment
  int seg_idx;    // segments entered so far - 1
  SPECVLM_HD void start(int64_t begin, int64_t end_, const int* prefix, int batch, int hkv) {
    f = begin;
    end = end_;
    j = 0;
    seg_idx = 0;
    if (f < end) sg = segment_at(f, end, prefix, batch, hkv);
  }
  SPECVLM_HD bool done() const { return f >= end; }
  SPECVLM_HD bool last_of_segment() const { return j == sg.n_tiles - 1; }
  SPECVLM_HD void next_tile(const int* prefix, int batch, int hkv) {
    ++f;
    if (++j == sg.n_tiles) next_segment(prefix, batch, hkv);
  }
  SPECVLM_HD void next_segment(const int* prefix, int batch, int hkv) {
    f = sg.item_begin + sg.tile0 + sg.n_tiles;
    j = 0;
    ++seg_idx;
    if (f < end) sg = segment_at(f, end, prefix, batch, hkv);
  }
};

}  // namespace specvlm
