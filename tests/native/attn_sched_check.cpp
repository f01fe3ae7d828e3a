// Host-side brute-force check of the attention work partition (csrc/attn_sched.h): built and run by
// tests/test_attn_sched.py.  Prints "ok" or the first violated property.
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "../../paper_2508_16201_b200/csrc/attn_sched.h"

using namespace specvlm;

static int check(const std::vector<int>& tiles, int n_layers, int hkv, int grid) {
  const int batch = (int)tiles.size();
  std::vector<int> prefix(batch + 1, 0);
  for (int b = 0; b < batch; ++b) prefix[b + 1] = prefix[b] + tiles[b];
  const int64_t total = (int64_t)n_layers * hkv * prefix[batch];
  if (total == 0) return 0;
  const int n = sched_active_ctas(total, grid);
  const int n_items = n_layers * batch * hkv;
  std::vector<int> covered(n_items, 0), parts(n_items, 0);
  std::vector<int64_t> item_begin(n_items, -1);
  std::vector<std::vector<int>> slots(n_items);
  if (slice_begin(0, n, total) != 0 || slice_begin(n, n, total) != total) return 1;
  for (int c = 0; c < n; ++c) {
    const int64_t t0 = slice_begin(c, n, total), t1 = slice_begin(c + 1, n, total);
    if (t1 <= t0) return 2;                                  // every active CTA has work
    if (t1 - t0 > (total + n - 1) / n) return 3;             // balanced
    std::vector<int> partial_slots;
    int64_t f = t0;
    int nseg = 0;
    while (f < t1) {
      const Segment s = segment_at(f, t1, prefix.data(), batch, hkv);
      if (s.n_tiles < 1 || s.tile0 < 0 || s.tile0 + s.n_tiles > s.item_tiles) return 4;
      if (s.item_tiles != tiles[s.b]) return 5;
      if (s.item != (s.layer * batch + s.b) * hkv + s.g || s.item < 0 || s.item >= n_items) return 6;
      if (s.item_begin != f - s.tile0) return 7;
      if (item_begin[s.item] >= 0 && item_begin[s.item] != s.item_begin) return 8;
      item_begin[s.item] = s.item_begin;
      for (int64_t k = f; k < f + s.n_tiles; ++k)
        if (slice_owner(k, n, total) != c) return 9;
      covered[s.item] += s.n_tiles;
      const bool complete = s.tile0 == 0 && s.n_tiles == s.item_tiles;
      if (!complete) {
        // only the first and the last segment of a slice may be partial
        const bool is_first = nseg == 0, is_last = f + s.n_tiles == t1;
        if (!is_first && !is_last) return 10;
        const int slot = partial_slot(c, t0, s.item_begin);
        if (slot != 2 * c && slot != 2 * c + 1) return 11;
        for (int q : partial_slots)
          if (q == slot) return 12;                          // two partials of one CTA never share a slot
        partial_slots.push_back(slot);
        slots[s.item].push_back(slot);
        parts[s.item] += 1;
      }
      f += s.n_tiles;
      ++nseg;
    }
    // the kernel's cursor visits the same segments, each tile once, whether it steps by tile
    // (producers, issuers) or by segment (softmax groups)
    SliceCursor w;
    w.start(t0, t1, prefix.data(), batch, hkv);
    std::vector<char> seen((size_t)(t1 - t0), 0);
    int wseg = 0;
    while (!w.done()) {
      const Segment s = w.sg;
      if (w.seg_idx != wseg || w.j != 0) return 16;
      const Segment lin = segment_at(s.item_begin + s.tile0, t1, prefix.data(), batch, hkv);
      if (lin.item != s.item || lin.tile0 != s.tile0 || lin.n_tiles != s.n_tiles) return 17;   // a segment of the linear walk
      for (int k = 0; k < s.n_tiles; ++k) {
        const int64_t g = s.item_begin + s.tile0 + k;
        if (g < t0 || g >= t1 || seen[(size_t)(g - t0)]) return 18;
        seen[(size_t)(g - t0)] = 1;
      }
      // tile-wise stepping reaches the same next segment as segment-wise stepping
      SliceCursor w2 = w;
      for (int k = 0; k < s.n_tiles; ++k) {
        if (w2.last_of_segment() != (k == s.n_tiles - 1)) return 19;
        w2.next_tile(prefix.data(), batch, hkv);
      }
      w.next_segment(prefix.data(), batch, hkv);
      if (w2.done() != w.done() || w2.seg_idx != w.seg_idx) return 20;
      if (!w.done() && (w2.sg.item != w.sg.item || w2.sg.tile0 != w.sg.tile0 || w2.f != w.f)) return 21;
      ++wseg;
    }
    if (wseg != nseg) return 22;
    for (char v : seen)
      if (!v) return 23;
  }
  for (int it = 0; it < n_items; ++it) {
    const int b = (it / hkv) % batch;
    if (covered[it] != tiles[b]) return 13;                  // every tile exactly once
    if (tiles[b] == 0) continue;
    const int c_first = slice_owner(item_begin[it], n, total);
    const int c_last = slice_owner(item_begin[it] + tiles[b] - 1, n, total);
    if (parts[it] != (c_last > c_first ? c_last - c_first + 1 : 0)) return 14;   // the merger's count
    if (c_last > c_first) {
      // the merging CTA recomputes the slots from the slice bounds alone
      for (int c = c_first, k = 0; c <= c_last; ++c, ++k)
        if (partial_slot(c, slice_begin(c, n, total), item_begin[it]) != slots[it][k]) return 15;
    }
  }
  return 0;
}

int main() {
  unsigned rng = 12345u;
  auto rnd = [&](int m) { rng = rng * 1664525u + 1013904223u; return (int)((rng >> 8) % (unsigned)m); };
  struct Fixed { std::vector<int> tiles; int L, H, grid; };
  const std::vector<Fixed> fixed = {
      {{101}, 80, 8, 148}, {{12}, 28, 4, 148}, {{100}, 28, 4, 148}, {{3}, 1, 1, 148}, {{1}, 1, 1, 148},
      {{0, 5, 0, 9, 0}, 3, 2, 7}, {{785, 1}, 2, 8, 148}, {{99, 197, 295, 393}, 80, 8, 148}};
  for (const Fixed& f : fixed) {
    const int rc = check(f.tiles, f.L, f.H, f.grid);
    if (rc) { std::printf("fixed case failed: property %d\n", rc); return 1; }
  }
  for (int iter = 0; iter < 4000; ++iter) {
    const int batch = 1 + rnd(6), L = 1 + rnd(5), H = 1 + rnd(4), grid = 1 + rnd(40);
    std::vector<int> tiles(batch);
    for (int& t : tiles) t = rnd(4) == 0 ? 0 : 1 + rnd(30);
    const int rc = check(tiles, L, H, grid);
    if (rc) { std::printf("random case %d failed: property %d\n", iter, rc); return 1; }
  }
  std::printf("ok\n");
  return 0;
}
