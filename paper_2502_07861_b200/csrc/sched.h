// Host-side bookkeeping of MergeAndReduce (Algorithm 3): which SoftmaxBalance calls fire,
// where their t input rows live and where their t/2 survivors go.  Pure integer code, no
// CUDA calls, so it can be exercised without a device.
//
// Per stream the arena holds one region per level:
//   level 0      : linear buffer [start0, start0+len0) of uncompressed rows (C^0 + window)
//   level 1..T-1 : 2t rows; the set C^l is empty or holds one half (t/2 rows) at base 0 or t
//   level T      : C^T, appended to for ever
// A batch may contain many consecutive blocks of a stream; survivors that will be consumed
// again inside the same batch travel through two shared ping-pong pools instead of the
// small per-level regions (pool (l & 1) receives level-l survivors, two halves per slot).
#pragma once

#include <algorithm>
#include <utility>
#include <vector>

#include "common.cuh"

namespace bkv {

struct StreamState {
  int64_t appended = 0;                  // tokens ever appended to C^0
  int64_t pending = 0;                   // tokens appended since the last compress
  int32_t start0 = 0, len0 = 0;          // level-0 segment
  int32_t lvl_len[kMaxLevels + 1] = {};  // rows held at levels 1..T
  int32_t lvl_base[kMaxLevels + 1] = {}; // base (0 or t) of the half held at levels 1..T-1
  int64_t calls_done[kMaxLevels + 1] = {};  // calls run per level (= next call ordinal)
};

struct Layout {
  int32_t t = 0, T = 0, W = 0;
  int64_t R = 0;                          // rows per stream
  int32_t region_off[kMaxLevels + 1] = {};
  int32_t cap0 = 0, capT = 0;
  int64_t pool_row[2] = {0, 0};           // first arena row of each pool
  int64_t pool_pairs = 0;                 // slots (of t rows) per pool
};

struct Plan {
  std::vector<std::vector<CallDesc>> levels;  // [T] calls per level, launch order
  std::vector<MoveDesc> moves;
  std::vector<SegUpdate> segs;
  int max_move_rows = 0;
};

// Blocks of t eligible tokens that are ready in C^0 (the newest W tokens are not eligible).
inline int64_t ready_blocks(const Layout& Lo, const StreamState& S) {
  const int64_t eligible = std::max<int64_t>(0, S.appended - Lo.W);
  return eligible / Lo.t - S.calls_done[0];
}

// Plans every call that `runs` (stream, number of level-0 blocks) triggers, level by level.
// Returns false if a pool would overflow (the caller sizes batches so that it cannot).
inline bool plan_batch(const Layout& Lo, StreamState* st, const std::vector<std::pair<int, int>>& runs, Plan& P) {
  const int t = Lo.t, T = Lo.T, half = t / 2;
  P.levels.assign(T, {});
  P.moves.clear(); P.segs.clear(); P.max_move_rows = 0;
  struct Cur { int stream; std::vector<int64_t> src; };
  std::vector<Cur> cur;
  for (const auto& run : runs) {
    const int s = run.first, nb = run.second;
    if (nb <= 0) continue;
    StreamState& S = st[s];
    Cur c{s, {}};
    const int64_t base = (int64_t)s * Lo.R + Lo.region_off[0] + S.start0;
    for (int k = 0; k < nb; ++k) c.src.push_back(base + (int64_t)k * t);
    S.start0 += nb * t;
    S.len0 -= nb * t;
    cur.push_back(std::move(c));
  }
  for (int l = 0; l < T; ++l) {
    int64_t pool_next = 0;
    std::vector<Cur> nxt;
    for (auto& c : cur) {
      StreamState& S = st[c.stream];
      const int n = (int)c.src.size();
      if (n == 0) continue;
      const int64_t sb = (int64_t)c.stream * Lo.R;
      Cur nc{c.stream, {}};
      if (l + 1 == T) {
        for (int k = 0; k < n; ++k) {
          CallDesc d{};
          d.src_row = c.src[k];
          d.dst_row = sb + Lo.region_off[T] + S.lvl_len[T] + (int64_t)k * half;
          d.dbg_off = -1; d.stream = c.stream; d.ordinal = (int32_t)S.calls_done[l]++;
          P.levels[l].push_back(d);
        }
        S.lvl_len[T] += n * half;
      } else {
        const int h = S.lvl_len[l + 1] ? 1 : 0;     // a half is already waiting in C^{l+1}
        const int slots = h + n, pairs = slots / 2, left = slots % 2;
        const int64_t pers = sb + Lo.region_off[l + 1];
        const int old_base = S.lvl_base[l + 1];
        const int new_base = h ? (old_base ? 0 : t) : 0;
        const int pool_pairs_needed = pairs - (h && pairs > 0 ? 1 : 0);
        if (pool_next + pool_pairs_needed > Lo.pool_pairs) return false;
        for (int k = 0; k < n; ++k) {
          const int j = h + k, pr = j / 2, within = j % 2;
          CallDesc d{};
          d.src_row = c.src[k];
          if (pr < pairs) {
            if (h && pr == 0) d.dst_row = pers + old_base + half;
            else d.dst_row = Lo.pool_row[l & 1] + (pool_next + pr - h) * (int64_t)t + (int64_t)within * half;
          } else {
            d.dst_row = pers + new_base;
          }
          d.dbg_off = -1; d.stream = c.stream; d.ordinal = (int32_t)S.calls_done[l]++;
          P.levels[l].push_back(d);
        }
        for (int pr = 0; pr < pairs; ++pr) {
          if (h && pr == 0) nc.src.push_back(pers + old_base);
          else nc.src.push_back(Lo.pool_row[l & 1] + (pool_next + pr - h) * (int64_t)t);
        }
        pool_next += pool_pairs_needed;
        S.lvl_len[l + 1] = left ? half : 0;
        S.lvl_base[l + 1] = left ? new_base : 0;
      }
      nxt.push_back(std::move(nc));
    }
    cur.swap(nxt);
  }
  for (const auto& run : runs) {
    const int s = run.first;
    if (run.second <= 0) continue;
    StreamState& S = st[s];
    const int64_t r0 = (int64_t)s * Lo.R + Lo.region_off[0];
    if (S.len0 == 0) {
      S.start0 = 0;
    } else if (S.start0 >= S.len0) {
      P.moves.push_back(MoveDesc{r0 + S.start0, r0, s, S.len0});
      P.max_move_rows = std::max(P.max_move_rows, (int)S.len0);
      S.start0 = 0;
    }
    const int32_t sbase = s * (T + 1);
    P.segs.push_back(SegUpdate{sbase, S.start0, S.len0, 0});
    for (int l = 1; l < T; ++l) P.segs.push_back(SegUpdate{sbase + l, S.lvl_base[l], S.lvl_len[l], 0});
    P.segs.push_back(SegUpdate{sbase + T, 0, S.lvl_len[T], 0});
  }
  return true;
}

}  // namespace bkv
