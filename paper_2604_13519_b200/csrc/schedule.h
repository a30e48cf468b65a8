// Work partition of the fused verify kernel, shared by device code and by a host-side check.
//
// A projection with T output tiles (128 weight rows each) and KB k-blocks (64 columns each) is a
// line of U = T * KB units, tile-major.  CTA c of n owns the contiguous range
// [unit_begin(c), unit_begin(c + 1)): every CTA streams the same number of weight bytes (to within
// one unit) whatever the shape.  A range cuts into segments, one per tile it touches; only the first
// and the last segment of a range can cover part of a tile.  A tile covered by several CTAs is
// finished by whichever of them arrives last; it adds the partial sums in CTA order, so the result
// does not depend on who that is.  With fewer units than CTAs only the first U CTAs take part, so that
// the CTAs sharing a tile are always consecutive and none of them is empty.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define TS_HD __host__ __device__ __forceinline__
#else
#define TS_HD inline
#endif

namespace ts {

TS_HD uint32_t unit_begin(uint32_t c, uint32_t U, uint32_t n) { return (uint32_t)(((uint64_t)c * U) / n); }

// the CTA whose range holds unit u: the largest c with unit_begin(c) <= u
TS_HD uint32_t unit_owner(uint32_t u, uint32_t U, uint32_t n) {
  return (uint32_t)((((uint64_t)u + 1) * n + U - 1) / U) - 1;
}

TS_HD uint32_t active_ctas(uint32_t U, uint32_t n) { return U < n ? U : n; }

struct Segment {
  int tile, kb0, kb1;   // k-blocks [kb0, kb1) of this tile
  int index;            // position of the segment inside the CTA's range (0 = first)
};

struct SegmentIter {
  uint32_t u, u1;
  int KB, index;
  TS_HD SegmentIter(uint32_t c, int T, int KB_, uint32_t n) : KB(KB_), index(0) {
    const uint32_t U = (uint32_t)T * (uint32_t)KB_;
    const uint32_t na = active_ctas(U, n);
    u = c < na ? unit_begin(c, U, na) : 0;
    u1 = c < na ? unit_begin(c + 1, U, na) : 0;
  }
  TS_HD bool next(Segment *s) {
    if (u >= u1) return false;
    s->tile = (int)(u / (uint32_t)KB);
    s->kb0 = (int)(u % (uint32_t)KB);
    const uint32_t left = u1 - u;
    s->kb1 = (left < (uint32_t)(KB - s->kb0)) ? s->kb0 + (int)left : KB;
    s->index = index++;
    u += (uint32_t)(s->kb1 - s->kb0);
    return true;
  }
};

struct TileCover {
  int c_first, n_seg;   // CTAs c_first .. c_first + n_seg - 1 each hold one segment of the tile
};

TS_HD TileCover tile_cover(int tile, int T, int KB, uint32_t n) {
  const uint32_t U = (uint32_t)T * (uint32_t)KB;
  const uint32_t na = active_ctas(U, n);
  TileCover tc;
  tc.c_first = (int)unit_owner((uint32_t)tile * KB, U, na);
  tc.n_seg = (int)unit_owner((uint32_t)tile * KB + KB - 1, U, na) - tc.c_first + 1;
  return tc;
}

// Partial segments park their sums in one of two slots per CTA: slot 0 for the first segment of the
// CTA's range, slot 1 for any later one (which, being partial, is the last).
TS_HD int slab_slot_of(int c, int tile, int T, int KB, uint32_t n) {
  const uint32_t U = (uint32_t)T * (uint32_t)KB;
  return (unit_begin((uint32_t)c, U, active_ctas(U, n)) < (uint32_t)tile * (uint32_t)KB) ? 1 : 0;
}

// KV positions [pos_beg, pos_end) of one attention split.  Only the whole units (2^unit_shift positions: a page or a
// 64-position block) that lie entirely inside the CACHE -- the `len` positions written by earlier steps -- are cut
// among the splits, balanced to within one unit with the remainder going to the first splits; the last split also
// takes everything after them: the cache's ragged tail and the chunk's own rows, up to `end`.  So every split but
// the last holds whole, fully visible units, only the last one waits for the chunk's K/V and masks, and -- the point
// of the rule -- the cut depends on the cached length alone: a row's blocks, their order and therefore its result
// bits do not change with the number of rows verified beside it.
TS_HD void split_positions(int len, int end, int n_splits, int split, int unit_shift, int *pos_beg, int *pos_end) {
  const int nu = len >> unit_shift;
  const int u0 = (int)(((int64_t)split * nu + n_splits - 1) / n_splits);
  const int u1 = (int)(((int64_t)(split + 1) * nu + n_splits - 1) / n_splits);
  *pos_beg = u0 << unit_shift;
  *pos_end = (split == n_splits - 1) ? end : (u1 << unit_shift);
}

}  // namespace ts
