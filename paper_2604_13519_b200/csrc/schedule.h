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

// KV positions of one attention split: whole pages, balanced to within one page.
TS_HD void split_pages(int n_pages, int n_splits, int split, int *p0, int *p1) {
  *p0 = (int)(((int64_t)split * n_pages) / n_splits);
  *p1 = (int)(((int64_t)(split + 1) * n_pages) / n_splits);
}


// The same cut in whole 64-position blocks (4 pages), so that only a sequence's last split ends in a partial block.
// Cut points are rounded up, so a remainder goes to the first splits: the last one, which alone waits for the chunk's
// own K/V rows and masks its last block, never gets the extra block.
TS_HD void split_blocks(int n_pages, int n_splits, int split, int *p0, int *p1) {
  const int nb = (n_pages + 3) >> 2;
  const int b0 = (int)(((int64_t)split * nb + n_splits - 1) / n_splits);
  const int b1 = (int)(((int64_t)(split + 1) * nb + n_splits - 1) / n_splits);
  *p0 = b0 << 2;
  *p1 = (b1 << 2) < n_pages ? (b1 << 2) : n_pages;
}

}  // namespace ts
