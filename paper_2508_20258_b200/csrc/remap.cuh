// Tile-order remaps in closed form, usable from host and device code.
//
// The paper's swizzle is a few integer operations at kernel entry that recompute the
// block id (GEMM case study, appendix listing).  sp::Sched carries the resolved scheme
// parameters; sp::slot_to_tile(sched, s) returns the logical tile id executed at slot s.
// Schemes that need a rank among skipped cells (space-filling curves on grids that are
// not a power-of-two square, caller tables) are served from a table built once
// (host: build_perm_host, device: the builder kernel in remap_device.cu); everything
// else is pure arithmetic evaluated by the GEMM scheduler itself.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SP_HD __host__ __device__ __forceinline__
#else
#define SP_HD inline
#endif

namespace sp {

enum : int { kRow = 0, kCol = 1, kGroupM = 2, kGroupN = 3, kMorton = 4, kHilbert = 5, kXcd = 6, kDieSplit = 7,
             kCustom = 8, kHilbertRect = 9 };

struct Sched {
  int scheme;        // sp_scheme
  int Tm, Tn, T;     // tile grid
  int group;         // GROUP_M / GROUP_N
  int serp;          // GROUP_M / GROUP_N (also as inner order): odd bands walk the other way (boustrophedon)
  int X, W, balanced;  // XCD: chiplets, window (already resolved: W >= 1), balanced flag
  int axis, inner, inner_group, interleave;  // DIE_SPLIT
  int use_table;     // 1: the scheduler reads perm[s] from memory
};

SP_HD int imin(int a, int b) { return a < b ? a : b; }

// Decode one index of the order-k Hilbert curve that starts at (0,0), first moves along x
// and ends at (2^k - 1, 0).  Digits are consumed least significant first: after `level`
// steps (x, y) is the position inside a 2^level square, which the next base-4 digit
// places (and reflects) inside the 2^(level+1) square.
SP_HD void hilbert_decode(int k, uint32_t d, int& x, int& y) {
  int px = 0, py = 0;
  for (int level = 0; level < k; ++level) {
    const int h = 1 << level;
    const uint32_t q = (d >> (2 * level)) & 3u;
    int nx, ny;
    if (q == 0) { nx = py; ny = px; }
    else if (q == 1) { nx = px; ny = py + h; }
    else if (q == 2) { nx = px + h; ny = py + h; }
    else { nx = 2 * h - 1 - py; ny = h - 1 - px; }
    px = nx; py = ny;
  }
  x = px; y = py;
}

SP_HD int isgn(int v) { return (v > 0) - (v < 0); }
SP_HD int iabs(int v) { return v < 0 ? -v : v; }
SP_HD int floor_half(int v) { return v >= 0 ? v / 2 : -((-v + 1) / 2); }

// Cell number d of the generalised Hilbert curve over a rectangle of `width` x `height` cells.  The curve is the
// "generalized Hilbert curve" for rectangles of arbitrary size published by Jakub Cerveny (2018; reference implementation
// under the BSD 2-clause licence): a rectangle spanned by a major vector a and a minor vector b is cut in two along a when
// it is long, else into three parts walked b-wise, a-wise and back.  This is not that implementation: instead of
// generating the whole curve it descends into the part that holds index d: O(log) steps, no table.  The curve starts at (0, 0) and
// moves one cell at a time (one diagonal step can occur when the sides' parities force it).
SP_HD void hilbert_rect_cell(int width, int height, int d, int& cx, int& cy) {
  int x = 0, y = 0, ax, ay, bx, by;
  if (width >= height) { ax = width; ay = 0; bx = 0; by = height; } else { ax = 0; ay = height; bx = width; by = 0; }
  for (;;) {
    const int w = iabs(ax + ay), h = iabs(bx + by);
    const int dax = isgn(ax), day = isgn(ay), dbx = isgn(bx), dby = isgn(by);
    if (h == 1) { cx = x + dax * d; cy = y + day * d; return; }
    if (w == 1) { cx = x + dbx * d; cy = y + dby * d; return; }
    int ax2 = floor_half(ax), ay2 = floor_half(ay), bx2 = floor_half(bx), by2 = floor_half(by);
    const int w2 = iabs(ax2 + ay2), h2 = iabs(bx2 + by2);
    if (2 * w > 3 * h) {                                   // long: two parts along a
      if ((w2 & 1) && w > 2) { ax2 += dax; ay2 += day; }
      const int n1 = iabs(ax2 + ay2) * h;
      if (d < n1) { ax = ax2; ay = ay2; }
      else { d -= n1; x += ax2; y += ay2; ax -= ax2; ay -= ay2; }
    } else {                                               // three parts
      if ((h2 & 1) && h > 2) { bx2 += dbx; by2 += dby; }
      const int hb = iabs(bx2 + by2);
      const int n1 = hb * iabs(ax2 + ay2), n2 = w * (h - hb);
      if (d < n1) {
        const int tx = ax2, ty = ay2;
        ax = bx2; ay = by2; bx = tx; by = ty;
      } else if (d < n1 + n2) {
        d -= n1; x += bx2; y += by2; bx -= bx2; by -= by2;
      } else {
        d -= n1 + n2;
        x += (ax - dax) + (bx2 - dbx); y += (ay - day) + (by2 - dby);
        const int nax = -bx2, nay = -by2, nbx = -(ax - ax2), nby = -(ay - ay2);
        ax = nax; ay = nay; bx = nbx; by = nby;
      }
    }
  }
}

SP_HD uint32_t compact_even_bits(uint32_t v) {
  v &= 0x55555555u;
  v = (v | (v >> 1)) & 0x33333333u;
  v = (v | (v >> 2)) & 0x0F0F0F0Fu;
  v = (v | (v >> 4)) & 0x00FF00FFu;
  v = (v | (v >> 8)) & 0x0000FFFFu;
  return v;
}

SP_HD void morton_decode(uint32_t z, int& x, int& y) {
  x = (int)compact_even_bits(z);
  y = (int)compact_even_bits(z >> 1);
}

SP_HD int curve_order(int Tm, int Tn) {
  const int m = Tm > Tn ? Tm : Tn;
  int k = 0;
  while ((1 << k) < m) ++k;
  return k;
}

// Cell `d` of a curve laid over a (Tm x Tn) grid: returns false when it falls outside.
SP_HD bool curve_cell(int kind, int k, int Tm, int Tn, uint32_t d, int& tm, int& tn) {
  int x, y;
  if (kind == kHilbert) hilbert_decode(k, d, x, y); else morton_decode(d, x, y);
  if (Tm >= Tn) { tm = y; tn = x; } else { tm = x; tn = y; }
  return tm < Tm && tn < Tn;
}

// Arithmetic orders on a (Tm x Tn) grid; returns the grid-local id tm * Tn + tn.
SP_HD int plain_order(int scheme, int Tm, int Tn, int G, int serp, int s) {
  switch (scheme) {
    case kCol: return (s % Tm) * Tn + s / Tm;
    case kGroupM: {
      const int band = G * Tn;
      const int b = s / band, first = b * G, g = imin(G, Tm - first), r = s - b * band;
      const int tn = (serp && (b & 1)) ? Tn - 1 - r / g : r / g;
      return (first + r % g) * Tn + tn;
    }
    case kGroupN: {
      const int band = G * Tm;
      const int b = s / band, first = b * G, g = imin(G, Tn - first), r = s - b * band;
      const int tm = (serp && (b & 1)) ? Tm - 1 - r / g : r / g;
      return tm * Tn + first + r % g;
    }
    default: return s;
  }
}

// The paper's formula on one window of n slots; local id in, local id out.
SP_HD int xcd_local(int n, int X, int balanced, int p) {
  const int x = p % X, j = p / X;
  if (!balanced) return x * ((n + X - 1) / X) + j;
  const int q = n / X, r = n % X;
  return x * q + imin(x, r) + j;
}

// DIE_SPLIT bookkeeping: which half a slot belongs to and its index inside that half.
struct HalfPos { int half, idx, rows, cols, row0, col0; };

SP_HD HalfPos die_split_pos(const Sched& c, int s) {
  HalfPos p;
  const int cut = c.axis == 0 ? (c.Tm + 1) / 2 : (c.Tn + 1) / 2;
  const int h0 = c.axis == 0 ? cut * c.Tn : cut * c.Tm;
  const int h1 = c.T - h0;
  if (!c.interleave) {
    p.half = s >= h0; p.idx = p.half ? s - h0 : s;
  } else if (s < 2 * h1) {
    p.half = s & 1; p.idx = s >> 1;
  } else {
    p.half = 0; p.idx = s - h1;
  }
  if (c.axis == 0) {
    p.rows = p.half ? c.Tm - cut : cut; p.cols = c.Tn; p.row0 = p.half ? cut : 0; p.col0 = 0;
  } else {
    p.rows = c.Tm; p.cols = p.half ? c.Tn - cut : cut; p.row0 = 0; p.col0 = p.half ? cut : 0;
  }
  return p;
}

// Slot of the idx-th element of half `half` (inverse of die_split_pos on (half, idx)).
SP_HD int die_split_slot(const Sched& c, int half, int idx) {
  const int cut = c.axis == 0 ? (c.Tm + 1) / 2 : (c.Tn + 1) / 2;
  const int h0 = c.axis == 0 ? cut * c.Tn : cut * c.Tm;
  const int h1 = c.T - h0;
  if (!c.interleave) return half ? h0 + idx : idx;
  if (idx < h1) return 2 * idx + half;
  return idx + h1;
}

// Die-pinned scheduling: the r-th unit (0-based) to arrive on L2 half `die`, where n[d] units are expected on half d
// and exactly n[0] + n[1] units exist.  A unit beyond the expected count of its half takes a rank left free on the
// other half, from the top down, so that every (half, rank) pair is taken exactly once under any placement.
SP_HD void pinned_ticket(int n0, int n1, int die, int r, int& die_out, int& rank_out) {
  const int n_own = die ? n1 : n0, n_other = die ? n0 : n1;
  if (r < n_own) { die_out = die; rank_out = r; }
  else { die_out = die ^ 1; rank_out = n_other - 1 - (r - n_own); }
}

SP_HD bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

// True when slot_to_tile needs no table for this configuration.
SP_HD bool arithmetic_scheme(const Sched& c) {
  switch (c.scheme) {
    case kRow: case kCol: case kGroupM: case kGroupN: case kXcd: case kHilbertRect: return true;
    case kMorton: case kHilbert: return c.Tm == c.Tn && is_pow2(c.Tm);
    case kDieSplit: return c.inner <= kGroupN;
    default: return false;
  }
}

// slot -> tile for arithmetic schemes (see arithmetic_scheme); table schemes read perm[s].
SP_HD int slot_to_tile(const Sched& c, int s) {
  switch (c.scheme) {
    case kRow: case kCol: case kGroupM: case kGroupN:
      return plain_order(c.scheme, c.Tm, c.Tn, c.group, c.serp, s);
    case kMorton: case kHilbert: {
      int tm, tn;
      curve_cell(c.scheme, curve_order(c.Tm, c.Tn), c.Tm, c.Tn, (uint32_t)s, tm, tn);
      return tm * c.Tn + tn;
    }
    case kHilbertRect: {
      int x, y;
      hilbert_rect_cell(c.Tn, c.Tm, s, x, y);
      return y * c.Tn + x;
    }
    case kXcd: {
      const int base = (s / c.W) * c.W;
      const int n = imin(c.W, c.T - base);
      return base + xcd_local(n, c.X, c.balanced, s - base);
    }
    case kDieSplit: {
      const HalfPos p = die_split_pos(c, s);
      const int local = plain_order(c.inner, p.rows, p.cols, c.inner_group, c.serp, p.idx);
      return (p.row0 + local / p.cols) * c.Tn + p.col0 + local % p.cols;
    }
    default: return s;
  }
}

}  // namespace sp
