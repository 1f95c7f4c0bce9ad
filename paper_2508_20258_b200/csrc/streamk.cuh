// Work decomposition of the persistent GEMM: data-parallel tiles plus an optional stream-K tail.
//
// The paper's remap decides WHICH tile a slot computes; it has no counterpart for splitting a tile along k.
// The split exists for wave quantisation: T tiles on U persistent units leave the last wave partly empty when
// U does not divide T.  With the tail switched on, the last `tiles` slots are not dealt out tile by tile.  Their
// tiles' k-blocks are laid end to end -- position p = j * KB + kb for the j-th tail slot -- and cut into `units`
// contiguous ranges of equal length (to within one k-block): unit u takes [u * W / units, (u + 1) * W / units),
// W = tiles * KB.  The kernel handles any such cut; sk_plan() below only ever asks for cuts whose ranges are equal
// fractions of one tile.
//
// A range crosses at most a few tiles.  Its pieces ("segments") are of three kinds:
//   full         -- all k-blocks of the tile: computed and stored as usual;
//   contributor  -- does not reach the tile's last k-block: the fp32 partial goes to this unit's workspace slot and
//                   a flag is raised;
//   owner        -- reaches the last k-block but not the first: waits for the contributors (all of them lower-numbered
//                   units), adds their partials to its accumulator in descending unit order, stores the tile.
// A unit walks its segments from the highest tile down.  Its contributor segment (there is at most one: the piece at
// the end of its range) therefore comes first and never waits, and its owner segment comes last, long after the
// lower-numbered units have finished the pieces it needs; waits only ever point to lower block indices.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SP_SK_HD __host__ __device__ __forceinline__
#else
#define SP_SK_HD inline
#endif

namespace sp {

enum : int { kWorkFull = 0, kWorkContrib = 1, kWorkOwner = 2 };

struct SkPlan {
  int tiles;       // tail slots [first_slot, first_slot + tiles); 0 = no tail
  int units;       // units that share the tail (units >= this one have no segment)
  int first_slot;  // T - tiles
};

struct Work {
  int slot;        // position in issue order: the tile is slot_to_tile(slot)
  int k0, k1;      // k-blocks [k0, k1) of that tile
  int kind;        // kWorkFull / kWorkContrib / kWorkOwner
};

SP_SK_HD long long sk_range_begin(const SkPlan& p, int unit, int KB) {
  return (long long)unit * ((long long)p.tiles * KB) / p.units;
}

// Number of segments of `unit` in the tail.
SP_SK_HD int sk_segments(const SkPlan& p, int unit, int KB) {
  if (p.tiles <= 0 || unit >= p.units) return 0;
  const long long a = sk_range_begin(p, unit, KB), b = sk_range_begin(p, unit + 1, KB);
  if (b <= a) return 0;
  return (int)((b - 1) / KB - a / KB) + 1;
}

// The j-th segment of `unit` in walking order (highest tile first).
SP_SK_HD Work sk_segment(const SkPlan& p, int unit, int j, int KB) {
  const long long a = sk_range_begin(p, unit, KB), b = sk_range_begin(p, unit + 1, KB);
  const long long tt = (b - 1) / KB - j;            // tail slot index
  const long long lo = tt * KB;
  Work w;
  w.slot = p.first_slot + (int)tt;
  w.k0 = a > lo ? (int)(a - lo) : 0;
  w.k1 = b < lo + KB ? (int)(b - lo) : KB;
  w.kind = w.k1 < KB ? kWorkContrib : (w.k0 > 0 ? kWorkOwner : kWorkFull);
  return w;
}

// Contributors of the owner segment of `unit` on tail slot `slot`: units unit-1, unit-2, ... down to the one whose
// range holds the tile's first k-block.  Returns how many.
SP_SK_HD int sk_contributors(const SkPlan& p, int unit, int slot, int KB) {
  const long long lo = (long long)(slot - p.first_slot) * KB;
  int n = 0;
  for (int u = unit - 1; u >= 0; --u) {
    ++n;
    if (sk_range_begin(p, u, KB) <= lo) break;
  }
  return n;
}

// Host policy: which slots form the tail for T tiles on `units` units with KB k-blocks per tile.
// Only the remainder R = T mod units is split, and only into equal pieces: each of its tiles goes to f = units / R
// units (2 <= f <= kMaxPieces, pieces of at least kMinRange k-blocks), piece i covering k-blocks [i * KB / f, (i + 1) * KB / f).
// Pieces with the same i run side by side and walk k in step, as the tiles of a full wave do, so the A and B panels
// they share are still read from L2 by all of them at the same time.  (Ranges of unequal phase -- the general
// stream-K cut, also over an extra full wave -- were measured: every unit then streams its operands alone, the tail
// turns DRAM-bound and takes longer than the partly empty wave it replaces.)
inline SkPlan sk_plan(int64_t T, int units, int KB) {
  constexpr int kMinRange = 4;
  constexpr int kMaxPieces = 8;
  SkPlan p = {0, units, (int)T};
  const int64_t R = T % units;
  if (R == 0) return p;
  int64_t f = units / R;
  if (f > KB / kMinRange) f = KB / kMinRange;
  if (f > kMaxPieces) f = kMaxPieces;      // the unit that stores a tile adds the other pieces one after the other
  if (f < 2) return p;
  p.tiles = (int)R;
  p.units = (int)(R * f);
  p.first_slot = (int)(T - R);
  return p;
}

}  // namespace sp
