// Even deal of a decode launch's 128-token tiles over persistent CTAs, shared by the wide-group
// attention kernel and its H2O score pass.  The kept tokens of every (layer, unit) of the launch
// are cut into 128-token tiles, numbered in launch order (largest budget first); CTA c takes the
// tiles [c * chunk, (c + 1) * chunk).  A CTA's run of tiles of one unit is a segment; a unit cut
// by a CTA boundary is finished by the piece that arrives last at the unit's ticket.
#pragma once
#include <algorithm>

#include "sq_internal.h"
#include "sq_tc.cuh"

namespace sq {

struct StreamArgs : DecodeArgsBase {
  int cum[kMaxLayers + 1];  // tiles before the k-th descriptor of the launch
  int chunk, total;         // tiles per CTA, tiles of the launch
};

// The segments of one CTA, in order.  Every role walks them with its own copy.
struct SegIter {
  int g, g_end, k;  // tile cursor, end of the CTA's range, descriptor index in launch order
  int seg;          // number of the current segment within the CTA
  int layer, unit, tile0, ntile, nt, len, u0;  // current segment: its unit's tiles are [u0, u0 + nt)
  __device__ void init(const StreamArgs& a, int cta) {
    g = min(a.total, cta * a.chunk);
    g_end = min(a.total, g + a.chunk);
    k = 0;
    seg = -1;
  }
  __device__ bool next(const StreamArgs& a) {
    if (g >= g_end) return false;
    while (a.cum[k + 1] <= g) ++k;
    layer = a.order[k];
    len = min(a.n_tok + 1, a.layers[layer].b);
    nt = (len + tc::kTM - 1) / tc::kTM;
    const int local = g - a.cum[k];
    unit = local / nt;
    tile0 = local - unit * nt;
    u0 = g - tile0;
    ntile = min(nt - tile0, g_end - g);
    g += ntile;
    ++seg;
    return true;
  }
  // pieces of the current unit: CTAs c_first .. c_first + n_piece - 1
  __device__ int c_first(const StreamArgs& a) const { return u0 / a.chunk; }
  __device__ int n_piece(const StreamArgs& a) const { return (u0 + nt - 1) / a.chunk - u0 / a.chunk + 1; }
};
// Partial slot of piece j of a unit whose first piece is CTA c_first: a CTA owns two slots, one
// for a segment that begins its unit (it can only be the CTA's last) and one for a segment that
// continues a unit begun by an earlier CTA (it can only be the CTA's first).
__device__ __forceinline__ int piece_slot(int c_first, int j) { return j == 0 ? 2 * c_first + 1 : 2 * (c_first + j); }


// Host: fills the tile table for the descriptors [k0, k0 + cnt) of the launch (launch order) and
// deals the tiles out over at most `slots` CTAs.  Returns the grid size (0: nothing to do, -1:
// too many tiles for 32-bit tile numbers).
inline int deal_tiles(StreamArgs& t, const DecodeArgs& a, const int* desc_tiles, int k0, int cnt, int slots) {
  t.order = a.order + k0;
  t.n_layer_total = cnt;
  long long total = 0;
  for (int k = 0; k < cnt; ++k) {
    t.cum[k] = (int)total;
    total += (long long)a.n_unit * desc_tiles[k0 + k];
    if (total > 0x3fffffffLL) return -1;
  }
  t.cum[cnt] = (int)total;
  if (total == 0) return 0;
  t.total = (int)total;
  t.chunk = (int)((total + slots - 1) / slots);
  return (int)((total + t.chunk - 1) / t.chunk);
}

}  // namespace sq
