// Work-item numbering shared by the decode kernels.
#pragma once
#include "sq_internal.h"

namespace sq {

constexpr int kStatStride = 4;  // per (item, head): max, sum, sum of the bf16-rounded weights, pad

constexpr unsigned kFull = 0xffffffffu;

struct ItemLoc {
  int layer, local, n_split, base;
};

__device__ __forceinline__ int n_split_of(const DecodeArgs& a, int b) {
  int len = min(a.n_tok + 1, b);
  return (len + a.split_tokens - 1) / a.split_tokens;
}

// Work items of a launch are numbered layer by layer in `order` (largest budget first), and
// within a layer as unit * n_split + split.  Each warp finds, by a prefix scan over the
// layers, either the layer an item index falls in (want_layer < 0) or the first item of a
// given layer.
__device__ __forceinline__ bool locate(const DecodeArgs& a, int idx, int want_layer, ItemLoc& out) {
  const int lane = threadIdx.x & 31;
  int running = 0;
  for (int c = 0; c < a.n_layer_total; c += 32) {
    const int i = c + lane;
    int l = -1, ns = 0, cnt = 0;
    if (i < a.n_layer_total) {
      int li = a.order[i];
      if (li >= a.layer_begin && li < a.layer_end) {
        l = li;
        ns = n_split_of(a, a.layers[li].b);
        cnt = a.n_unit * ns;
      }
    }
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(kFull, incl, o);
      if (lane >= o) incl += t;
    }
    unsigned hit = (want_layer >= 0) ? __ballot_sync(kFull, l == want_layer)
                                     : __ballot_sync(kFull, cnt > 0 && idx < running + incl);
    if (hit) {
      const int src = __ffs(hit) - 1;
      out.layer = __shfl_sync(kFull, l, src);
      out.n_split = __shfl_sync(kFull, ns, src);
      out.base = running + __shfl_sync(kFull, incl - cnt, src);
      out.local = idx - out.base;
      return true;
    }
    running += __shfl_sync(kFull, incl, 31);
  }
  return false;
}

}  // namespace sq
