// Work-item numbering shared by the decode kernels.
#pragma once
#include <cuda_bf16.h>

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


// Split-K merge without a second launch (policies without scores): every piece of a unit
// bumps the unit's ticket after its partials are written; the piece that arrives last reads
// all of them back (in piece order, so the result does not depend on who merges), writes the
// output and resets the ticket.  No piece ever waits for another.  With lse_out set, the merged
// log-sum-exp (log2 domain, from the unrounded weight sums) of every head is stored there too.
template <typename T>
__device__ __forceinline__ void merge_if_last(const DecodeArgs& a, const ItemLoc& it, int unit,
                                              float* lse_out = nullptr) {
  __shared__ int s_last;
  __shared__ float s_mM[kMaxGroup], s_mInv[kMaxGroup];
  const int tid = threadIdx.x, nt = blockDim.x, G = a.group, D = a.head_dim, ns = it.n_split;
  int* ticket = a.tickets + (size_t)it.layer * a.n_unit + unit;
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    s_last = (atomicAdd(ticket, 1) == ns - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid == 0) *ticket = 0;
  const size_t item0 = (size_t)it.base + (size_t)unit * ns;
  const float* stat = a.part_stat + item0 * G * kStatStride;
  for (int h = tid; h < G; h += nt) {
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, __ldcg(stat + ((size_t)s * G + h) * kStatStride));
    float Lw = 0.f, Lt = 0.f;
    for (int s = 0; s < ns; ++s) {
      const float* st = stat + ((size_t)s * G + h) * kStatStride;
      const float ms = __ldcg(st);
      const float f = (ms > -INFINITY) ? exp2f(ms - M) : 0.f;
      Lw += __ldcg(st + 2) * f;
      if (lse_out) Lt += __ldcg(st + 1) * f;
    }
    s_mM[h] = M;
    s_mInv[h] = 1.f / Lw;
    if (lse_out) lse_out[h] = M + log2f(Lt);
  }
  __syncthreads();
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
  T* ob = reinterpret_cast<T*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G) * D;
  const float* po = a.part_o + item0 * G * D;
  for (int idx = tid; idx < G * D; idx += nt) {
    const int h = idx / D;
    float O = 0.f;
    for (int s = 0; s < ns; ++s) {
      const float ms = __ldcg(stat + ((size_t)s * G + h) * kStatStride);
      O += __ldcg(po + (size_t)s * G * D + idx) * ((ms > -INFINITY) ? exp2f(ms - s_mM[h]) : 0.f);
    }
    if (sizeof(T) == 2)
      reinterpret_cast<__nv_bfloat16*>(ob)[idx] = __float2bfloat16_rn(O * s_mInv[h]);
    else
      reinterpret_cast<float*>(ob)[idx] = O * s_mInv[h];
  }
}

}  // namespace sq
