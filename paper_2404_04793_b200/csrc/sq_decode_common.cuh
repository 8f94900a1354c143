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

// Work items of a launch are numbered descriptor by descriptor in the order of a.order (largest
// budget first), and within a descriptor as unit * n_split + split.  Without split-K every
// descriptor has n_unit items and the lookup is a division; with it the running item counts
// a.cum (kernel parameters: constant memory) are searched.
// UNIFORM: 1 = the launch is known to have no split-K (the search code is not even compiled in:
// the register-capped kernel keeps its budget), 0 = it is known to have it, -1 = read a.uniform.
template <int UNIFORM = -1, class Args = DecodeArgs>
__device__ __forceinline__ bool locate_desc(const Args& a, int k, ItemLoc& out) {
  if (k >= a.n_layer_total) return false;
  out.layer = a.order[k];
  if constexpr (UNIFORM == 1) {
    out.n_split = 1;
    out.base = k * a.n_unit;
  } else {
    if (UNIFORM < 0 && a.uniform) {
      out.n_split = 1;
      out.base = k * a.n_unit;
    } else {
      out.base = a.cum[k];
      out.n_split = (a.cum[k + 1] - out.base) / a.n_unit;
    }
  }
  out.local = 0;
  return true;
}
template <int UNIFORM = -1, class Args = DecodeArgs>
__device__ __forceinline__ bool locate(const Args& a, int idx, ItemLoc& out) {
  int k;
  if constexpr (UNIFORM == 1) {
    k = idx / a.n_unit;
  } else {
    if (UNIFORM < 0 && a.uniform) {
      k = idx / a.n_unit;
    } else {
      if (idx >= a.cum[a.n_layer_total]) return false;
      int lo = 0, hi = a.n_layer_total;  // cum[lo] <= idx < cum[hi]
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (a.cum[mid] <= idx) lo = mid;
        else hi = mid;
      }
      k = lo;
    }
  }
  if (!locate_desc<UNIFORM, Args>(a, k, out)) return false;
  out.local = idx - out.base;
  return true;
}

// Split-K merge without a second launch (policies without scores): every piece of a unit
// bumps the unit's ticket after its partials are written; the piece that arrives last reads
// all of them back (in piece order, so the result does not depend on who merges), writes the
// output and resets the ticket.  No piece ever waits for another.  With lse_out set, the merged
// log-sum-exp (log2 domain, from the unrounded weight sums) of every head is stored there too.
// The merge is run by a group of nt threads (tid = index within the group) that synchronise
// through sync(), which returns false when the group gives up.
template <typename T, int kBatch, typename Sync>
__device__ __forceinline__ void merge_if_last_group(const DecodeArgsBase& a, const ItemLoc& it, int unit, float* lse_out,
                                                    int tid, int nt, Sync sync) {
  __shared__ int s_last;
  __shared__ float s_mM[kMaxGroup], s_mInv[kMaxGroup];
  const int G = a.group, D = a.head_dim, ns = it.n_split;
  int* ticket = a.tickets + (size_t)it.layer * a.n_unit + unit;
  if (!sync()) return;  // the group's partials are written
  if (tid == 0) {
    __threadfence();
    s_last = (atomicAdd(ticket, 1) == ns - 1);
  }
  if (!sync()) return;
  if (!s_last) return;
  __threadfence();
  if (tid == 0) *ticket = 0;
  const size_t item0 = (size_t)it.base + (size_t)unit * ns;
  const float* stat = a.part_stat + item0 * G * kStatStride;
  // The partials were written by other SMs, so every read is an L2 round trip: the loops below
  // keep many independent loads in flight per thread instead of one dependent chain.
  for (int h = tid; h < G; h += nt) {
    float M = -INFINITY;
#pragma unroll 4
    for (int s = 0; s < ns; ++s) M = fmaxf(M, __ldcg(stat + ((size_t)s * G + h) * kStatStride));
    float Lw = 0.f, Lt = 0.f;
#pragma unroll 4
    for (int s = 0; s < ns; ++s) {
      const float4 st = __ldcg(reinterpret_cast<const float4*>(stat + ((size_t)s * G + h) * kStatStride));
      const float f = (st.x > -INFINITY) ? exp2f(st.x - M) : 0.f;
      Lw += st.z * f;
      Lt += st.y * f;
    }
    s_mM[h] = M;
    s_mInv[h] = 1.f / Lw;
    if (lse_out) lse_out[h] = M + log2f(Lt);
  }
  if (!sync()) return;
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
  T* ob = reinterpret_cast<T*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G) * D;
  const float* po = a.part_o + item0 * G * D;
  // four consecutive outputs (same head) per slot, kBatch slots per thread at a time
  const int n4 = G * D / 4;
  for (int base = tid; base < n4; base += nt * kBatch) {
    float4 O[kBatch];
    int h[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      O[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      const int i4 = base + u * nt;
      h[u] = (i4 < n4) ? (i4 * 4) / D : -1;
    }
    for (int s = 0; s < ns; ++s) {
      float4 v[kBatch];
      float ms[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        ms[u] = -INFINITY;
        if (h[u] >= 0) {
          v[u] = __ldcg(reinterpret_cast<const float4*>(po + (size_t)s * G * D) + base + u * nt);
          ms[u] = __ldcg(stat + ((size_t)s * G + h[u]) * kStatStride);
        }
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const float f = (ms[u] > -INFINITY) ? exp2f(ms[u] - s_mM[max(h[u], 0)]) : 0.f;
        O[u].x += v[u].x * f;
        O[u].y += v[u].y * f;
        O[u].z += v[u].z * f;
        O[u].w += v[u].w * f;
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      if (h[u] < 0) continue;
      const float inv = s_mInv[h[u]];
      const int i4 = base + u * nt;
      if (sizeof(T) == 2) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(O[u].x * inv, O[u].y * inv);
        __nv_bfloat162 hi = __floats2bfloat162_rn(O[u].z * inv, O[u].w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<unsigned*>(&lo);
        pk.y = *reinterpret_cast<unsigned*>(&hi);
        reinterpret_cast<uint2*>(ob)[i4] = pk;
      } else {
        reinterpret_cast<float4*>(ob)[i4] = make_float4(O[u].x * inv, O[u].y * inv, O[u].z * inv, O[u].w * inv);
      }
    }
  }
  // the shared scratch may be reused by the group's next merge only after everyone is done
  sync();
}

// The whole CTA merges.
template <typename T, int kBatch = 4>
__device__ __forceinline__ void merge_if_last(const DecodeArgsBase& a, const ItemLoc& it, int unit,
                                              float* lse_out = nullptr) {
  merge_if_last_group<T, kBatch>(a, it, unit, lse_out, (int)threadIdx.x, (int)blockDim.x, [] {
    __syncthreads();
    return true;
  });
}

}  // namespace sq
