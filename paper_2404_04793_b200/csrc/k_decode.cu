// Decode step of Algorithm 1 (steps 15-22) for a range of layers in one launch: append the new
// token into the slot C_seq frees, attend over the kept slots (split-K flash-decode, all query
// heads of a KV head share one pass over K/V), and for H2O add the received probabilities to
// the per-token scores and choose the slot the next append will reuse.
#include <cstdlib>
#include <cstring>

#include "sq_device.cuh"
#include "sq_internal.h"
#include "sq_select.cuh"
#include "sq_decode_common.cuh"

namespace sq {

// One CTA (NW warps) per (layer, unit, split).  A K or V row is D*sizeof(T) bytes = LPR lanes
// x 16 bytes, so a warp reads 32/LPR consecutive rows per load instruction, fully coalesced.
// Each lane keeps its 16-byte slice of up to GT query heads (pre-scaled by log2(e)/sqrt(d))
// and of their output accumulators in fp32; logits are reduced over the LPR lanes by
// shuffles, and the softmax runs online in the log2 domain over batches of U rows.
// UNIFORM: the launch has no split-K (see locate()).
// NW = 4 everywhere but in the build for launches of few, unsplit units (one layer of a small
// batch): those leave most warp slots of the GPU empty with 4 warps per unit, and each warp then
// walks its rows in a chain of dependent round trips to memory; 16 warps per unit make the chain
// a quarter as long.
template <typename T, int D, int GT, int UNIFORM, class Args, int NW = 4>
__global__ void __launch_bounds__(NW * 32, NW == 4 ? (GT == 1 ? (UNIFORM == 1 ? 8 : 6) : 1) : 2) decode_attn_kernel(Args a) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;   // lanes per row
  constexpr int RPW = 32 / LPR;  // rows per warp per load
  constexpr int U = 4;           // rows in flight per lane
  __shared__ float sm_o[NW][GT][D];
  __shared__ float sm_m[NW][GT], sm_l[NW][GT];

  ItemLoc it;
  if (!locate<UNIFORM, Args>(a, blockIdx.x, it)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane % LPR, rg = lane / LPR;
  const LayerDesc* ldp = a.layers + it.layer;
  const int b = ldp->b, cap = ldp->cap;
  const int unit = it.local / it.n_split, split = it.local - unit * it.n_split;
  const int len = min(a.n_tok + 1, b);
  const bool h2o = (a.policy == SQ_POLICY_H2O);
  int w;  // slot that receives the new token
  if (h2o) {
    w = (a.n_tok < b) ? a.n_tok : reinterpret_cast<const int*>(a.pool + ldp->victim_off)[unit];
    if (w < 0 || w >= b) {
      if (tid == 0) atomicOr(a.status, 2);
      w = 0;
    }
  } else {
    w = ring_slot(a.n_tok, b, ldp->ring_base, ldp->ring_origin);
  }
  const int t0 = split * a.split_tokens, t1 = min(len, t0 + a.split_tokens);
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
  const T* Kb = reinterpret_cast<const T*>(a.pool + ldp->k_off) + (size_t)unit * cap * D;
  const T* Vb = reinterpret_cast<const T*>(a.pool + ldp->v_off) + (size_t)unit * cap * D;
  const T* qb = reinterpret_cast<const T*>(a.q) + (tok * a.n_q_head + (size_t)kvh * a.group) * D;
  const T* kn = reinterpret_cast<const T*>(a.k_new) + (tok * a.n_kv_head + kvh) * D;
  const T* vn = reinterpret_cast<const T*>(a.v_new) + (tok * a.n_kv_head + kvh) * D;
  T* ob = reinterpret_cast<T*>(a.out) + (tok * a.n_q_head + (size_t)kvh * a.group) * D;
  float* logit = a.logits + ldp->logit_off + (size_t)unit * cap * a.group;  // [slot][group]
  float* stat = a.part_stat + (size_t)blockIdx.x * a.group * kStatStride;
  float* po = a.part_o + (size_t)blockIdx.x * a.group * D;

  for (int hb = 0; hb < a.group; hb += GT) {
    float qr[GT][EPV], o[GT][EPV], m[GT], l[GT];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
      m[g] = -INFINITY;
      l[g] = 0.f;
      if (hb + g < a.group) {
        widen<T>(ld_stream(qb + (size_t)(hb + g) * D + sub * EPV), qr[g]);
      } else {
#pragma unroll
        for (int e = 0; e < EPV; ++e) qr[g][e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < EPV; ++e) {
        qr[g][e] *= a.scale_log2;
        o[g][e] = 0.f;
      }
    }
    for (int r0 = t0 + warp * (U * RPW); r0 < t1; r0 += NW * U * RPW) {
      uint4 kq[U], vq[U];
      bool ok[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int row = r0 + u * RPW + rg;
        ok[u] = row < t1;
        const int rr = ok[u] ? row : t0;
        const T* kp = (rr == w) ? kn : Kb + (size_t)rr * D;
        const T* vp = (rr == w) ? vn : Vb + (size_t)rr * D;
        kq[u] = ld_stream(kp + sub * EPV);
        vq[u] = ld_stream(vp + sub * EPV);
      }
      float s[U][GT];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float kf[EPV];
        widen<T>(kq[u], kf);
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          float d = 0.f;
#pragma unroll
          for (int e = 0; e < EPV; ++e) d = fmaf(qr[g][e], kf[e], d);
#pragma unroll
          for (int off = LPR / 2; off > 0; off >>= 1) d += __shfl_xor_sync(kFull, d, off);
          s[u][g] = ok[u] ? d : -INFINITY;
        }
      }
      if (h2o) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (!ok[u]) continue;
          const int row = r0 + u * RPW + rg;
#pragma unroll
          for (int g = 0; g < GT; ++g)
            if (sub == g && hb + g < a.group) logit[(size_t)row * a.group + hb + g] = s[u][g];
        }
      }
      float mn[GT];
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        float mx = s[0][g];
#pragma unroll
        for (int u = 1; u < U; ++u) mx = fmaxf(mx, s[u][g]);
        mn[g] = fmaxf(m[g], mx);
        if (mn[g] > -INFINITY) {
          const float corr = exp2f(m[g] - mn[g]);
          l[g] *= corr;
#pragma unroll
          for (int e = 0; e < EPV; ++e) o[g][e] *= corr;
          m[g] = mn[g];
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float vf[EPV];
        widen<T>(vq[u], vf);
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          const float p = (s[u][g] > -INFINITY) ? exp2f(s[u][g] - mn[g]) : 0.f;
          l[g] += p;
#pragma unroll
          for (int e = 0; e < EPV; ++e) o[g][e] = fmaf(p, vf[e], o[g][e]);
        }
      }
    }
    // merge the row groups of the warp
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        const float m2 = __shfl_xor_sync(kFull, m[g], off);
        const float l2 = __shfl_xor_sync(kFull, l[g], off);
        const float mx = fmaxf(m[g], m2);
        const float f1 = (m[g] > -INFINITY) ? exp2f(m[g] - mx) : 0.f;
        const float f2 = (m2 > -INFINITY) ? exp2f(m2 - mx) : 0.f;
        l[g] = l[g] * f1 + l2 * f2;
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
          const float o2 = __shfl_xor_sync(kFull, o[g][e], off);
          o[g][e] = o[g][e] * f1 + o2 * f2;
        }
        m[g] = mx;
      }
    }
    if (rg == 0) {
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        if (sub == 0) {
          sm_m[warp][g] = m[g];
          sm_l[warp][g] = l[g];
        }
#pragma unroll
        for (int e = 0; e < EPV; ++e) sm_o[warp][g][sub * EPV + e] = o[g][e];
      }
    }
    __syncthreads();
    for (int idx = tid; idx < GT * D; idx += NW * 32) {
      const int g = idx / D, e = idx - g * D, h = hb + g;
      if (h >= a.group) continue;
      float M = -INFINITY;
#pragma unroll
      for (int ww = 0; ww < NW; ++ww) M = fmaxf(M, sm_m[ww][g]);
      float L = 0.f, O = 0.f;
#pragma unroll
      for (int ww = 0; ww < NW; ++ww) {
        const float mw = sm_m[ww][g];
        const float f = (mw > -INFINITY) ? exp2f(mw - M) : 0.f;
        L += sm_l[ww][g] * f;
        O += sm_o[ww][g][e] * f;
      }
      if (it.n_split == 1)
        ob[(size_t)h * D + e] = narrow<T>(O / L);
      else
        po[(size_t)h * D + e] = O;
      if (e == 0) {
        stat[h * kStatStride] = M;
        stat[h * kStatStride + 1] = L;
        stat[h * kStatStride + 2] = L;
      }
    }
    __syncthreads();
  }

  // the CTA whose range holds slot w stores the new token (nobody reads that slot this step)
  if (w >= t0 && w < t1) {
    if (tid < 2 * LPR) {
      const bool is_v = tid >= LPR;
      const int v = is_v ? tid - LPR : tid;
      const T* src = (is_v ? vn : kn) + v * EPV;
      T* dst = const_cast<T*>(is_v ? Vb : Kb) + (size_t)w * D + v * EPV;
      *reinterpret_cast<uint4*>(dst) = ld_stream(src);
    }
    if (tid == 64) {
      reinterpret_cast<int*>(a.pool + ldp->pos_off)[(size_t)unit * cap + w] = a.n_tok;
      if (h2o) reinterpret_cast<float*>(a.pool + ldp->acc_off)[(size_t)unit * cap + w] = 0.f;
    }
  }
  if (!h2o && it.n_split > 1) merge_if_last<T, (GT == 1 ? 2 : 4)>(a, it, unit);
}

// One CTA per (layer, unit): merges the split-K partials into the output and, for H2O, adds
// each kept token's probabilities (summed over the group's heads in head order) to its score
// and picks the slot the next append replaces.
template <typename T>
__global__ void __launch_bounds__(kSelThreads, 5) decode_combine_kernel(DecodeArgs a) {
  __shared__ SelScratch sc;
  __shared__ __align__(16) float s_M[kMaxGroup], s_invL[kMaxGroup], s_invLw[kMaxGroup];
  // one CTA per (descriptor of the launch, unit)
  const int unit = blockIdx.x % a.n_unit;
  ItemLoc it;
  if (!locate_desc(a, blockIdx.x / a.n_unit, it)) return;
  const int layer = it.layer;
  const int tid = threadIdx.x, D = a.head_dim, G = a.group, ns = it.n_split;
  const LayerDesc* ldp = a.layers + layer;
  const int b = ldp->b, cap = ldp->cap;
  const size_t item0 = (size_t)it.base + (size_t)unit * ns;
  const float* stat = a.part_stat + item0 * G * kStatStride;
  for (int h = tid; h < G; h += kSelThreads) {
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, stat[((size_t)s * G + h) * kStatStride]);
    float L = 0.f, Lw = 0.f;
    for (int s = 0; s < ns; ++s) {
      const float* st = stat + ((size_t)s * G + h) * kStatStride;
      const float f = (st[0] > -INFINITY) ? exp2f(st[0] - M) : 0.f;
      L += st[1] * f;
      Lw += st[2] * f;
    }
    s_M[h] = M;
    s_invL[h] = 1.f / L;     // normaliser of the probabilities (H2O scores)
    s_invLw[h] = 1.f / Lw;   // normaliser matching the weights the output was accumulated with
  }
  __syncthreads();
  if (ns > 1) {
    const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
    const size_t tok = (size_t)(layer - a.layer_begin) * a.batch + seq;
    T* ob = reinterpret_cast<T*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G) * D;
    const float* po = a.part_o + item0 * G * D;
    for (int idx = tid; idx < G * D; idx += kSelThreads) {
      const int h = idx / D;
      float O = 0.f;
      for (int s = 0; s < ns; ++s) {
        const float ms = stat[((size_t)s * G + h) * kStatStride];
        O += po[(size_t)s * G * D + idx] * ((ms > -INFINITY) ? exp2f(ms - s_M[h]) : 0.f);
      }
      ob[idx] = narrow<T>(O * s_invLw[h]);
    }
  }
  if (a.policy != SQ_POLICY_H2O) return;
  const int len = min(a.n_tok + 1, b);
  const bool full = (len == b);
  const int thr = a.n_tok + 1 - ldp->b_recent;  // next step: positions <= thr are outside the recent window
  const int* pos = reinterpret_cast<const int*>(a.pool + ldp->pos_off) + (size_t)unit * cap;
  float* acc = reinterpret_cast<float*>(a.pool + ldp->acc_off) + (size_t)unit * cap;
  const float* logit = a.logits + ldp->logit_off + (size_t)unit * cap * G;
  unsigned long long best = ~0ull;
  int best_slot = -1;
  // four slots per thread in flight: their logits, score and position loads are independent
  constexpr int kIl = 4;
  for (int s0 = tid; s0 < len; s0 += kIl * kSelThreads) {
    float gain[kIl], old[kIl];
    int p[kIl];
#pragma unroll
    for (int u = 0; u < kIl; ++u) {
      const int slot = s0 + u * kSelThreads;
      gain[u] = 0.f;
      old[u] = 0.f;
      p[u] = 0x7fffffff;
      if (slot < len) {
        old[u] = acc[slot];
        if (full) p[u] = pos[slot];
      }
    }
    if ((G & 3) == 0) {
      for (int h = 0; h < G; h += 4) {
        const float4 m4 = *reinterpret_cast<const float4*>(s_M + h), i4 = *reinterpret_cast<const float4*>(s_invL + h);
#pragma unroll
        for (int u = 0; u < kIl; ++u) {
          const int slot = s0 + u * kSelThreads;
          if (slot < len) {
            const float4 l4 = *reinterpret_cast<const float4*>(logit + (size_t)slot * G + h);
            gain[u] += exp2f(l4.x - m4.x) * i4.x;
            gain[u] += exp2f(l4.y - m4.y) * i4.y;
            gain[u] += exp2f(l4.z - m4.z) * i4.z;
            gain[u] += exp2f(l4.w - m4.w) * i4.w;
          }
        }
      }
    } else {
      // odd group sizes: one slot at a time, so a slot's G consecutive logits stay in L1
#pragma unroll 1
      for (int u = 0; u < kIl; ++u) {
        const int slot = s0 + u * kSelThreads;
        if (slot >= len) continue;
        float g1 = 0.f;
        for (int h = 0; h < G; ++h) g1 += exp2f(logit[(size_t)slot * G + h] - s_M[h]) * s_invL[h];
        gain[u] = g1;
      }
    }
#pragma unroll
    for (int u = 0; u < kIl; ++u) {
      const int slot = s0 + u * kSelThreads;
      if (slot >= len) continue;
      const float v = old[u] + gain[u];
      acc[slot] = v;
      if (full && p[u] <= thr) {
        const unsigned long long r = victim_rank(v, p[u]);
        if (r < best) {
          best = r;
          best_slot = slot;
        }
      }
    }
  }
  if (full) {
    best_slot = block_argmin(sc, best, best_slot);
    if (tid == 0) reinterpret_cast<int*>(a.pool + ldp->victim_off)[unit] = best_slot;
  }
}

// H2O bookkeeping for launches without split-K and groups of at most 32 heads: one WARP per
// (descriptor, unit) instead of one CTA.  A unit holds a few hundred to a few thousand slots,
// too little to occupy 256 threads for longer than the block's set-up and reductions take; as
// warps, every unit of a step is resident at once and nothing synchronises beyond a warp.
// The arithmetic per slot (head order of the sum, the reciprocal of the row sum) is that of
// decode_combine_kernel, so both give the same bits.
constexpr int kWarpUpdWarps = 8;
__global__ void __launch_bounds__(32 * kWarpUpdWarps, 3) h2o_update_warp_kernel(DecodeArgsBase a) {
  __shared__ __align__(16) float s_M[kWarpUpdWarps][32], s_invL[kWarpUpdWarps][32];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int idx = blockIdx.x * kWarpUpdWarps + wib;
  if (idx >= a.n_layer_total * a.n_unit) return;
  const int k = idx / a.n_unit, unit = idx - k * a.n_unit;
  const int layer = a.order[k], G = a.group;
  const LayerDesc* ldp = a.layers + layer;
  const int b = ldp->b, cap = ldp->cap;
  const float* stat = a.part_stat + ((size_t)k * a.n_unit + unit) * G * kStatStride;
  if (lane < G) {
    const float2 ml = *reinterpret_cast<const float2*>(stat + lane * kStatStride);
    s_M[wib][lane] = ml.x;
    s_invL[wib][lane] = 1.f / ml.y;
  }
  __syncwarp();
  const float* wM = s_M[wib];
  const float* wI = s_invL[wib];
  const int len = min(a.n_tok + 1, b);
  const bool full = (len == b);
  const int thr = a.n_tok + 1 - ldp->b_recent;  // next step: positions <= thr are outside the recent window
  const int* pos = reinterpret_cast<const int*>(a.pool + ldp->pos_off) + (size_t)unit * cap;
  float* acc = reinterpret_cast<float*>(a.pool + ldp->acc_off) + (size_t)unit * cap;
  const float* logit = a.logits + ldp->logit_off + (size_t)unit * cap * G;
  unsigned long long best = ~0ull;
  int best_slot = -1;
  constexpr int kIl = 8;  // slots per lane in flight: their logits, score and position loads are independent
  for (int s0 = lane; s0 < len; s0 += kIl * 32) {
    float gain[kIl], old[kIl];
    int p[kIl];
#pragma unroll
    for (int u = 0; u < kIl; ++u) {
      const int slot = s0 + u * 32;
      gain[u] = 0.f;
      old[u] = 0.f;
      p[u] = 0x7fffffff;
      if (slot < len) {
        old[u] = acc[slot];
        if (full) p[u] = pos[slot];
      }
    }
    if ((G & 3) == 0) {
      for (int h = 0; h < G; h += 4) {
        const float4 m4 = *reinterpret_cast<const float4*>(wM + h), i4 = *reinterpret_cast<const float4*>(wI + h);
        float4 l4[kIl];
#pragma unroll
        for (int u = 0; u < kIl; ++u) {
          const int slot = s0 + u * 32;
          l4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (slot < len) l4[u] = *reinterpret_cast<const float4*>(logit + (size_t)slot * G + h);
        }
#pragma unroll
        for (int u = 0; u < kIl; ++u) {
          gain[u] += exp2f(l4[u].x - m4.x) * i4.x;
          gain[u] += exp2f(l4[u].y - m4.y) * i4.y;
          gain[u] += exp2f(l4[u].z - m4.z) * i4.z;
          gain[u] += exp2f(l4[u].w - m4.w) * i4.w;
        }
      }
    } else {
#pragma unroll 1
      for (int u = 0; u < kIl; ++u) {
        const int slot = s0 + u * 32;
        if (slot >= len) continue;
        float g1 = 0.f;
        for (int h = 0; h < G; ++h) g1 += exp2f(logit[(size_t)slot * G + h] - wM[h]) * wI[h];
        gain[u] = g1;
      }
    }
#pragma unroll
    for (int u = 0; u < kIl; ++u) {
      const int slot = s0 + u * 32;
      if (slot >= len) continue;
      const float v = old[u] + gain[u];
      acc[slot] = v;
      if (full && p[u] <= thr) {
        const unsigned long long r = victim_rank(v, p[u]);
        if (r < best) {
          best = r;
          best_slot = slot;
        }
      }
    }
  }
  if (full) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long c2 = __shfl_xor_sync(kFull, best, o);
      const int s2 = __shfl_xor_sync(kFull, best_slot, o);
      if (c2 < best) {
        best = c2;
        best_slot = s2;
      }
    }
    if (lane == 0) reinterpret_cast<int*>(a.pool + ldp->victim_off)[unit] = best_slot;
  }
}

template <typename T, int D>
static void launch_attn_g(const DecodeArgs& a, int n_items, cudaStream_t s) {
  if (a.group == 1) {
    // the register-capped kernel gets its own build for launches without split-K
    // few unsplit units (at most two 16-warp CTAs per SM, all resident at once): 16 warps per unit
    if (a.uniform && n_items <= 2 * 148) decode_attn_kernel<T, D, 1, 1, DecodeArgsBase, 16><<<n_items, 512, 0, s>>>(a);
    else if (a.uniform) decode_attn_kernel<T, D, 1, 1, DecodeArgsBase><<<n_items, 128, 0, s>>>(a);  // sliced: no table
    else decode_attn_kernel<T, D, 1, 0, DecodeArgs><<<n_items, 128, 0, s>>>(a);
  } else if (a.group <= 4) {
    decode_attn_kernel<T, D, 4, -1, DecodeArgs><<<n_items, 128, 0, s>>>(a);
  } else {
    decode_attn_kernel<T, D, 8, -1, DecodeArgs><<<n_items, 128, 0, s>>>(a);
  }
}

// Which attention kernel serves a shape: wide bf16 groups at head_dim 64 go to the tcgen05
// kernel, other grouped bf16 heads to the mma.sync kernel, everything else (fp32, one query head
// per KV head, shapes those do not cover) to the fp32-pipe kernel.
cudaError_t launch_decode(const DecodeArgs& a, int dtype, int n_items, bool need_combine, size_t pool_bytes,
                          size_t q_rows, const int* desc_tiles, cudaStream_t s) {
  if (n_items <= 0) return cudaSuccess;
  bool done = false;
  if (dtype == SQ_BF16 && a.group > 32) {
    // long units that do not fill the CTA slots: the even deal; else one CTA per unit and piece
    cudaError_t e = launch_decode_attn_tc_stream(a, desc_tiles, pool_bytes, q_rows, s);
    if (e == cudaErrorNotSupported) e = launch_decode_attn_tc(a, n_items, pool_bytes, q_rows, s);
    if (e == cudaSuccess) {
      // H2O: the attention kernel left the row log-sum-exps; the scores and the next victim come
      // from a second pass over K instead of logits carried through memory
      if (a.policy == SQ_POLICY_H2O) return launch_h2o_gain_tc(a, n_items, pool_bytes, q_rows, s);
      done = true;
    } else if (e != cudaErrorNotSupported) {
      return e;
    }
  }
  // every other kernel needs the per-slot logits for H2O: a context sized for the tcgen05 pair
  // does not hold them, and nothing may fall back silently
  if (!done && a.policy == SQ_POLICY_H2O && !a.has_logits) return cudaErrorNotSupported;
  if (!done && dtype == SQ_BF16 && a.group > 1) {
    cudaError_t e = launch_decode_attn_mma(a, n_items, s);
    if (e == cudaSuccess) done = true;
    else if (e != cudaErrorNotSupported) return e;
  }
  if (done) {
  } else if (dtype == SQ_F32) {
    if (a.head_dim == 64) launch_attn_g<float, 64>(a, n_items, s);
    else launch_attn_g<float, 128>(a, n_items, s);
  } else {
    if (a.head_dim == 64) launch_attn_g<__nv_bfloat16, 64>(a, n_items, s);
    else launch_attn_g<__nv_bfloat16, 128>(a, n_items, s);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || !need_combine) return e;
  const int n_cta = a.n_layer_total * a.n_unit;
  // More units than the CTA-per-unit kernel holds in one wave (5 CTAs per SM), and nothing to
  // merge: only the scores and the next victim remain, one warp per unit.  Smaller launches
  // (one layer of a small batch) finish sooner with a CTA per unit.
  if (a.policy == SQ_POLICY_H2O && a.uniform && a.group <= 32 && n_cta > 148 * 5) {
    h2o_update_warp_kernel<<<(n_cta + kWarpUpdWarps - 1) / kWarpUpdWarps, 32 * kWarpUpdWarps, 0, s>>>(a);
    return cudaGetLastError();
  }
  if (dtype == SQ_F32)
    decode_combine_kernel<float><<<n_cta, kSelThreads, 0, s>>>(a);
  else
    decode_combine_kernel<__nv_bfloat16><<<n_cta, kSelThreads, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace sq
