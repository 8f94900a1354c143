// H2O bookkeeping of one unit after its attention is final (Algorithm 1, step 19 onwards for
// the heavy-hitter policy): every kept token's score grows by the probability it received,
// summed over the group's heads in head order, and if the cache is full the slot the next
// append replaces is chosen.  Called by all threads of a block (at most 256) once the heads'
// maxima and reciprocal sums are in shared memory and the unit's logits are in global memory.
#pragma once
#include "sq_internal.h"
#include "sq_select.cuh"

namespace sq {

__device__ __forceinline__ void h2o_update_unit(const DecodeArgs& a, const LayerDesc* ldp, int unit, const float* s_M,
                                                const float* s_invL, SelScratch& sc) {
  const int tid = threadIdx.x, nt = blockDim.x, G = a.group, b = ldp->b, cap = ldp->cap;
  const int len = min(a.n_tok + 1, b);
  const bool full = (len == b);
  const int thr = a.n_tok + 1 - ldp->b_recent;  // next step: positions <= thr are outside the recent window
  const int* pos = reinterpret_cast<const int*>(a.pool + ldp->pos_off) + (size_t)unit * cap;
  float* acc = reinterpret_cast<float*>(a.pool + ldp->acc_off) + (size_t)unit * cap;
  const float* logit = a.logits + ldp->logit_off + (size_t)unit * cap * G;
  unsigned long long best = ~0ull;
  int best_slot = -1;
  for (int slot = tid; slot < len; slot += nt) {
    float gain = 0.f;
    for (int h = 0; h < G; ++h) gain += exp2f(logit[(size_t)slot * G + h] - s_M[h]) * s_invL[h];
    const float v = acc[slot] + gain;
    acc[slot] = v;
    if (full) {
      const int p = pos[slot];
      if (p <= thr) {
        const unsigned long long r = victim_rank(v, p);
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

}  // namespace sq
