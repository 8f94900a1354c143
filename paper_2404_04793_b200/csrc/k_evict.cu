// C_seq(K, b) on its own (Section 4.1): compresses a layer's cache in place to a tighter
// budget.  One CTA per unit: decide which slots stay (Sliding Window / StreamingLLM by
// position, H2O by radix select over the scores), then close the gaps by moving the kept rows
// towards slot 0 in slot order, 32 slots at a time through shared memory (a row's new slot is
// never behind its old one, so a tile can be written once it has been read).
#include "sq_device.cuh"
#include "sq_internal.h"
#include "sq_select.cuh"

namespace sq {

constexpr int kTile = 32;
constexpr int kMaxVecPerRow = 32;  // 512-byte rows (fp32, head_dim 128)

__global__ void __launch_bounds__(kSelThreads) evict_kernel(EvictArgs a) {
  __shared__ SelScratch sc;
  __shared__ uint4 stage[kTile * 2 * kMaxVecPerRow];
  __shared__ int s_dst[kTile], s_pos[kTile];
  __shared__ float s_acc[kTile];
  const int unit = blockIdx.x, tid = threadIdx.x;
  const LayerDesc& lo = a.ld_old;
  const int cap = lo.cap, n = a.len, b = a.ld_new.b;
  int* pos = reinterpret_cast<int*>(a.pool + lo.pos_off) + (size_t)unit * cap;
  float* acc = reinterpret_cast<float*>(a.pool + lo.acc_off) + (size_t)unit * cap;
  const bool h2o = (a.policy == SQ_POLICY_H2O);
  if (n <= b) return;

  // --- which slots stay ---
  int recent_from;  // positions >= recent_from are kept as "recent"
  int n_sink = 0;
  uint32_t thr = 0u;
  int pos_thr = -1;
  bool heavy = false;
  if (a.policy == SQ_POLICY_SLIDING_WINDOW) {
    recent_from = a.n_tok - b;
  } else if (a.policy == SQ_POLICY_STREAMING_LLM) {
    n_sink = min(a.n_sink, b);
    recent_from = a.n_tok - (b - n_sink);
  } else {
    recent_from = a.n_tok - a.ld_new.b_recent;
    heavy = a.ld_new.b_heavy > 0;
    if (heavy) {
      auto key = [&](int i) { return score_key(acc[i]); };
      auto cand = [&](int i) { return pos[i] < recent_from; };
      unsigned int n_at, ties;
      thr = block_radix_select(sc, n, (unsigned)a.ld_new.b_heavy, key, cand, &n_at, &ties);
      if (ties == n_at) {
        pos_thr = 0x7fffffff;
      } else {
        auto pkey = [&](int i) { return 0x7fffffffu - (uint32_t)pos[i]; };
        auto tied = [&](int i) { return pos[i] < recent_from && score_key(acc[i]) == thr; };
        unsigned int d0, d1;
        uint32_t pt = block_radix_select(sc, n, n_at, pkey, tied, &d0, &d1);
        pos_thr = (int)(0x7fffffffu - pt);
      }
    }
  }

  // --- stable compaction ---
  const int vpr = a.row_bytes / 16;
  uint4* kb = reinterpret_cast<uint4*>(a.pool + lo.k_off) + (size_t)unit * cap * vpr;
  uint4* vb = reinterpret_cast<uint4*>(a.pool + lo.v_off) + (size_t)unit * cap * vpr;
  int written = 0;
  for (int s0 = 0; s0 < n; s0 += kTile) {
    if (tid < 32) {
      const int slot = s0 + tid;
      bool keep = false;
      int p = -1;
      float sc_v = 0.f;
      if (slot < n) {
        p = pos[slot];
        if (h2o) sc_v = acc[slot];
        if (p >= recent_from || p < n_sink) {
          keep = true;
        } else if (heavy) {
          uint32_t kk = score_key(sc_v);
          keep = (kk > thr) || (kk == thr && p <= pos_thr);
        }
      }
      const unsigned bal = __ballot_sync(0xffffffffu, keep);
      s_dst[tid] = keep ? written + __popc(bal & ((1u << tid) - 1u)) : -1;
      s_pos[tid] = p;
      s_acc[tid] = sc_v;
      if (tid == 0) sc.total = __popc(bal);
    }
    __syncthreads();
    for (int idx = tid; idx < kTile * 2 * vpr; idx += kSelThreads) {
      const int j = idx / (2 * vpr), r = idx - j * 2 * vpr;
      if (s_dst[j] < 0) continue;
      const size_t src = (size_t)(s0 + j) * vpr;
      stage[idx] = (r < vpr) ? kb[src + r] : vb[src + r - vpr];
    }
    __syncthreads();
    for (int idx = tid; idx < kTile * 2 * vpr; idx += kSelThreads) {
      const int j = idx / (2 * vpr), r = idx - j * 2 * vpr;
      const int d = s_dst[j];
      if (d < 0) continue;
      if (d >= b) {
        atomicOr(a.status, 4);
        continue;
      }
      if (r < vpr) kb[(size_t)d * vpr + r] = stage[idx];
      else vb[(size_t)d * vpr + r - vpr] = stage[idx];
      if (r == 0) {
        pos[d] = s_pos[j];
        if (h2o) acc[d] = s_acc[j];
      }
    }
    written += sc.total;
    __syncthreads();
  }
  if (tid == 0 && written != b) atomicOr(a.status, 8);

  // --- H2O: the slot the next append replaces ---
  if (h2o) {
    const int vthr = a.n_tok - a.ld_new.b_recent;
    unsigned long long best = ~0ull;
    int slot = -1;
    for (int i = tid; i < b; i += kSelThreads) {
      int p = pos[i];
      if (p <= vthr) {
        unsigned long long r = victim_rank(acc[i], p);
        if (r < best) {
          best = r;
          slot = i;
        }
      }
    }
    slot = block_argmin(sc, best, slot);
    if (tid == 0) reinterpret_cast<int*>(a.pool + lo.victim_off)[unit] = slot;
  }
}

cudaError_t launch_evict(const EvictArgs& a, cudaStream_t s) {
  if (a.row_bytes / 16 > kMaxVecPerRow) return cudaErrorInvalidValue;
  evict_kernel<<<a.n_unit, kSelThreads, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace sq
