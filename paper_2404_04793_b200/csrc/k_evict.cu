// C_seq(K, b) on its own (Section 4.1): compresses a layer's cache in place to a tighter
// budget.  One CTA per (unit, layer) of the call:
//   1. decide which slots stay (Sliding Window / StreamingLLM by position, H2O by radix select
//      over the scores) and record the decisions as a bitmask in shared memory with a running
//      count per 32 slots, so that any thread knows a row's new slot without touching memory;
//   2. close the gaps by moving the kept rows towards slot 0 in slot order.  A row's new slot
//      is never behind its old one, so a chunk of rows (with its positions and scores) is
//      fetched into shared memory with cp.async and stored to its new slots once it has
//      landed; chunks go in slot order, so a store never overwrites a row not yet read.
// The kernel is templated on the chunk size and on the number of chunks in flight per CTA.
// Measured (budgets halved on full caches, GB/s of rows read + written, Llama-2-7B- /
// Mistral-7B-H2O- / Llama-2-70B-shaped): 32 KB x 3 in flight (2 CTAs per SM) 2837 / 1868 / 3343;
// 16 KB x 3: 3727 / 2573 / 4513; 8 KB x 4: 3812 / 2776 / 4582; 16 KB x 2: 4180 / 2947 / 4901;
// 16 KB x 1: 4148 / 2987 / 5024; 32 KB x 1 (7 CTAs per SM): 4176 / 2982 / 5124.  The overlap
// that matters comes from many resident CTAs, not from a deep ring inside one, so the build
// uses one 32 KB chunk per CTA.
#include "sq_device.cuh"
#include "sq_internal.h"
#include "sq_select.cuh"

namespace sq {

namespace {
constexpr int kMaxVecPerRow = 32;       // 512-byte rows (fp32, head_dim 128)

__device__ __forceinline__ void cp_async(void* dst_smem, const void* src, int bytes16) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst_smem);
  if (bytes16)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src));
  else
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
__device__ __forceinline__ void cp_async_wait_all_but(int n) {
  switch (n) {
    case 0: asm volatile("cp.async.wait_group 0;"); break;
    case 1: asm volatile("cp.async.wait_group 1;"); break;
    case 2: asm volatile("cp.async.wait_group 2;"); break;
    case 3: asm volatile("cp.async.wait_group 3;"); break;
    case 4: asm volatile("cp.async.wait_group 4;"); break;
    default: asm volatile("cp.async.wait_group 5;"); break;
  }
}

// H2O: among the first b slots, the token outside the recent window (position <= last_old) that
// goes first: smallest score, on equal scores the highest position.  -1 if there is none.
__device__ __forceinline__ int h2o_next_victim(SelScratch& sc, const int* pos, const float* acc, int b, int last_old) {
  unsigned long long best = ~0ull;
  int slot = -1;
  for (int i = threadIdx.x; i < b; i += kSelThreads) {
    const int p = pos[i];
    if (p <= last_old) {
      const unsigned long long r = victim_rank(acc[i], p);
      if (r < best) {
        best = r;
        slot = i;
      }
    }
  }
  return block_argmin(sc, best, slot);
}
}  // namespace

// Dynamic shared memory: kStages chunks of rows, then per stage the chunk's positions and
// scores, then the keep bitmask (one word per 32 slots) and its running count.
template <int kChunkBytes, int kStages>
__global__ void __launch_bounds__(kSelThreads) evict_kernel(EvictArgs a) {
  constexpr int kMaxChunkRows = kChunkBytes / (2 * 128);  // 128-byte rows (bf16, head_dim 64)
  extern __shared__ __align__(16) unsigned char dyn[];
  __shared__ SelScratch sc;
  uint4* stage = reinterpret_cast<uint4*>(dyn);
  int* s_pos = reinterpret_cast<int*>(dyn + (size_t)kStages * kChunkBytes);
  float* s_acc = reinterpret_cast<float*>(s_pos + kStages * kMaxChunkRows);
  unsigned* s_mask = reinterpret_cast<unsigned*>(s_acc + kStages * kMaxChunkRows);
  const int unit = blockIdx.x, tid = threadIdx.x;
  const EvictLayer& ev = a.tab[blockIdx.y];
  const LayerDesc& lo = ev.ld_old;
  const LayerDesc& ln = ev.ld_new;
  const int cap = lo.cap, n = ev.len, b = ln.b, n_tok = ev.n_tok;
  const int n_words = (n + 31) / 32;
  int* s_before = reinterpret_cast<int*>(s_mask + (cap + 31) / 32);  // kept slots before each word
  int* pos = reinterpret_cast<int*>(a.pool + lo.pos_off) + (size_t)unit * cap;
  float* acc = reinterpret_cast<float*>(a.pool + lo.acc_off) + (size_t)unit * cap;
  const bool h2o = (a.policy == SQ_POLICY_H2O);
  if (n <= b) {
    // nothing to drop.  A cache that the new budget makes exactly full still needs the slot its
    // next append replaces (H2O): no earlier kernel has chosen one while it was below budget.
    if (h2o && n == b) {
      const int slot = h2o_next_victim(sc, pos, acc, b, n_tok - ln.b_recent);
      if (tid == 0) reinterpret_cast<int*>(a.pool + lo.victim_off)[unit] = slot;
    }
    return;
  }

  // --- which slots stay ---
  int recent_from;  // positions >= recent_from are kept as "recent"
  int n_sink = 0;
  uint32_t thr = 0u;
  int pos_thr = -1;
  bool heavy = false;
  if (a.policy == SQ_POLICY_SLIDING_WINDOW) {
    recent_from = n_tok - b;
  } else if (a.policy == SQ_POLICY_STREAMING_LLM) {
    n_sink = min(a.n_sink, b);
    recent_from = n_tok - (b - n_sink);
  } else {
    recent_from = n_tok - ln.b_recent;
    heavy = ln.b_heavy > 0;
    if (heavy) {
      auto key = [&](int i) { return score_key(acc[i]); };
      auto cand = [&](int i) { return pos[i] < recent_from; };
      unsigned int n_at, ties;
      thr = block_radix_select(sc, n, (unsigned)ln.b_heavy, key, cand, &n_at, &ties);
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

  // --- 1. keep bitmask and running counts ---
  for (int w0 = (tid >> 5); w0 < n_words; w0 += kSelThreads / 32) {
    const int slot = w0 * 32 + (tid & 31);
    bool keep = false;
    if (slot < n) {
      const int p = pos[slot];
      if (p >= recent_from || p < n_sink) {
        keep = true;
      } else if (heavy) {
        const uint32_t kk = score_key(acc[slot]);
        keep = (kk > thr) || (kk == thr && p <= pos_thr);
      }
    }
    const unsigned bal = __ballot_sync(0xffffffffu, keep);
    if ((tid & 31) == 0) s_mask[w0] = bal;
  }
  __syncthreads();
  if (tid < 32) {  // one warp scans the word counts
    int running = 0;
    for (int w0 = 0; w0 < n_words; w0 += 32) {
      const int w = w0 + tid;
      const int cnt = (w < n_words) ? __popc(s_mask[w]) : 0;
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (tid >= o) incl += t;
      }
      if (w < n_words) s_before[w] = running + incl - cnt;
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (tid == 0) sc.total = running;
  }
  __syncthreads();
  const int written = sc.total;
  auto kept = [&](int slot) { return (s_mask[slot >> 5] >> (slot & 31)) & 1u; };
  auto new_slot = [&](int slot) { return s_before[slot >> 5] + __popc(s_mask[slot >> 5] & ((1u << (slot & 31)) - 1u)); };

  // --- 2. stable compaction through the cp.async ring ---
  const int vpr = a.row_bytes / 16;                  // 8, 16 or 32 sixteen-byte pieces per row
  const int lv = 31 - __clz(2 * vpr);                // a slot's K and V pieces: 1 << lv
  const int rows = kChunkBytes / (2 * a.row_bytes);  // slots per chunk
  const int n_chunks = (n + rows - 1) / rows;
  uint4* kb = reinterpret_cast<uint4*>(a.pool + lo.k_off) + (size_t)unit * cap * vpr;
  uint4* vb = reinterpret_cast<uint4*>(a.pool + lo.v_off) + (size_t)unit * cap * vpr;
  auto issue = [&](int c) {
    if (c < n_chunks) {
      const int s0 = c * rows, st = c % kStages;
      uint4* sg = stage + (size_t)st * (kChunkBytes / 16);
      for (int idx = tid; idx < rows * 2 * vpr; idx += kSelThreads) {
        const int j = idx >> lv, r = idx & ((1 << lv) - 1);
        const int slot = s0 + j;
        if (slot >= n || !kept(slot)) continue;
        const size_t src = (size_t)slot * vpr;
        cp_async(sg + idx, (r < vpr) ? (kb + src + r) : (vb + src + r - vpr), 1);
        if (r == 0) {
          cp_async(s_pos + st * kMaxChunkRows + j, pos + slot, 0);
          if (h2o) cp_async(s_acc + st * kMaxChunkRows + j, acc + slot, 0);
        }
      }
    }
    cp_async_commit();  // one group per chunk, empty past the end, so the wait counts stay aligned
  };
  // chunks before the first kept row that moves hold nothing to do
  int c_begin = n_chunks;
  for (int w = 0; w < n_words; ++w) {
    const unsigned m = s_mask[w];
    if (s_before[w] + __popc(m) != (w + 1) * 32 || w == n_words - 1) {  // first word with a gap (or the last)
      c_begin = (w * 32) / rows;
      break;
    }
  }
  for (int c = c_begin; c < c_begin + kStages - 1; ++c) issue(c);
  for (int c = c_begin; c < n_chunks; ++c) {
    issue(c + kStages - 1);
    cp_async_wait_all_but(kStages - 1);
    __syncthreads();
    const int s0 = c * rows, st = c % kStages;
    const uint4* sg = stage + (size_t)st * (kChunkBytes / 16);
    for (int idx = tid; idx < rows * 2 * vpr; idx += kSelThreads) {
      const int j = idx >> lv, r = idx & ((1 << lv) - 1);
      const int slot = s0 + j;
      if (slot >= n || !kept(slot)) continue;
      const int d = new_slot(slot);
      if (d >= b) {
        atomicOr(a.status, 4);
        continue;
      }
      if (r < vpr) kb[(size_t)d * vpr + r] = sg[idx];
      else vb[(size_t)d * vpr + r - vpr] = sg[idx];
      if (r == 0) {
        pos[d] = s_pos[st * kMaxChunkRows + j];
        if (h2o) acc[d] = s_acc[st * kMaxChunkRows + j];
      }
    }
    __syncthreads();  // the stage is refilled by the next iteration's loads
  }
  if (tid == 0 && written != b) atomicOr(a.status, 8);

  // --- H2O: the slot the next append replaces ---
  if (h2o) {
    const int slot = h2o_next_victim(sc, pos, acc, b, n_tok - ln.b_recent);
    if (tid == 0) reinterpret_cast<int*>(a.pool + lo.victim_off)[unit] = slot;
  }
}

template <int kChunkBytes, int kStages>
static cudaError_t launch_evict_cfg(const EvictArgs& a, cudaStream_t s) {
  constexpr int kMaxChunkRows = kChunkBytes / (2 * 128);
  const size_t words = ((size_t)a.max_cap + 31) / 32;
  const size_t smem = (size_t)kStages * kChunkBytes + (size_t)kStages * kMaxChunkRows * 8 + words * 8;
  if (smem > 200 * 1024) return cudaErrorInvalidValue;  // caches beyond ~1.4 M slots per unit
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(evict_kernel<kChunkBytes, kStages>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  evict_kernel<kChunkBytes, kStages><<<dim3(a.n_unit, a.n_layers), kSelThreads, smem, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_evict(const EvictArgs& a, cudaStream_t s) {
  if (a.row_bytes / 16 > kMaxVecPerRow || a.row_bytes < 128 || (a.row_bytes & (a.row_bytes - 1)))
    return cudaErrorInvalidValue;
  return launch_evict_cfg<32 * 1024, 1>(a, s);
}

}  // namespace sq
