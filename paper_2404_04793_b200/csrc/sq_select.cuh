// Block-level selection primitives for C_seq (Sections 2.2 / 5.1): an exact top-k by
// (score descending, position ascending) through radix select, and the "next victim" argmin.
// All routines are called by every thread of a 256-thread block.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sq {

constexpr int kSelThreads = 256;

// Monotone map from a finite float to an unsigned key (larger float -> larger key);
// -0 and +0 map to the same key.
__device__ __forceinline__ uint32_t score_key(float a) {
  uint32_t u = __float_as_uint(a);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelScratch {
  unsigned int hist[256];
  unsigned int warp_cnt[kSelThreads / 32];
  uint32_t prefix;
  unsigned int k_rem;
  unsigned int total;
  unsigned long long best[kSelThreads / 32];
  int best_slot[kSelThreads / 32];
};

// Radix select over the entries i in [0, n) with in_set(i): finds the key value T such that
// keeping every entry with key > T plus *n_at of the entries with key == T keeps exactly k
// (1 <= k <= number of entries in the set).  Returns T; *ties = entries with key == T.
template <class KeyFn, class SetFn>
__device__ uint32_t block_radix_select(SelScratch& sc, int n, unsigned int k, KeyFn key, SetFn in_set,
                                       unsigned int* n_at, unsigned int* ties) {
  const int tid = threadIdx.x;
  if (tid == 0) {
    sc.prefix = 0u;
    sc.k_rem = k;
  }
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += kSelThreads) sc.hist[i] = 0u;
    __syncthreads();
    const uint32_t prefix = sc.prefix;
    const uint32_t mask = (shift == 24) ? 0u : (0xffffffffu << (shift + 8));
    for (int i = tid; i < n; i += kSelThreads) {
      if (!in_set(i)) continue;
      uint32_t kk = key(i);
      if ((kk & mask) == prefix) atomicAdd(&sc.hist[(kk >> shift) & 0xffu], 1u);
    }
    __syncthreads();
    if (tid < 32) {
      // The digit is the highest d with (entries in bins above d) + hist[d] >= rem.  Lane l owns
      // the eight bins 255 - 8l ... 248 - 8l; a warp scan gives the entries above each lane's
      // bins, and the one lane whose bins hold the crossing walks them.
      const unsigned int rem = sc.k_rem;
      unsigned int c[8], sum = 0u;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        c[j] = sc.hist[255 - (8 * tid + j)];
        sum += c[j];
      }
      unsigned int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (tid >= o) incl += t;
      }
      unsigned int above = incl - sum;
      const bool here = (above < rem) && (incl >= rem);
      const bool none = (__ballot_sync(0xffffffffu, here) == 0u);  // rem beyond the set: digit 0, as a serial walk ends
      if (here || (none && tid == 31)) {
        int j = 0;
        for (; j < 7; ++j) {
          if (above + c[j] >= rem) break;
          above += c[j];
        }
        if (none) {  // lane 31: bins 7..0, the walk stops at bin 0 with everything above it counted
          j = 7;
          above = incl - c[7];
        }
        sc.k_rem = rem - above;
        sc.prefix = prefix | ((uint32_t)(255 - (8 * tid + j)) << shift);
        sc.total = c[j];
      }
    }
    __syncthreads();
  }
  *n_at = sc.k_rem;
  *ties = sc.total;
  uint32_t t = sc.prefix;
  __syncthreads();
  return t;
}

// Exclusive prefix count of `flag` over the block's threads (in thread order) plus the
// block total.
__device__ __forceinline__ int block_excl_count(SelScratch& sc, bool flag, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned int bal = __ballot_sync(0xffffffffu, flag);
  int within = __popc(bal & ((1u << lane) - 1u));
  if (lane == 0) sc.warp_cnt[warp] = __popc(bal);
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kSelThreads / 32; ++w) {
    int c = sc.warp_cnt[w];
    if (w < warp) base += c;
    tot += c;
  }
  __syncthreads();
  *total = tot;
  return base + within;
}

// Block-wide minimum of a 64-bit composite with its slot; every thread gets the winner.
__device__ __forceinline__ int block_argmin(SelScratch& sc, unsigned long long comp, int slot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long c2 = __shfl_xor_sync(0xffffffffu, comp, o);
    int s2 = __shfl_xor_sync(0xffffffffu, slot, o);
    if (c2 < comp) {
      comp = c2;
      slot = s2;
    }
  }
  if (lane == 0) {
    sc.best[warp] = comp;
    sc.best_slot[warp] = slot;
  }
  __syncthreads();
  unsigned long long bc = sc.best[0];
  int bs = sc.best_slot[0];
#pragma unroll
  for (int w = 1; w < kSelThreads / 32; ++w) {
    if (sc.best[w] < bc) {
      bc = sc.best[w];
      bs = sc.best_slot[w];
    }
  }
  __syncthreads();
  return bs;
}

// Eviction order of H2O among the tokens outside the recent window: the first to go has the
// smallest score and, on equal scores, the highest position.
__device__ __forceinline__ unsigned long long victim_rank(float acc, int pos) {
  return ((unsigned long long)score_key(acc) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)pos);
}

}  // namespace sq
