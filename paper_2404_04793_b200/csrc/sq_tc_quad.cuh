// Quad form of the wide-group softmax role (decode_attn_tc_kernel).
#pragma once
#include "sq_tc.cuh"

namespace sq {
namespace tc {

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Quad form of the softmax role, for a tensor-memory quarter with at most 8 head rows (g = 71:
// rows 64..70): the 16-lane shapes give thread t the columns 8k + 2(t%4), +1 of row t/4, so the
// warp's 32 lanes share 8 rows instead of 24 of them idling through every exp2 of a row each.  A
// thread then holds a fourth of its row's weights.  Kept out of line so that the row form, which
// the other quarters run, keeps its registers (inlined, the second path cost the row form 15
// registers and 2-3 % of its speed).  Measured on the Falcon shape, one fused launch: Sliding
// Window -2 to -3 %, H2O -5 to -7 % per decode step; in the even-deal kernel the same change was
// 3-7 % slower, so that kernel keeps the row form for every quarter.
struct QuadCtx {
  uint32_t s_addr, p_addr, bar_sfree;
  float scale_log2;
  int lane;
};
// the row's maximum over the tile's valid tokens (log2 domain), equal in the row's four threads
static __device__ __noinline__ float quad_tile_max(const QuadCtx q, int n_valid) {
  const int qcol = q.lane & 3;
  float mx = -INFINITY;
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    uint32_t r[16];
    tmem_ld16x256_x4_nowait(q.s_addr + c * 32, r);
    tmem_wait_ld16(r);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int col = c * 32 + 8 * k + 2 * qcol;
      if (col < n_valid) mx = fmaxf(mx, __uint_as_float(r[4 * k]));
      if (col + 1 < n_valid) mx = fmaxf(mx, __uint_as_float(r[4 * k + 1]));
    }
  }
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
  return mx * q.scale_log2;
}
// this thread's 32 weights of its row for one tile (two per group of 8 columns): P to tensor
// memory, the thread's part of the sums to sums[0] (exact, H2O) and sums[1] (bf16-rounded);
// with EARLY, S is handed back before the last quarter is worked out unless the tile may have to be
// redone; returns whether it was
template <bool H2O, bool FULL, bool EARLY>
static __device__ __noinline__ bool quad_tile_weights(const QuadCtx q, float m_ref, int n_valid, float* sums) {
  const int qcol = q.lane & 3;
  const unsigned long long scale2 = f32x2(q.scale_log2, q.scale_log2), neg_m2 = f32x2(-m_ref, -m_ref);
  unsigned long long acc2 = f32x2(0.f, 0.f);
  float w_a = 0.f, w_b = 0.f;
  auto chunk = [&](const uint32_t (&r)[16], int c) {
    uint32_t pk[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int col = c * 32 + 8 * k + 2 * qcol;
      float p0, p1;
      f32x2_split(fma_f32x2(f32x2(__uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1])), scale2, neg_m2), p0, p1);
      p0 = ex2(p0);
      p1 = ex2(p1);
      if (!FULL) {
        if (col >= n_valid) p0 = 0.f;
        if (col + 1 >= n_valid) p1 = 0.f;
      }
      if (H2O) acc2 = add_f32x2(acc2, f32x2(p0, p1));
      const uint32_t u = pack_bf16x2(p0, p1);
      w_a = add_bf16_lo(w_a, u);
      w_b = add_bf16_hi(w_b, u);
      pk[2 * k] = u;       // row t/4, tokens col, col + 1
      pk[2 * k + 1] = 0u;  // row t/4 + 8: no head
    }
    tmem_st16x128_x4_u32(q.p_addr + c * 16, pk);
  };
  uint32_t ra[16], rb[16];
  tmem_ld16x256_x4_nowait(q.s_addr, ra);
  tmem_wait_ld16(ra);
  tmem_ld16x256_x4_nowait(q.s_addr + 32, rb);
  chunk(ra, 0);
  tmem_wait_ld16(rb);
  tmem_ld16x256_x4_nowait(q.s_addr + 64, ra);
  chunk(rb, 1);
  tmem_wait_ld16(ra);
  tmem_ld16x256_x4_nowait(q.s_addr + 96, rb);
  chunk(ra, 2);
  tmem_wait_ld16(rb);
  // as in the row form: S goes back early unless the tile may have to be redone
  float mx = __uint_as_float(rb[0]);
#pragma unroll
  for (int k = 0; k < 4; ++k) mx = max3(mx, __uint_as_float(rb[4 * k]), __uint_as_float(rb[4 * k + 1]));
  const bool safe = w_a + w_b <= 32768.f && fmaf(mx, q.scale_log2, -m_ref) <= 10.f;
  const bool released = EARLY && __all_sync(0xffffffffu, safe);
  if (released) {
    tc_fence_before();
    if (q.lane == 0) mbar_arrive(q.bar_sfree);
  }
  chunk(rb, 3);
  tmem_wait_st();
  float s0, s1;
  f32x2_split(acc2, s0, s1);
  sums[0] = s0 + s1;
  sums[1] = w_a + w_b;
  return released;
}

}  // namespace tc
}  // namespace sq
