// Decode attention for wide multi-query groups (33..128 query heads per KV head, head_dim 64,
// bf16) on the 5th-generation tensor cores.  With g = 71 (Falcon-shaped MQA) the step needs
// g flop per byte of K/V -- hundreds of TFLOP/s at HBM speed -- so both contractions run as
// tcgen05.mma with accumulators in tensor memory:
//   S[head rows x 128 tokens] = Q K_tile^T      (Q, K tile in shared memory, K-major)
//   O[head rows x 64]        += P V_tile         (P bf16 in TENSOR memory, V tile MN-major)
// One CTA per (layer, unit, split), two CTAs per SM; per 128-token tile the roles are
//   warp 0      TMA: K and V tiles into a ring of stages (128-byte swizzle, every CTA its own tiles)
//   warp 1      MMA issue (one thread)
//   warps 2..5  thread = one head row (TMEM lane): p = exp2(s*scale - m_ref) straight from the
//               accumulator row, no shuffles; P is packed to bf16 and stored back to tensor
//               memory as the A operand of the second MMA.  A quarter of tensor memory with at
//               most 8 head rows (g = 71: the third) is worked by its warp in quads instead, four
//               threads to a row (sq_tc_quad.cuh)
// Measured on B200: one M=128, K=16 MMA costs 45-48 cycles for N <= 64 and 64 cycles for N = 128,
// and operands read from shared memory compete with the TMA writes for its 128 B/clk; keeping P
// in tensor memory (64 columns) removes 56 KB of shared-memory traffic per tile.  Inside the
// kernel, two CTAs sharing the pipe, an MMA holds the issuing thread for about 80 cycles and a
// tcgen05.commit for about 180.
// A row's reference m_ref is its maximum over the first tile; later tiles reuse it and only
// when a weight would exceed 2^16 is the reference moved (O and the sums rescaled through
// tcgen05.ld/st, the tile redone): every weight stays finite and the result is that of the
// exact softmax.  Every barrier wait is bounded.
// What bounds the kernel (measured on B200 with per-tile clock stamps and with copies that leave
// work out): a softmax warp needs 1250 cycles per tile alone on its scheduler and 2150-2250 when
// it shares it with the other CTA's (the special-function unit: 128 exp2 per row and tile at one
// warp instruction per 8 cycles), against 2780 cycles of HBM time per pair of tiles at 1.9 GHz;
// a polynomial exp2 on the FMA pipe for a part of the weights was slower at every share tried.
// Streaming K and V alone (no products, no softmax) reaches 7.3 TB/s and draws 970 W of the
// board's 1000 W; with the products 6.4 TB/s, with the softmax as well 4.6-4.7 TB/s, both at the
// power limit with the SM clock near 1.5-1.6 GHz: run for longer than a few milliseconds the
// kernel is bound by power, and what helps is fewer instructions per weight.
#include <type_traits>

#include "sq_decode_common.cuh"
#include "sq_internal.h"
#include "sq_tc.cuh"
#include "sq_tc_quad.cuh"

namespace sq {

using namespace tc;

namespace {
constexpr int kD = 64;
constexpr int kTileBytes = kTM * kD * 2;  // 16 KB: one K or V tile
constexpr float kMaxWeight = 65536.f;     // 2^16
constexpr int kColS = 0, kColP = 128, kColO = 192, kTmemCols = 256;
__host__ __device__ constexpr uint32_t idesc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

}  // namespace

// ROWS: head rows of Q held in shared memory (96 or 128).
template <int STAGES, int ROWS, bool H2O>
__global__ void __launch_bounds__(192, 2)
    decode_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                          const __grid_constant__ CUtensorMap tm_v, DecodeArgs a) {
  constexpr int kQBytes = ROWS * 128;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // The first MMA addresses 128 rows of Q; with ROWS = 96 rows 96..127 alias the K stage that
  // follows (rows are independent, those accumulator rows are never read).
  unsigned char* q_s = smem;
  unsigned char* k_s = q_s + kQBytes;              // STAGES tiles
  unsigned char* v_s = k_s + STAGES * kTileBytes;  // STAGES tiles
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(v_s + STAGES * kTileBytes);
  static_assert(6 + 2 * STAGES <= 16, "barrier block");
  const uint32_t bar_q = s_u32(bars + 0), bar_odone = s_u32(bars + 1), bar_sfull = s_u32(bars + 2),
                 bar_sfree = s_u32(bars + 3), bar_pready = s_u32(bars + 4), bar_pfree = s_u32(bars + 5);
  auto bar_full = [&](int s) { return s_u32(bars + 6 + s); };
  auto bar_empty = [&](int s) { return s_u32(bars + 6 + STAGES + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  ItemLoc it;
  if (!locate(a, blockIdx.x, it)) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LayerDesc* ldp = a.layers + it.layer;
  const int b = ldp->b, cap = ldp->cap, G = a.group;
  const int unit = it.local / it.n_split, split = it.local - unit * it.n_split;
  const int len = min(a.n_tok + 1, b);
  int w;
  if (H2O) {
    w = (a.n_tok < b) ? a.n_tok : reinterpret_cast<const int*>(a.pool + ldp->victim_off)[unit];
    if (w < 0 || w >= b) {
      if (tid == 0) atomicOr(a.status, 2);
      w = 0;
    }
  } else {
    w = ring_slot(a.n_tok, b, ldp->ring_base, ldp->ring_origin);
  }
  const int t0 = split * a.split_tokens, t1 = min(len, t0 + a.split_tokens);
  const int n_tiles = (t1 - t0 + kTM - 1) / kTM;
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
  using bf16 = __nv_bfloat16;
  // (pointers are formed where they are used: the softmax loop needs the registers)

  // the CTA whose range holds slot w stores the new token first (generic proxy), then lets
  // the TMA reads (async proxy) see it
  if (w >= t0 && w < t1) {
    if (tid < 16) {
      bf16* Kb = reinterpret_cast<bf16*>(a.pool + ldp->k_off) + (size_t)unit * cap * kD;
      bf16* Vb = reinterpret_cast<bf16*>(a.pool + ldp->v_off) + (size_t)unit * cap * kD;
      const bf16* kn = reinterpret_cast<const bf16*>(a.k_new) + (tok * a.n_kv_head + kvh) * kD;
      const bf16* vn = reinterpret_cast<const bf16*>(a.v_new) + (tok * a.n_kv_head + kvh) * kD;
      const bool is_v = tid >= 8;
      const int c = tid & 7;
      const uint4 val = *reinterpret_cast<const uint4*>((is_v ? vn : kn) + c * 8);
      *reinterpret_cast<uint4*>((is_v ? Vb : Kb) + (size_t)w * kD + c * 8) = val;
    }
    if (tid == 16) {
      reinterpret_cast<int*>(a.pool + ldp->pos_off)[(size_t)unit * cap + w] = a.n_tok;
      if (H2O) reinterpret_cast<float*>(a.pool + ldp->acc_off)[(size_t)unit * cap + w] = 0.f;
    }
    __threadfence();
    fence_proxy_async();
  }
  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_odone, 1);
    mbar_init(bar_sfull, 1);
    mbar_init(bar_sfree, 4);   // one arrival per softmax warp
    mbar_init(bar_pready, 4);
    mbar_init(bar_pfree, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      // rows of this unit in the [rows][64] views of the pool (tensor maps) and of q
      const long long k_row0 = ldp->k_off / (kD * 2) + (long long)unit * cap;
      const long long v_row0 = ldp->v_off / (kD * 2) + (long long)unit * cap;
      const long long q_row0 = (long long)(tok * a.n_q_head + (size_t)kvh * G);
      mbar_expect_tx(bar_q, kQBytes);
      tma_load_2d(s_u32(q_s), &tm_q, 0, (int)q_row0, bar_q);
      int issued = 0;
      for (int i = 0; i < n_tiles; ++i) {
        const int st = i % STAGES;
        if (i >= STAGES && !mbar_wait(bar_empty(st), ((i / STAGES) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(bar_full(st), 2 * kTileBytes);
        tma_load_2d(s_u32(k_s + st * kTileBytes), &tm_k, 0, (int)(k_row0 + t0 + i * kTM), bar_full(st));
        tma_load_2d(s_u32(v_s + st * kTileBytes), &tm_v, 0, (int)(v_row0 + t0 + i * kTM), bar_full(st));
        issued = i + 1;
      }
      if (*abort_flag) {
        mbar_wait(bar_q, 0, abort_flag);
        for (int i = max(0, issued - STAGES); i < issued; ++i)
          for (int k = 0; k < kSpinLimit && !mbar_try_wait(bar_full(i % STAGES), (i / STAGES) & 1); ++k) {
          }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: one thread ----------------
    if (lane == 0) {
      const uint32_t q_addr = s_u32(q_s);
      auto issue_s = [&](int i) -> bool {
        const int st = i % STAGES;
        if (!mbar_wait(bar_full(st), (i / STAGES) & 1, abort_flag)) return false;
        if (i >= 1 && !mbar_wait(bar_sfree, (i - 1) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t k_addr = s_u32(k_s + st * kTileBytes);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k)
          umma_bf16(tmem_base + kColS, umma_desc(q_addr + k * 32), umma_desc(k_addr + k * 32), idesc(128, false),
                    k > 0 ? 1u : 0u);
        umma_commit(bar_sfull);
        return true;
      };
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      if (ok) ok = issue_s(0);
      for (int i = 0; ok && i < n_tiles; ++i) {
        if (i + 1 < n_tiles) ok = issue_s(i + 1);
        if (!ok) break;
        const int st = i % STAGES;
        ok = mbar_wait(bar_pready, i & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t v_addr = s_u32(v_s + st * kTileBytes);
#pragma unroll
        for (int k = 0; k < kTM / 16; ++k)
          // A = P in tensor memory: 16 tokens = 8 columns per step; B = V, MN-major: 2 KB per step
          umma_bf16_ta(tmem_base + kColO, tmem_base + kColP + k * 8, umma_desc(v_addr + k * 2048), idesc(kD, true),
                       (i > 0 || k > 0) ? 1u : 0u);
        umma_commit(bar_empty(st));
        umma_commit(bar_pfree);
        umma_commit(bar_odone);
      }
    }
    __syncwarp();
  } else {
    // ---------------- softmax: thread = one head row ----------------
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const bool live = row < G;                // this lane's row is a real head
    const bool warp_live = quarter * 32 < G;  // tcgen05.ld/st are warp-wide: whole warps opt in or out
    const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_sel + kColS, p_addr = tmem_base + lane_sel + kColP,
                   o_addr = tmem_base + lane_sel + kColO;
    float m_ref = -INFINITY, l = 0.f, l_w = 0.f;  // the row's reference; sums of its weights, exact and as rounded to bf16
    bool ok = true;
    // quad form (see QuadCtx): m_ref is the row's (equal in its four threads), l and l_w are the
    // thread's part; the row's totals are formed once, at the end
    const int rows_here = G - quarter * 32;
    const bool quad = rows_here >= 1 && rows_here <= 8 && n_tiles >= 6;  // short items: the set-up would not pay
    const QuadCtx qc{s_addr, p_addr, bar_sfree, a.scale_log2, lane};
    auto quad_sum = [&](float v) {
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      return v + __shfl_xor_sync(0xffffffffu, v, 2);
    };
    // the value the quad of row `lane` holds, for the lanes that own a row of O (others: their own)
    auto from_row_quad = [&](float v) { return __shfl_sync(0xffffffffu, v, lane < 8 ? lane * 4 : lane); };

    // Row maximum of the tile's valid tokens, in the log2 domain.
    auto tile_max = [&](int n_valid) {
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float v[32];
        tmem_ld32(s_addr + c * 32, v);
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (c * 32 + j < n_valid) mx = fmaxf(mx, v[j]);
      }
      return mx * a.scale_log2;
    };
    // p = exp2(s*scale - m_ref) for the whole tile: P (bf16) to tensor memory; sums of the weights
    // (exact fp32 for the H2O normaliser, of the bf16-rounded weights for the output) to *sum /
    // *sum_w; returns an upper bound of the largest weight.  The role is bound by the
    // special-function unit (one exp2 per 8 cycles per warp) and by the issue slots of one or two
    // softmax warps per scheduler, so the scaling runs as packed fp32x2 instructions and the
    // rounded weights are summed by mixed-precision adds: six instructions per two weights.
    // FULL (a compile-time tag): every token of the tile is valid, so no masking code is emitted
    // (with a run-time flag the compare / select pair ran for every weight of every tile).
    auto tile_weights = [&](auto full_tag, int n_valid, float* sum, float* sum_w, bool* s_released) {
      constexpr bool full = decltype(full_tag)::value;
      const unsigned long long scale2 = f32x2(a.scale_log2, a.scale_log2), neg_m2 = f32x2(-m_ref, -m_ref);
      unsigned long long acc2 = f32x2(0.f, 0.f);  // exact sums (H2O), even and odd tokens
      float w_a = 0.f, w_b = 0.f;                 // sums of the rounded weights
      auto chunk = [&](const uint32_t (&r)[32], int c) {
#pragma unroll
        for (int hc = 0; hc < 2; ++hc) {  // P goes back sixteen tokens (eight columns) at a time
          uint32_t pk[8];
#pragma unroll
          for (int jj = 0; jj < 16; jj += 2) {
            const int j = hc * 16 + jj;
            float p0, p1;
            f32x2_split(fma_f32x2(f32x2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), scale2, neg_m2), p0, p1);
            p0 = ex2(p0);
            p1 = ex2(p1);
            if (!full) {
              if (c * 32 + j >= n_valid) p0 = 0.f;
              if (c * 32 + j + 1 >= n_valid) p1 = 0.f;
            }
            if (H2O) acc2 = add_f32x2(acc2, f32x2(p0, p1));
            const uint32_t u = pack2(p0, p1);  // round to nearest bf16, p0 in the low half
            w_a = add_bf16_lo(w_a, u);
            w_b = add_bf16_hi(w_b, u);
            pk[jj / 2] = u;
          }
          tmem_st8_u32(p_addr + c * 16 + hc * 8, pk);  // tokens c*32 + hc*16 .. +15 of this row
        }
      };
      // the next chunk's tensor-memory load is in flight while this one is processed
      uint32_t ra[32], rb[32];
      tmem_ld32_nowait(s_addr, ra);
      tmem_wait_ld(ra);
      tmem_ld32_nowait(s_addr + 32, rb);
      chunk(ra, 0);
      tmem_wait_ld(rb);
      tmem_ld32_nowait(s_addr + 64, ra);
      chunk(rb, 1);
      tmem_wait_ld(ra);
      tmem_ld32_nowait(s_addr + 96, rb);
      chunk(ra, 2);
      tmem_wait_ld(rb);
      {
        // The last quarter of S is in registers.  Unless the tile may have to be redone (the
        // weights so far, or a logit of this quarter, too large), S is handed back now, so the
        // tensor core computes the next tile's S while these 32 weights are worked out.
        float mx = __uint_as_float(rb[0]);
#pragma unroll
        for (int j = 1; j + 1 < 32; j += 2) mx = max3(mx, __uint_as_float(rb[j]), __uint_as_float(rb[j + 1]));
        mx = fmaxf(mx, __uint_as_float(rb[31]));
        const float so_far = w_a + w_b;
        // 32 weights of at most 2^10 and 2^15 before them stay below kMaxWeight
        const bool safe = so_far <= 32768.f && fmaf(mx, a.scale_log2, -m_ref) <= 10.f;
        *s_released = __all_sync(0xffffffffu, safe);
        if (*s_released) {
          tc_fence_before();
          if (lane == 0) mbar_arrive(bar_sfree);
        }
      }
      chunk(rb, 3);
      tmem_wait_st();
      float s0, s1;
      f32x2_split(acc2, s0, s1);
      *sum = s0 + s1;
      *sum_w = w_a + w_b;
      return w_a + w_b;  // the tile's weight sum bounds its largest weight
    };

    for (int i = 0; ok && i < n_tiles; ++i) {
      const int st = i % STAGES;
      const int tile_row0 = t0 + i * kTM;
      const int n_valid = min(kTM, t1 - tile_row0);
      ok = mbar_wait(bar_sfull, i & 1, abort_flag);
      if (ok && i >= 1) ok = mbar_wait(bar_pfree, (i - 1) & 1, abort_flag);
      if (ok && n_valid < kTM) {
        // rows of the V tile past the unit's last token may hold anything: zero them
        ok = mbar_wait(bar_full(st), (i / STAGES) & 1, abort_flag);
        if (ok && row >= n_valid) {
          uint4* vrow = reinterpret_cast<uint4*>(v_s + st * kTileBytes + row * 128);
#pragma unroll
          for (int c = 0; c < 8; ++c) vrow[c] = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();  // the zeroed rows must be visible to the tensor core
      }
      if (!ok) break;
      tc_fence_after();
      bool s_released = false;
      if (warp_live) {
        if (i == 0) {
          m_ref = quad ? quad_tile_max(qc, n_valid) : tile_max(n_valid);
          if (quad) {
            // rows 80..95 of P are never written in the quad form: clear them once
            float z[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) z[j] = 0.f;
            tmem_st32(p_addr, z);
            tmem_st32(p_addr + 32, z);
          }
        }
        float sum, sum_w;
        auto weights = [&]() {
          if (quad) {
            float sums[2];
            s_released = (n_valid == kTM) ? quad_tile_weights<H2O, true, true>(qc, m_ref, n_valid, sums)
                                          : quad_tile_weights<H2O, false, true>(qc, m_ref, n_valid, sums);
            sum = sums[0];
            sum_w = sums[1];
            return sum_w;
          }
          return (n_valid == kTM) ? tile_weights(std::true_type{}, n_valid, &sum, &sum_w, &s_released)
                                  : tile_weights(std::false_type{}, n_valid, &sum, &sum_w, &s_released);
        };
        float pmax = weights();
        if (__any_sync(0xffffffffu, pmax > kMaxWeight)) {
          // rare: move the reference of the rows that need it; O and the sums (complete up to
          // tile i-1) shrink with it, then the tile is redone.  The whole warp takes part in
          // the TMEM round trip.
          const float mx2 = quad ? quad_tile_max(qc, n_valid) : tile_max(n_valid);
          // quad form: the row moves when any of its four threads needs it
          const bool need = quad ? __any_sync(0xfu << (lane & 28), pmax > kMaxWeight) : pmax > kMaxWeight;
          ok = mbar_wait(bar_odone, (i - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const float f = need ? ex2(m_ref - mx2) : 1.f;
          // O is held a row per lane in either form
          float f_o = f;
          if (quad) {
            f_o = from_row_quad(f);
            if (lane >= 8) f_o = 1.f;
          }
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            float o[32];
            tmem_ld32(o_addr + c * 32, o);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] *= f_o;
            tmem_st32(o_addr + c * 32, o);
          }
          l *= f;
          l_w *= f;
          if (need) m_ref = mx2;
          pmax = weights();
        }
        l += sum;
        l_w += sum_w;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar_pready);
        if (!s_released) mbar_arrive(bar_sfree);
      }
    }
    // ---------------- epilogue: O / l -> out (or the split-K partial) ----------------
    if (ok) ok = mbar_wait(bar_odone, (n_tiles - 1) & 1, abort_flag);
    if (ok && warp_live) {
      tc_fence_after();
      bf16* ob = reinterpret_cast<bf16*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G) * kD;
      float* stat = a.part_stat + (size_t)blockIdx.x * G * kStatStride;
      float* po = a.part_o + (size_t)blockIdx.x * G * kD;
      if (quad) {
        // the row's totals from its four threads, then to the lane that holds the row of O
        l = from_row_quad(quad_sum(l));
        l_w = from_row_quad(quad_sum(l_w));
        m_ref = from_row_quad(m_ref);
      }
      const float inv = 1.f / l_w;
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        float o[32];
        tmem_ld32(o_addr + c * 32, o);
        if (!live) continue;
        if (it.n_split == 1) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            *reinterpret_cast<uint4*>(ob + (size_t)row * kD + c * 32 + q4 * 8) =
                make_uint4(pack2(o[q4 * 8] * inv, o[q4 * 8 + 1] * inv), pack2(o[q4 * 8 + 2] * inv, o[q4 * 8 + 3] * inv),
                           pack2(o[q4 * 8 + 4] * inv, o[q4 * 8 + 5] * inv), pack2(o[q4 * 8 + 6] * inv, o[q4 * 8 + 7] * inv));
        } else {
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            *reinterpret_cast<float4*>(po + (size_t)row * kD + c * 32 + q4 * 4) =
                make_float4(o[q4 * 4], o[q4 * 4 + 1], o[q4 * 4 + 2], o[q4 * 4 + 3]);
        }
      }
      if (live) {
        stat[row * kStatStride] = m_ref;
        stat[row * kStatStride + 1] = H2O ? l : l_w;
        stat[row * kStatStride + 2] = l_w;
        // H2O: the unit's row log-sum-exps (log2 domain), read by the score-update pass that follows
        if (H2O && it.n_split == 1) (a.logits + ldp->lse_off + (size_t)unit * G)[row] = m_ref + log2f(l);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
  }
  if (tid == 0 && *abort_flag) atomicOr(a.status, kStatusTimeout);
  if (it.n_split > 1) merge_if_last<bf16>(a, it, unit, H2O ? a.logits + ldp->lse_off + (size_t)unit * G : nullptr);
}

template <int STAGES, int ROWS, bool H2O>
static cudaError_t launch_tc_cfg(const DecodeArgs& a, int n_items, const CUtensorMap& tq, const CUtensorMap& tk,
                                 const CUtensorMap& tv, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)ROWS * 128 + (size_t)2 * STAGES * kTileBytes + 8 * 16 + 16;
  auto kern = decode_attn_tc_kernel<STAGES, ROWS, H2O>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  kern<<<n_items, 192, smem, s>>>(tq, tk, tv, a);
  return cudaGetLastError();
}

// Returns cudaErrorNotSupported when the shape is outside this kernel's range.
cudaError_t launch_decode_attn_tc(const DecodeArgs& a, int n_items, size_t pool_bytes, size_t q_rows, cudaStream_t s) {
  if (a.head_dim != kD || a.group <= 32 || a.group > 128) return cudaErrorNotSupported;
  const long long pool_rows = (long long)(pool_bytes / (kD * 2));
  if (pool_rows + kTM > 0x7fffffffLL || (long long)q_rows + kTM > 0x7fffffffLL) return cudaErrorNotSupported;
  const int rows = a.group <= 96 ? 96 : 128;
  CUtensorMap tm_q, tm_k, tm_v;
  if (!make_tile_map(&tm_q, a.q, (long long)q_rows, kD, rows) || !make_tile_map(&tm_k, a.pool, pool_rows, kD, kTM) ||
      !make_tile_map(&tm_v, a.pool, pool_rows, kD, kTM))
    return cudaErrorNotSupported;
  const bool h2o = a.policy == SQ_POLICY_H2O;
  if (rows == 96)
    return h2o ? launch_tc_cfg<3, 96, true>(a, n_items, tm_q, tm_k, tm_v, s)
               : launch_tc_cfg<3, 96, false>(a, n_items, tm_q, tm_k, tm_v, s);
  return h2o ? launch_tc_cfg<2, 128, true>(a, n_items, tm_q, tm_k, tm_v, s)
             : launch_tc_cfg<2, 128, false>(a, n_items, tm_q, tm_k, tm_v, s);
}

}  // namespace sq
