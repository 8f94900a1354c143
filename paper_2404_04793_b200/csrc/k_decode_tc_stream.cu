// The even-deal form of the wide-group decode attention kernel (k_decode_tc.cu: 33..128 query
// heads per KV head, head_dim 64, bf16; S = Q K^T and O += P V as tcgen05.mma, P in tensor
// memory), for launches whose units are long but too few to fill the GPU: one layer of a large
// batch has about as many units as there are CTA slots (224 units for 296 slots at the largest
// Falcon-shaped cell), so with one CTA per unit a quarter of the slots idle, and cutting every
// unit into pieces costs each piece a CTA's set-up.
//
// Work split.  The kept tokens of every (layer, unit) of the launch are cut into 128-token tiles,
// numbered in launch order (largest budget first), and dealt out evenly: the grid is two
// persistent CTAs per SM and CTA c takes the tiles [c * chunk, (c + 1) * chunk), so every CTA
// streams the same number of K/V bytes whatever the budgets and however few units a launch has
// (one layer of a batch is a fraction of a wave of units).  A CTA's run of tiles of one unit is
// a segment.  A segment that covers its whole unit writes the output; otherwise it leaves an
// un-normalised partial (reference, weight sums, O) in one of the CTA's two partial slots and
// the piece that arrives last at the unit's ticket merges them in piece order (deterministic;
// no piece waits for another).
//
// Per 128-token tile the roles are
//   warp 0      TMA: Q per segment, K and V tiles into a ring of stages (128-byte swizzle, every
//               CTA loads its own tiles); stores the new token's row before the tile that holds
//               its slot is fetched
//   warp 1      MMA issue (one thread)
//   warps 2..5  thread = one head row (TMEM lane): p = exp2(s*scale - m_ref) straight from the
//               accumulator row, no shuffles; P is packed to bf16 and stored back to tensor
//               memory as the A operand of the second MMA; at a segment's end the same warps
//               normalise and store O (or the partial) and, if theirs was the last piece, merge
// Measured on B200: one M=128, K=16 MMA costs 45-48 cycles for N <= 64 and 64 cycles for N = 128
// with the A operand in tensor memory, 68 with both operands in shared memory (whatever their
// major-ness), and operands read from shared memory compete with the TMA writes for its
// 128 B/clk; keeping P in tensor memory removes 56 KB of shared-memory traffic per tile.
// A row's reference m_ref is its maximum over the segment's first tile; later tiles reuse it and
// only when a weight would exceed 2^16 is the reference moved (O and the sums rescaled through
// tcgen05.ld/st, the tile redone): every weight stays finite and the result is that of the
// exact softmax.  Every barrier wait is bounded.
//
// Measured per launch of one layer (ncu, cold cache) against one CTA per unit and split-K piece:
// 224 units of 115 / 20 tiles: 202 / 60 us against 149 us on average over both kinds (4.05 vs
// 4.76 ms per decode step); 128 units of 23 / 4 tiles: 51 / 25 us against 32 us on average; 32
// units of 115 / 20 tiles: 61 / 41 us against 55 / 31 us.  A persistent CTA pays about 5 us more
// than a one-unit CTA before its first tile and every unit cut by a CTA boundary pays a merge, so
// this form is taken only where it wins: at least half as many units as CTA slots, fewer than
// twice as many, and at least 16 tiles per unit.
#include <algorithm>
#include <type_traits>

#include "sq_decode_common.cuh"
#include "sq_internal.h"
#include "sq_stream.cuh"
#include "sq_tc.cuh"

namespace sq {

using namespace tc;

namespace {
constexpr int kD = 64;
constexpr int kTileBytes = kTM * kD * 2;  // 16 KB: one K or V tile
constexpr float kMaxWeight = 65536.f;     // 2^16
constexpr int kColS = 0, kColP = 128, kColO = 192, kTmemCols = 256;
constexpr int kCtasPerSm = 2;

__host__ __device__ constexpr uint32_t idesc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// Every lane waits (a suspended try_wait wakes sooner than one polling lane plus a shuffle:
// measured 3.73 vs 4.27 ms per decode step of the largest Falcon-shaped cell); the warp agrees
// on the outcome, so that it leaves its loop as a whole.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}

// Merge of a unit's pieces by the group of `nt` threads that arrived last at the unit's ticket:
// the pieces are read back in piece order, so the result does not depend on who merges.  sync()
// is the group's barrier (false: the group gives up).  With lse_out set, the merged log-sum-exp
// (log2 domain, from the unrounded weight sums) of every head is stored there as well.
template <typename Sync>
__device__ __forceinline__ void merge_pieces(const StreamArgs& a, int layer, int unit, int c_first, int n_piece, float* lse_out,
                                             int tid, int nt, float* s_m, float* s_inv, Sync sync) {
  const int G = a.group;
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(layer - a.layer_begin) * a.batch + seq;
  for (int h = tid; h < G; h += nt) {
    float M = -INFINITY;
    for (int s = 0; s < n_piece; ++s)
      M = fmaxf(M, __ldcg(a.part_stat + ((size_t)piece_slot(c_first, s) * G + h) * kStatStride));
    float Lw = 0.f, Lt = 0.f;
    for (int s = 0; s < n_piece; ++s) {
      const float4 st = __ldcg(reinterpret_cast<const float4*>(a.part_stat + ((size_t)piece_slot(c_first, s) * G + h) * kStatStride));
      const float f = exp2f(st.x - M);
      Lw += st.z * f;
      Lt += st.y * f;
    }
    s_m[h] = M;
    s_inv[h] = 1.f / Lw;
    if (lse_out) lse_out[h] = M + log2f(Lt);
  }
  if (!sync()) return;
  __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G) * kD;
  const int n4 = G * kD / 4;  // four consecutive outputs of one head per step
  for (int i4 = tid; i4 < n4; i4 += nt) {
    const int h = (i4 * 4) / kD;
    float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < n_piece; ++s) {
      const int slot = piece_slot(c_first, s);
      const float4 v = __ldcg(reinterpret_cast<const float4*>(a.part_o + (size_t)slot * G * kD) + i4);
      const float f = exp2f(__ldcg(a.part_stat + ((size_t)slot * G + h) * kStatStride) - s_m[h]);
      O.x += v.x * f;
      O.y += v.y * f;
      O.z += v.z * f;
      O.w += v.w * f;
    }
    const float inv = s_inv[h];
    uint2 pk;
    pk.x = pack2(O.x * inv, O.y * inv);
    pk.y = pack2(O.z * inv, O.w * inv);
    reinterpret_cast<uint2*>(ob)[i4] = pk;
  }
}
}  // namespace

// ROWS: head rows of Q held in shared memory (96 or 128).
template <int STAGES, int ROWS, bool H2O>
__global__ void __launch_bounds__(192, kCtasPerSm)
    decode_attn_tc_stream_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                          const __grid_constant__ CUtensorMap tm_v, const StreamArgs a) {
  constexpr int kQBytes = ROWS * 128;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // The first MMA addresses 128 rows of Q; with ROWS = 96 rows 96..127 alias the K stage that
  // follows (rows are independent, those accumulator rows are never read).
  unsigned char* q_s = smem;
  unsigned char* k_s = q_s + kQBytes;              // STAGES tiles
  unsigned char* v_s = k_s + STAGES * kTileBytes;  // STAGES tiles
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(v_s + STAGES * kTileBytes);
  static_assert(9 + 2 * STAGES <= 16, "barrier block");
  const uint32_t bar_qfull = s_u32(bars + 0), bar_qempty = s_u32(bars + 1), bar_odone = s_u32(bars + 2),
                 bar_sfull = s_u32(bars + 3), bar_sfree = s_u32(bars + 4), bar_pready = s_u32(bars + 5),
                 bar_pfree = s_u32(bars + 6), bar_epi = s_u32(bars + 7);
  auto bar_full = [&](int s) { return s_u32(bars + 9 + s); };
  auto bar_empty = [&](int s) { return s_u32(bars + 9 + STAGES + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* s_last = reinterpret_cast<int*>(tmem_slot + 2);
  float* s_mm = reinterpret_cast<float*>(bars + 18);  // [128] merge scratch: maxima
  float* s_minv = s_mm + kTM;                         // [128] merge scratch: 1 / weight sum

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = a.group;
  using bf16 = __nv_bfloat16;

  if (tid == 0) {
    mbar_init(bar_qfull, 1);
    mbar_init(bar_qempty, 1);
    mbar_init(bar_odone, 1);
    mbar_init(bar_sfull, 1);
    mbar_init(bar_sfree, 4);  // one arrival per softmax warp
    mbar_init(bar_pready, 4);
    mbar_init(bar_pfree, 1);
    mbar_init(bar_epi, 4);
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
  SegIter it;
  it.init(a, blockIdx.x);

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    int g = 0;          // tiles issued so far
    int q_issued = 0;   // segments whose Q has been issued
    bool ok = true;
    while (ok && it.next(a)) {
      const LayerDesc* ldp = a.layers + it.layer;
      const int b = ldp->b, cap = ldp->cap, unit = it.unit;
      const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
      const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
      const int t0 = it.tile0 * kTM, t1 = min(it.len, (it.tile0 + it.ntile) * kTM);
      // the slot the new token takes: the next free one while the cache grows, else the policy's victim
      int w;
      if (H2O) {
        w = (a.n_tok < b) ? a.n_tok : reinterpret_cast<const int*>(a.pool + ldp->victim_off)[unit];
        if (w < 0 || w >= b) {
          if (lane == 0) atomicOr(a.status, 2);
          w = 0;
        }
      } else {
        w = ring_slot(a.n_tok, b, ldp->ring_base, ldp->ring_origin);
      }
      if (w >= t0 && w < t1) {
        // this segment fetches the tile that holds slot w: store the new row first (generic
        // proxy), then let the TMA reads (async proxy) see it
        if (lane < 16) {
          bf16* Kb = reinterpret_cast<bf16*>(a.pool + ldp->k_off) + (size_t)unit * cap * kD;
          bf16* Vb = reinterpret_cast<bf16*>(a.pool + ldp->v_off) + (size_t)unit * cap * kD;
          const bf16* kn = reinterpret_cast<const bf16*>(a.k_new) + (tok * a.n_kv_head + kvh) * kD;
          const bf16* vn = reinterpret_cast<const bf16*>(a.v_new) + (tok * a.n_kv_head + kvh) * kD;
          const bool is_v = lane >= 8;
          const int c = lane & 7;
          const uint4 val = *reinterpret_cast<const uint4*>((is_v ? vn : kn) + c * 8);
          *reinterpret_cast<uint4*>((is_v ? Vb : Kb) + (size_t)w * kD + c * 8) = val;
        }
        if (lane == 16) {
          reinterpret_cast<int*>(a.pool + ldp->pos_off)[(size_t)unit * cap + w] = a.n_tok;
          if (H2O) reinterpret_cast<float*>(a.pool + ldp->acc_off)[(size_t)unit * cap + w] = 0.f;
        }
        __threadfence();
        fence_proxy_async();
        __syncwarp();
      }
      // Q has one buffer: the previous segment's last S product must have read it
      if (it.seg >= 1) ok = warp_wait(bar_qempty, (it.seg - 1) & 1, abort_flag);
      if (!ok) break;
      // rows of this unit in the [rows][64] views of the pool (tensor maps) and of q
      const long long k_row0 = ldp->k_off / (kD * 2) + (long long)unit * cap + t0;
      const long long v_row0 = ldp->v_off / (kD * 2) + (long long)unit * cap + t0;
      if (lane == 0) {
        mbar_expect_tx(bar_qfull, kQBytes);
        tma_load_2d(s_u32(q_s), &tm_q, 0, (int)(tok * a.n_q_head + (size_t)kvh * G), bar_qfull);
      }
      q_issued = it.seg + 1;
      for (int i = 0; ok && i < it.ntile; ++i, ++g) {
        const int st = g % STAGES;
        if (g >= STAGES) ok = warp_wait(bar_empty(st), ((g / STAGES) - 1) & 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(bar_full(st), 2 * kTileBytes);
          tma_load_2d(s_u32(k_s + st * kTileBytes), &tm_k, 0, (int)(k_row0 + i * kTM), bar_full(st));
          tma_load_2d(s_u32(v_s + st * kTileBytes), &tm_v, 0, (int)(v_row0 + i * kTM), bar_full(st));
        }
      }
    }
    if (*abort_flag && lane == 0) {
      // copies in flight must land before the CTA's shared memory is released
      if (q_issued > 0)
        for (int k = 0; k < kSpinLimit && !mbar_try_wait(bar_qfull, (q_issued - 1) & 1); ++k) {
        }
      for (int i = max(0, g - STAGES); i < g; ++i)
        for (int k = 0; k < kSpinLimit && !mbar_try_wait(bar_full(i % STAGES), (i / STAGES) & 1); ++k) {
        }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    {
      const uint32_t q_addr = s_u32(q_s);
      int gs = 0, gp = 0;  // S and O products issued so far
      bool ok = true;
      // S product of tile i of the current segment
      auto issue_s = [&](int i) {
        const int st = gs % STAGES;
        if (i == 0) ok = mbar_wait(bar_qfull, it.seg & 1, abort_flag);
        if (ok) ok = mbar_wait(bar_full(st), (gs / STAGES) & 1, abort_flag);
        if (ok && gs >= 1) ok = mbar_wait(bar_sfree, (gs - 1) & 1, abort_flag);
        if (!ok) return;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t k_addr = s_u32(k_s + st * kTileBytes);
#pragma unroll
          for (int k = 0; k < kD / 16; ++k)
            umma_bf16(tmem_base + kColS, umma_desc(q_addr + k * 32), umma_desc(k_addr + k * 32), idesc(128, false), k > 0 ? 1u : 0u);
          umma_commit(bar_sfull);
          if (i == it.ntile - 1) umma_commit(bar_qempty);
        }
        __syncwarp();
        ++gs;
      };
      bool more = it.next(a);
      if (more) issue_s(0);
      while (ok && more) {
        for (int i = 0; ok && i < it.ntile; ++i) {
          if (i + 1 < it.ntile) issue_s(i + 1);
          if (!ok) break;
          const int st = gp % STAGES;
          ok = mbar_wait(bar_pready, gp & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
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
          __syncwarp();
          ++gp;
        }
        if (!ok) break;
        // the next segment's first S product goes out only now: its Q is fetched after this
        // segment's last S product, and the last O product must not wait for that fetch
        more = it.next(a);
        if (more) issue_s(0);
      }
    }
    __syncwarp();
  } else {
    // ---------------- softmax: thread = one head row ----------------
    const int quarter = warp & 3, etid = (warp - 2) * 32 + lane;
    const int row = quarter * 32 + lane;
    const bool live = row < G;                // this lane's row is a real head
    const bool warp_live = quarter * 32 < G;  // tcgen05.ld/st are warp-wide: whole warps opt in or out
    const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_sel + kColS, p_addr = tmem_base + lane_sel + kColP,
                   o_addr = tmem_base + lane_sel + kColO;
    float m_ref = -INFINITY, l_true = 0.f, l_w = 0.f;
    int g0 = 0;  // tiles of the CTA before the current segment
    int epi_use = 0;
    bool ok = true;
    int t1 = 0;
    auto epi_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_epi);
      ok = warp_wait(bar_epi, epi_use & 1, abort_flag);
      ++epi_use;
      return ok;
    };

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
    auto tile_weights = [&](auto full_tag, int n_valid, float* sum, float* sum_w) {
      constexpr bool full = decltype(full_tag)::value;
      const unsigned long long scale2 = f32x2(a.scale_log2, a.scale_log2), neg_m2 = f32x2(-m_ref, -m_ref);
      unsigned long long acc2 = f32x2(0.f, 0.f);
      float w_a = 0.f, w_b = 0.f;
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
      chunk(rb, 3);
      tmem_wait_st();
      float s0, s1;
      f32x2_split(acc2, s0, s1);
      *sum = s0 + s1;
      *sum_w = w_a + w_b;
      return w_a + w_b;  // the tile's weight sum bounds its largest weight
    };

    while (ok && it.next(a)) {
      const int t0 = it.tile0 * kTM;
      t1 = min(it.len, (it.tile0 + it.ntile) * kTM);
      m_ref = -INFINITY;
      l_true = 0.f;
      l_w = 0.f;
      for (int i = 0; ok && i < it.ntile; ++i) {
        const int g = g0 + i, st = g % STAGES;
        const int n_valid = min(kTM, t1 - (t0 + i * kTM));
        ok = warp_wait(bar_sfull, g & 1, abort_flag);
        if (ok && g >= 1) ok = warp_wait(bar_pfree, (g - 1) & 1, abort_flag);
        if (ok && n_valid < kTM) {
          // rows of the V tile past the unit's last token may hold anything: zero them
          ok = warp_wait(bar_full(st), (g / STAGES) & 1, abort_flag);
          if (ok && row >= n_valid) {
            uint4* vrow = reinterpret_cast<uint4*>(v_s + st * kTileBytes + row * 128);
#pragma unroll
            for (int c = 0; c < 8; ++c) vrow[c] = make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async();  // the zeroed rows must be visible to the tensor core
        }
        if (!ok) break;
        tc_fence_after();
        if (warp_live) {
          if (i == 0) m_ref = tile_max(n_valid);
          float sum, sum_w;
          auto weights = [&]() {
            return (n_valid == kTM) ? tile_weights(std::true_type{}, n_valid, &sum, &sum_w)
                                    : tile_weights(std::false_type{}, n_valid, &sum, &sum_w);
          };
          float pmax = weights();
          if (__any_sync(0xffffffffu, pmax > kMaxWeight)) {
            // rare: move the reference of the rows that need it; O and the sums (complete up to
            // the previous tile) shrink with it, then the tile is redone.  The whole warp takes
            // part in the TMEM round trip.
            const float mx2 = tile_max(n_valid);
            const bool need = pmax > kMaxWeight;
            ok = warp_wait(bar_odone, (g - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const float f = need ? ex2(m_ref - mx2) : 1.f;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
              float o[32];
              tmem_ld32(o_addr + c * 32, o);
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] *= f;
              tmem_st32(o_addr + c * 32, o);
            }
            l_true *= f;
            l_w *= f;
            if (need) m_ref = mx2;
            pmax = weights();
          }
          l_true += sum;
          l_w += sum_w;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_pready);
          mbar_arrive(bar_sfree);
        }
      }
      if (!ok) break;
      // ---------------- end of the segment: O / l -> out, or the piece's partial ----------------
      const int g_last = g0 + it.ntile - 1;
      g0 += it.ntile;
      ok = warp_wait(bar_odone, g_last & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const int unit = it.unit;
      const LayerDesc* ldp = a.layers + it.layer;
      const int c_first = it.c_first(a), n_piece = it.n_piece(a);
      float* lse = H2O ? a.logits + ldp->lse_off + (size_t)unit * G : nullptr;
      if (warp_live) {
        const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
        const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
        const int slot = piece_slot(c_first, (int)blockIdx.x - c_first);
        bf16* orow = reinterpret_cast<bf16*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G + row) * kD;
        float* prow = a.part_o + ((size_t)slot * G + row) * kD;
        const float inv = 1.f / l_w;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          float o[32];
          tmem_ld32(o_addr + c * 32, o);
          if (!live) continue;
          if (n_piece == 1) {
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
              *reinterpret_cast<uint4*>(orow + c * 32 + q4 * 8) =
                  make_uint4(pack2(o[q4 * 8] * inv, o[q4 * 8 + 1] * inv), pack2(o[q4 * 8 + 2] * inv, o[q4 * 8 + 3] * inv),
                             pack2(o[q4 * 8 + 4] * inv, o[q4 * 8 + 5] * inv), pack2(o[q4 * 8 + 6] * inv, o[q4 * 8 + 7] * inv));
          } else {
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4)
              *reinterpret_cast<float4*>(prow + c * 32 + q4 * 4) = make_float4(o[q4 * 4], o[q4 * 4 + 1], o[q4 * 4 + 2], o[q4 * 4 + 3]);
          }
        }
        if (live) {
          if (n_piece == 1) {
            // H2O: the unit's row log-sum-exps (log2 domain), read by the score-update pass that follows
            if (H2O) lse[row] = m_ref + log2f(l_true);
          } else {
            *reinterpret_cast<float4*>(a.part_stat + ((size_t)slot * G + row) * kStatStride) =
                make_float4(m_ref, H2O ? l_true : l_w, l_w, 0.f);
          }
        }
      }
      tc_fence_before();  // the next segment's O products overwrite the accumulator read above
      if (n_piece > 1) {
        // the partial is written: take the unit's ticket; the piece that arrives last merges
        __threadfence();
        if (!epi_sync()) break;
        int* ticket = a.tickets + (size_t)it.layer * a.n_unit + unit;
        if (etid == 0) {
          __threadfence();
          *s_last = (atomicAdd(ticket, 1) == n_piece - 1);
        }
        if (!epi_sync()) break;
        if (*s_last) {
          __threadfence();
          if (etid == 0) *ticket = 0;
          merge_pieces(a, it.layer, unit, c_first, n_piece, lse, etid, 128, s_mm, s_minv, epi_sync);
        }
        if (!epi_sync()) break;  // s_last and the merge scratch are free again
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
}

template <int STAGES, int ROWS, bool H2O>
static cudaError_t launch_tc_stream_cfg(const StreamArgs& t, int n_cta, const CUtensorMap& tq, const CUtensorMap& tk,
                                 const CUtensorMap& tv, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)ROWS * 128 + (size_t)2 * STAGES * kTileBytes + 18 * 8 + 2 * kTM * 4;
  auto kern = decode_attn_tc_stream_kernel<STAGES, ROWS, H2O>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  kern<<<n_cta, 192, smem, s>>>(tq, tk, tv, t);
  return cudaGetLastError();
}

// desc_tiles[k]: 128-token tiles per unit of the k-th descriptor of the launch (launch order).
// Returns cudaErrorNotSupported when the shape is outside this kernel's range.
cudaError_t launch_decode_attn_tc_stream(const DecodeArgs& a, const int* desc_tiles, size_t pool_bytes, size_t q_rows,
                                  cudaStream_t s) {
  if (a.head_dim != kD || a.group <= 32 || a.group > 128) return cudaErrorNotSupported;
  const long long pool_rows = (long long)(pool_bytes / (kD * 2));
  if (pool_rows + kTM > 0x7fffffffLL || (long long)q_rows + kTM > 0x7fffffffLL) return cudaErrorNotSupported;
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  const int rows = a.group <= 96 ? 96 : 128;
  CUtensorMap tm_q, tm_k, tm_v;
  if (!make_tile_map(&tm_q, a.q, (long long)q_rows, kD, rows) || !make_tile_map(&tm_k, a.pool, pool_rows, kD, kTM) ||
      !make_tile_map(&tm_v, a.pool, pool_rows, kD, kTM))
    return cudaErrorNotSupported;
  const bool h2o = a.policy == SQ_POLICY_H2O;
  StreamArgs t;
  static_cast<DecodeArgsBase&>(t) = a;
  const int slots = kCtasPerSm * n_sm;
  {
    // where this form wins (see the head of this file)
    const long long units = (long long)a.n_layer_total * a.n_unit;
    int min_tiles = 1 << 30;
    for (int k = 0; k < a.n_layer_total; ++k) min_tiles = std::min(min_tiles, desc_tiles[k]);
    if (2 * units < slots || units >= 2LL * slots || min_tiles < 16) return cudaErrorNotSupported;
  }

  // the tile table holds kMaxLayers descriptors: larger launches (per-sequence budgets) go in groups
  for (int k0 = 0; k0 < a.n_layer_total; k0 += kMaxLayers) {
    const int cnt = std::min(kMaxLayers, a.n_layer_total - k0);
    const int n_cta = deal_tiles(t, a, desc_tiles, k0, cnt, slots);
    if (n_cta < 0) return cudaErrorNotSupported;
    if (n_cta == 0) continue;
    cudaError_t e;
    if (rows == 96) e = h2o ? launch_tc_stream_cfg<3, 96, true>(t, n_cta, tm_q, tm_k, tm_v, s) : launch_tc_stream_cfg<3, 96, false>(t, n_cta, tm_q, tm_k, tm_v, s);
    else e = h2o ? launch_tc_stream_cfg<2, 128, true>(t, n_cta, tm_q, tm_k, tm_v, s) : launch_tc_stream_cfg<2, 128, false>(t, n_cta, tm_q, tm_k, tm_v, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace sq
