// H2O score update for wide multi-query groups (33..128 query heads per KV head, head_dim 64,
// bf16): second pass of a decode step, after the attention kernel has written every head's row
// log-sum-exp.  Each kept token's score grows by the sum over the group's heads of its softmax
// probability (Algorithm 1's cache update with the H2O policy), and the token that the next
// append replaces is chosen.
// The logits are recomputed rather than carried through memory: a token has g fp32 logits but
// only 128 bytes of K, so re-reading K is 2-4x cheaper than writing and reading the logits.
// The product is taken transposed, S^T[128 tokens x heads] = K_tile Q^T as tcgen05.mma with the
// accumulator in tensor memory, so that a thread owns one token: its probabilities
// p = exp2(s*scale - lse_h) are summed over the heads in registers (no shuffles, no atomics,
// head order fixed: deterministic), and the score read-modify-write is one coalesced access.
//   warp 0      TMA: Q once, K tiles into a ring of stages (128-byte swizzle, every CTA its own tiles)
//   warp 1      MMA issue into a ring of accumulator buffers (three when the head columns fit
//               three times into 256 tensor-memory columns, else two)
//   warps 2..9  thread = one token (TMEM lane); warps 2..5 take the even tiles, warps 6..9 the
//               odd ones.  With three buffers the product of a set's next tile is finished
//               before the set is done with its current one, so the hand-over (barrier, MMA
//               issue: several hundred cycles measured) is off the critical path
// Split-K pieces of a unit leave their candidate in global memory; the piece that arrives last
// (atomic ticket, nobody waits) picks the winner.  Every barrier wait is bounded.
#include "sq_decode_common.cuh"
#include "sq_internal.h"
#include "sq_select.cuh"
#include "sq_tc.cuh"

namespace sq {

using namespace tc;

namespace {
constexpr int kD = 64;
constexpr int kTileBytes = kTM * kD * 2;  // 16 KB: one K tile
__host__ __device__ constexpr uint32_t idesc_n(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
struct Candidate {
  unsigned long long rank;
  int slot, pad;
};
}  // namespace

// SETS: groups of four token warps (tile i goes to set i % SETS); TMEM_COLS: tensor-memory columns of the CTA
// (256: three buffers of up to 80 head columns or two of up to 128; 128: one buffer); CTAS: CTAs per SM aimed at.
// UNIFORM / Args: 1 / DecodeArgsBase for launches without split-K (no lookup-table search compiled in), else 0 / DecodeArgs.
template <int STAGES, int SETS, int TMEM_COLS, int CTAS, int UNIFORM, class Args>
__global__ void __launch_bounds__(64 + 128 * SETS, CTAS)
    h2o_gain_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, Args a,
                       int n_cols, int n_buf) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* q_s = smem;                    // up to 128 head rows
  unsigned char* k_s = q_s + kTM * 128;         // STAGES tiles
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(k_s + STAGES * kTileBytes);
  static_assert(7 + 2 * STAGES <= 16, "barrier block");
  const uint32_t bar_q = s_u32(bars + 0);
  auto bar_sfull = [&](int j) { return s_u32(bars + 1 + j); };
  auto bar_sfree = [&](int j) { return s_u32(bars + 4 + j); };
  auto bar_full = [&](int s) { return s_u32(bars + 7 + s); };
  auto bar_empty = [&](int s) { return s_u32(bars + 7 + STAGES + s); };
  const int buf_cols = (n_buf == 3) ? n_cols : 128;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* s_nlse = reinterpret_cast<float*>(bars + 18);                     // [128] minus the row log-sum-exp
  Candidate* s_cand = reinterpret_cast<Candidate*>(s_nlse + kTM);          // one per token warp

  ItemLoc it;
  if (!locate<UNIFORM, Args>(a, blockIdx.x, it)) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LayerDesc* ldp = a.layers + it.layer;
  const int b = ldp->b, cap = ldp->cap, G = a.group;
  const int unit = it.local / it.n_split, split = it.local - unit * it.n_split;
  const int len = min(a.n_tok + 1, b);
  const bool full = (len == b);
  const int thr = a.n_tok + 1 - ldp->b_recent;  // next step: positions <= thr are outside the recent window
  const int t0 = split * a.split_tokens, t1 = min(len, t0 + a.split_tokens);
  const int n_tiles = (t1 - t0 + kTM - 1) / kTM;
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
  const int* pos = reinterpret_cast<const int*>(a.pool + ldp->pos_off) + (size_t)unit * cap;
  float* acc = reinterpret_cast<float*>(a.pool + ldp->acc_off) + (size_t)unit * cap;

  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int j = 0; j < 3; ++j) {
      mbar_init(bar_sfull(j), 1);
      mbar_init(bar_sfree(j), 4);  // one arrival per token warp
    }
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "n"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid >= 64 && tid < 64 + kTM) {
    const int h = tid - 64;
    const float* lse = a.logits + ldp->lse_off + (size_t)unit * G;
    // columns past the group read +inf here, so their weight is exp2(-inf) = 0
    s_nlse[h] = (h < G) ? -lse[h] : -INFINITY;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      // rows of this unit in the [rows][64] views of the pool and of q (tensor maps)
      const long long k_row0 = ldp->k_off / (kD * 2) + (long long)unit * cap;
      const long long q_row0 = (long long)(tok * a.n_q_head + (size_t)kvh * G);
      mbar_expect_tx(bar_q, n_cols * 128);
      tma_load_2d(s_u32(q_s), &tm_q, 0, (int)q_row0, bar_q);
      int issued = 0;
      for (int i = 0; i < n_tiles; ++i) {
        const int st = i % STAGES;
        if (i >= STAGES && !mbar_wait(bar_empty(st), ((i / STAGES) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(bar_full(st), kTileBytes);
        tma_load_2d(s_u32(k_s + st * kTileBytes), &tm_k, 0, (int)(k_row0 + t0 + i * kTM), bar_full(st));
        issued = i + 1;
      }
      if (*abort_flag) {
        // copies in flight must land before the CTA's shared memory is released
        mbar_wait(bar_q, 0, abort_flag);
        for (int i = max(0, issued - STAGES); i < issued; ++i)
          for (int k = 0; k < kSpinLimit && !mbar_try_wait(bar_full(i % STAGES), (i / STAGES) & 1); ++k) {
          }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: S^T = K_tile Q^T ----------------
    const uint32_t q_addr = s_u32(q_s);
    const uint32_t id = idesc_n(n_cols);
    bool ok = mbar_wait(bar_q, 0, abort_flag);
    for (int i = 0; ok && i < n_tiles; ++i) {
      const int st = i % STAGES, use = i / n_buf, j = i - use * n_buf;
      ok = mbar_wait(bar_full(st), (i / STAGES) & 1, abort_flag);
      if (ok && use >= 1) ok = mbar_wait(bar_sfree(j), (use - 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) {
        const uint32_t k_addr = s_u32(k_s + st * kTileBytes);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k)
          umma_bf16(tmem_base + j * buf_cols, umma_desc(k_addr + k * 32), umma_desc(q_addr + k * 32), id, k > 0 ? 1u : 0u);
        umma_commit(bar_empty(st));
        umma_commit(bar_sfull(j));
      }
      __syncwarp();
    }
  } else {
    // ---------------- thread = one token ----------------
    const int quarter = warp & 3, set = (warp - 2) >> 2;
    constexpr int kThreads = 64 + 128 * SETS;
    (void)kThreads;
    const int row = quarter * 32 + lane;
    const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
    const int n32 = G >> 5, n8 = ((G & 31) + 7) >> 3;
    const float c = a.scale_log2;
    unsigned long long best = ~0ull;
    int best_slot = -1;
    bool ok = true;
    for (int i = set; ok && i < n_tiles; i += SETS) {
      const int use = i / n_buf, j = i - use * n_buf;
      const int slot = t0 + i * kTM + row;
      const bool valid = slot < t1;
      // the score and position loads overlap the wait for the accumulator
      float old = 0.f;
      int p = 0x7fffffff;
      if (valid) {
        old = acc[slot];
        if (full) p = pos[slot];
      }
      ok = __all_sync(kFull, mbar_wait(bar_sfull(j), use & 1, abort_flag));  // tcgen05.ld is warp-wide
      if (!ok) break;
      tc_fence_after();
      const uint32_t s_addr = tmem_base + lane_sel + j * buf_cols;
      float g0 = 0.f, g1 = 0.f;
      auto add32 = [&](const uint32_t (&r)[32], int ch) {
        const float4* nl = reinterpret_cast<const float4*>(s_nlse + ch * 32);
#pragma unroll
        for (int q4 = 0; q4 < 8; ++q4) {
          const float4 l4 = nl[q4];
          g0 += ex2(fmaf(__uint_as_float(r[q4 * 4]), c, l4.x));
          g1 += ex2(fmaf(__uint_as_float(r[q4 * 4 + 1]), c, l4.y));
          g0 += ex2(fmaf(__uint_as_float(r[q4 * 4 + 2]), c, l4.z));
          g1 += ex2(fmaf(__uint_as_float(r[q4 * 4 + 3]), c, l4.w));
        }
      };
      // the next chunk's tensor-memory load is in flight while this one is summed
      uint32_t ra[32], rb[32];
      tmem_ld32_nowait(s_addr, ra);
#pragma unroll 1
      for (int ch = 0; ch < n32; ch += 2) {
        tmem_wait_ld(ra);
        if (ch + 1 < n32) tmem_ld32_nowait(s_addr + (ch + 1) * 32, rb);
        add32(ra, ch);
        if (ch + 1 < n32) {
          tmem_wait_ld(rb);
          if (ch + 2 < n32) tmem_ld32_nowait(s_addr + (ch + 2) * 32, ra);
          add32(rb, ch + 1);
        }
      }
#pragma unroll 1
      for (int ch = 0; ch < n8; ++ch) {
        float v[8];
        tmem_ld8(s_addr + n32 * 32 + ch * 8, v);
        const float4* nl = reinterpret_cast<const float4*>(s_nlse + n32 * 32 + ch * 8);
#pragma unroll
        for (int q4 = 0; q4 < 2; ++q4) {
          const float4 l4 = nl[q4];
          g0 += ex2(fmaf(v[q4 * 4], c, l4.x));
          g1 += ex2(fmaf(v[q4 * 4 + 1], c, l4.y));
          g0 += ex2(fmaf(v[q4 * 4 + 2], c, l4.z));
          g1 += ex2(fmaf(v[q4 * 4 + 3], c, l4.w));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_sfree(j));
      if (valid) {
        const float v = old + (g0 + g1);
        acc[slot] = v;
        if (full && p <= thr) {
          const unsigned long long r = victim_rank(v, p);
          if (r < best) {
            best = r;
            best_slot = slot;
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long r2 = __shfl_xor_sync(kFull, best, o);
      const int s2 = __shfl_xor_sync(kFull, best_slot, o);
      if (r2 < best) {
        best = r2;
        best_slot = s2;
      }
    }
    if (lane == 0) {
      s_cand[set * 4 + quarter].rank = best;
      s_cand[set * 4 + quarter].slot = best_slot;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(TMEM_COLS) : "memory");
  }
  if (tid != 0) return;
  if (*abort_flag) {
    atomicOr(a.status, kStatusTimeout);
    return;
  }
  if (!full) return;  // the cache still grows: the next token takes a fresh slot
  Candidate best = s_cand[0];
  for (int q = 1; q < 4 * SETS; ++q)
    if (s_cand[q].rank < best.rank) best = s_cand[q];
  // looked up again rather than carried through the token loop: the registers are needed there
  if (!locate<UNIFORM, Args>(a, blockIdx.x, it)) return;
  const LayerDesc* ldt = a.layers + it.layer;
  const int unit_t = it.local / it.n_split, split_t = it.local - unit_t * it.n_split;
  int* victim = reinterpret_cast<int*>(a.pool + ldt->victim_off) + unit_t;
  if (it.n_split == 1) {
    *victim = best.slot;
    return;
  }
  // split-K: park this piece's candidate where its attention partials were, take a ticket
  Candidate* parked = reinterpret_cast<Candidate*>(a.part_stat + ((size_t)it.base + (size_t)unit_t * it.n_split) * a.group * kStatStride);
  const size_t stride = (size_t)a.group * kStatStride * sizeof(float) / sizeof(Candidate);
  parked[split_t * stride] = best;
  __threadfence();
  int* ticket = a.tickets + (size_t)it.layer * a.n_unit + unit_t;
  if (atomicAdd(ticket, 1) != it.n_split - 1) return;
  __threadfence();
  *ticket = 0;
  unsigned long long br = ~0ull;
  int bs = -1;
  for (int s = 0; s < it.n_split; ++s) {
    const unsigned long long r = __ldcg(&parked[s * stride].rank);
    const int sl = __ldcg(&parked[s * stride].slot);
    if (r < br) {
      br = r;
      bs = sl;
    }
  }
  *victim = bs;
}

// Returns cudaErrorNotSupported when the shape is outside this kernel's range.
cudaError_t launch_h2o_gain_tc(const DecodeArgs& a, int n_items, size_t pool_bytes, size_t q_rows, cudaStream_t s) {
  if (a.head_dim != kD || a.group <= 32 || a.group > 128) return cudaErrorNotSupported;
  const long long pool_rows = (long long)(pool_bytes / (kD * 2));
  if (pool_rows + kTM > 0x7fffffffLL || (long long)q_rows + kTM > 0x7fffffffLL) return cudaErrorNotSupported;
  const int n_cols = (a.group + 15) & ~15;
  CUtensorMap tm_q, tm_k;
  if (!make_tile_map(&tm_q, a.q, (long long)q_rows, kD, n_cols) || !make_tile_map(&tm_k, a.pool, pool_rows, kD, kTM))
    return cudaErrorNotSupported;
  constexpr int kStages = 4, kSets = 2, kTmemCols = 256;
  constexpr size_t smem = 1024 + (size_t)kTM * 128 + (size_t)kStages * kTileBytes + 18 * 8 + kTM * 4 + 8 * sizeof(Candidate);
  auto kern_u = h2o_gain_tc_kernel<kStages, kSets, kTmemCols, 2, 1, DecodeArgsBase>;
  auto kern_s = h2o_gain_tc_kernel<kStages, kSets, kTmemCols, 2, 0, DecodeArgs>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern_u, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern_s, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int n_buf = kTmemCols == 128 ? 1 : (3 * n_cols <= kTmemCols ? 3 : 2);
  if (a.uniform) kern_u<<<n_items, 64 + 128 * kSets, smem, s>>>(tm_q, tm_k, a, n_cols, n_buf);  // sliced: no table
  else kern_s<<<n_items, 64 + 128 * kSets, smem, s>>>(tm_q, tm_k, a, n_cols, n_buf);
  return cudaGetLastError();
}

}  // namespace sq
