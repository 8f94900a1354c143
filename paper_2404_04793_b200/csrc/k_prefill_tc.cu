// H2O prompt scores on the 5th-generation tensor cores (bf16).
//
// acc[t] = sum over the query heads sharing a KV head and over query rows r >= t of
//          softmax_row_r(Q K^T / sqrt(d))[t]                       (causal)
// is two sweeps over 128x128 tiles of the score matrix, each tile one tcgen05.mma chain
// (M = N = 128, K = head_dim, bf16 in, fp32 accumulators in tensor memory):
//   sweep 1, CTA = (sequence, query head, 128 query rows): S = Q_tile K_tile^T for the key tiles
//     up to the diagonal; thread r of the four softmax warps owns TMEM lane r = one query row and
//     keeps its running max / sum -> row log-sum-exp.
//   sweep 2, CTA = (sequence, KV head, 128 keys): the operands swap, S^T = K_tile Q_tile^T for all
//     query tiles from the diagonal down and all heads of the group; thread t owns one key and
//     adds exp2(s*scale - lse[row]) over the tile's columns -> the key's column sum, with no
//     cross-thread reduction and no atomics (deterministic).
// Roles per CTA (6 warps): warp 0 issues TMA tile loads (128-byte swizzle, every CTA its own tiles) into
// a ring of shared-memory stages; warp 1 allocates tensor memory and issues the MMAs, signalling
// completion through tcgen05.commit -> mbarrier; warps 2-5 drain the accumulators with
// tcgen05.ld.  Two accumulator buffers let the next tile's MMA run under this tile's exponentials.
// Every mbarrier wait is bounded: on expiry the CTA raises a status bit and winds down.
#include <type_traits>

#include "sq_internal.h"
#include "sq_tc.cuh"

namespace sq {

using namespace tc;

// Threads per CTA: a TMA warp, an MMA warp and eight drain warps.  A warp reaches only the 32
// tensor-memory lanes of its quarter (warp index mod 4), so each quarter of the accumulator rows
// is drained by two warps that take 64 of the tile's 128 columns each: four drain warps per
// scheduler (two CTAs per SM) instead of two, so the special-function pipe is fed while other
// warps wait for an accumulator or a tensor-memory load.
constexpr int kPrefillThreads = 64 + 256;

// SWEEP 1: rows = queries, streamed tiles = keys; SWEEP 2: rows = keys, streamed tiles = queries.
template <int D, int STAGES, int SWEEP>
__global__ void __launch_bounds__(kPrefillThreads, 2)
    prefill_scores_tc_kernel(const __grid_constant__ CUtensorMap tm_rows, const __grid_constant__ CUtensorMap tm_stream,
                             ScoreArgs a, float scale_log2, int* status) {
  constexpr int SUB = D / 64;                  // 64-column sub-tiles per operand tile
  constexpr int TILE_BYTES = SUB * kSubBytes;  // one operand tile
  constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTM >> 3) << 17) | ((uint32_t)(kTM >> 4) << 24);
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* a_s = smem;
  unsigned char* b_s = smem + TILE_BYTES;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(b_s + STAGES * TILE_BYTES);
  // barriers (at most 15 of the 16 slots), then the TMEM base, the abort flag and the lse staging
  static_assert(7 + 2 * STAGES <= 16, "barrier block");
  const uint32_t bar_a = s_u32(bars + 0);
  auto bar_full = [&](int s) { return s_u32(bars + 1 + s); };
  auto bar_empty = [&](int s) { return s_u32(bars + 1 + STAGES + s); };
  auto bar_sfull = [&](int b) { return s_u32(bars + 1 + 2 * STAGES + b); };
  auto bar_sfree = [&](int b) { return s_u32(bars + 3 + 2 * STAGES + b); };
  auto bar_lse = [&](int b) { return s_u32(bars + 5 + 2 * STAGES + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* lse_s = reinterpret_cast<float*>(tmem_slot + 4);  // [2][128], sweep 2 only

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int P = a.prompt, g = a.n_q_head / a.n_kv_head;
  const int n_tile = (P + kTM - 1) / kTM;
  // grid = (head, sequence, tile): the tile index varies slowest, so the CTAs with the most streamed
  // tiles of every head and sequence start first and the short ones fill the tail of the launch
  const int bi = blockIdx.y;
  int row_tile, n_stream;
  long long rows0;  // first row of this CTA's fixed tile in the rows tensor
  int hq = 0, hk = 0;
  if (SWEEP == 1) {
    hq = blockIdx.x;
    hk = hq / g;
    row_tile = n_tile - 1 - blockIdx.z;  // longest rows first
    n_stream = row_tile + 1;
    rows0 = ((long long)bi * a.n_q_head + hq) * P + (long long)row_tile * kTM;
  } else {
    hk = blockIdx.x;
    row_tile = blockIdx.z;               // key tile 0 sees every query tile: longest first
    n_stream = g * (n_tile - row_tile);
    rows0 = ((long long)bi * a.n_kv_head + hk) * P + (long long)row_tile * kTM;
  }
  // first row of streamed tile i, and (sweep 2) its head / query tile
  auto stream_row0 = [&](int i, int& h_out, int& qt_out) -> long long {
    if (SWEEP == 1) {
      h_out = 0;
      qt_out = i;
      return ((long long)bi * a.n_kv_head + hk) * P + (long long)i * kTM;
    }
    const int per = n_tile - row_tile;
    h_out = i / per;
    qt_out = row_tile + (i - h_out * per);
    return ((long long)bi * a.n_q_head + hk * g + h_out) * P + (long long)qt_out * kTM;
  };

  if (tid == 0) {
    mbar_init(bar_a, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_sfull(b), 1);
      mbar_init(bar_sfree(b), 256);
      mbar_init(bar_lse(b), 256);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(s_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      mbar_expect_tx(bar_a, TILE_BYTES);
#pragma unroll
      for (int sb = 0; sb < SUB; ++sb) tma_load_2d(s_u32(a_s + sb * kSubBytes), &tm_rows, sb * 64, (int)rows0, bar_a);
      int issued = 0;
      for (int i = 0; i < n_stream; ++i) {
        const int st = i % STAGES;
        if (i >= STAGES && !mbar_wait(bar_empty(st), ((i / STAGES) - 1) & 1, abort_flag)) break;
        int h, qt;
        const long long r0 = stream_row0(i, h, qt);
        mbar_expect_tx(bar_full(st), TILE_BYTES);
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb)
          tma_load_2d(s_u32(b_s + st * TILE_BYTES + sb * kSubBytes), &tm_stream, sb * 64, (int)r0, bar_full(st));
        issued = i + 1;
      }
      if (*abort_flag) {
        // winding down early: let the copies already in flight land before the CTA exits
        mbar_wait(bar_a, 0, abort_flag);
        for (int i = max(0, issued - STAGES); i < issued; ++i) {
          for (int k = 0; k < kSpinLimit && !mbar_try_wait(bar_full(i % STAGES), (i / STAGES) & 1); ++k) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    bool ok = mbar_wait(bar_a, 0, abort_flag);
    for (int i = 0; ok && i < n_stream; ++i) {
      const int st = i % STAGES, buf = i & 1;
      ok = mbar_wait(bar_full(st), (i / STAGES) & 1, abort_flag);
      if (ok && i >= 2) ok = mbar_wait(bar_sfree(buf), ((i >> 1) - 1) & 1, abort_flag);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (lane == 0) {
        const uint32_t d_tmem = tmem_base + buf * kTM;
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t a_addr = s_u32(a_s + (k / 4) * kSubBytes) + (k % 4) * 32;
          const uint32_t b_addr = s_u32(b_s + st * TILE_BYTES + (k / 4) * kSubBytes) + (k % 4) * 32;
          umma_bf16(d_tmem, umma_desc(a_addr), umma_desc(b_addr), kIdesc, k > 0 ? 1u : 0u);
        }
        umma_commit(bar_empty(st));  // the stage may be refilled once these MMAs have read it
        umma_commit(bar_sfull(buf)); // the accumulator buffer is complete
      }
      __syncwarp();
    }
  } else {
    // ---------------- accumulator drain: thread = one row of the fixed tile ----------------
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;  // which 64 columns of every tile this warp drains
    const int row = quarter * 32 + lane;
    const int row_idx = row_tile * kTM + row;  // query index (sweep 1) / key index (sweep 2)
    const int t256 = (warp - 2) * 32 + lane;
    float m = -INFINITY, l = 0.f, colsum = 0.f;
    bool ok = true;
    // sweep 2: the row log-sum-exp of query t256 of streamed tile i; fetched one tile ahead, so
    // that its trip to memory runs under the previous tile's arithmetic
    auto fetch_lse = [&](int i) -> float {
      int h, qt;
      stream_row0(i, h, qt);
      const int q = qt * kTM + t256;
      return (q < P) ? a.lse2[((size_t)bi * a.n_q_head + hk * g + h) * P + q] : INFINITY;
    };
    float lse_next = 0.f;
    if (SWEEP == 2 && t256 < kTM && n_stream > 0) lse_next = fetch_lse(0);
    for (int i = 0; ok && i < n_stream; ++i) {
      const int buf = i & 1;
      int h, qt;
      stream_row0(i, h, qt);
      if (SWEEP == 2) {
        if (t256 < kTM) {
          lse_s[buf * kTM + t256] = lse_next;
          if (i + 1 < n_stream) lse_next = fetch_lse(i + 1);
        }
        mbar_arrive(bar_lse(buf));  // all 128 row sums of this query tile are staged
        ok = mbar_wait(bar_lse(buf), (i >> 1) & 1, abort_flag);
      }
      if (ok) ok = mbar_wait(bar_sfull(buf), (i >> 1) & 1, abort_flag);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // The tile on the diagonal masks half of its elements; every other tile masks none.  The two
      // cases are separate instantiations of the drain loop, so that tiles off the diagonal (all
      // but one per row of tiles) carry no compare / select per element.
      auto drain_tile = [&](auto diag_c) {
        constexpr bool DIAG = decltype(diag_c)::value;
#pragma unroll 1
        for (int c = 2 * half; c < 2 * half + 2; ++c) {
          float v[32];
          tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kTM + c * 32, v);
          if (SWEEP == 1) {
            if (DIAG) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c * 32 + j > row) v[j] = -INFINITY;  // key after the query
            }
            float mx = v[0];
#pragma unroll
            for (int j = 1; j < 32; ++j) mx = fmaxf(mx, v[j]);
            const float m_new = fmaxf(m, mx * scale_log2);
            if (m_new > -INFINITY) {
              float sum = 0.f;
#pragma unroll
              for (int j = 0; j < 32; ++j) sum += ex2(fmaf(v[j], scale_log2, -m_new));
              l = l * ex2(m - m_new) + sum;
              m = m_new;
            }
          } else {
            const float4* ls = reinterpret_cast<const float4*>(lse_s + buf * kTM + c * 32);
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              const float4 lv = ls[j4];
              const float e0 = ex2(fmaf(v[4 * j4 + 0], scale_log2, -lv.x));
              const float e1 = ex2(fmaf(v[4 * j4 + 1], scale_log2, -lv.y));
              const float e2 = ex2(fmaf(v[4 * j4 + 2], scale_log2, -lv.z));
              const float e3 = ex2(fmaf(v[4 * j4 + 3], scale_log2, -lv.w));
              if (DIAG) {
                const int q0 = c * 32 + 4 * j4;  // query before the key: no attention
                colsum += (q0 + 0 >= row ? e0 : 0.f) + (q0 + 1 >= row ? e1 : 0.f) + (q0 + 2 >= row ? e2 : 0.f) +
                          (q0 + 3 >= row ? e3 : 0.f);
              } else {
                colsum += (e0 + e1) + (e2 + e3);
              }
            }
          }
        }
      };
      if (qt == row_tile) drain_tile(std::true_type{});
      else drain_tile(std::false_type{});
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(bar_sfree(buf));
    }
    // the two halves of a row meet in shared memory (the staging area is free once every drain
    // thread is past its last tile); every drain thread reaches both barriers, aborted or not
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (half == 1) {
      lse_s[2 * row] = (SWEEP == 1) ? m : colsum;
      lse_s[2 * row + 1] = l;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (half == 0 && ok && !*abort_flag && row_idx < P) {
      const float o0 = lse_s[2 * row], o1 = lse_s[2 * row + 1];
      if (SWEEP == 1) {
        // this half holds column 0 of every tile, so m is finite; the other half may be empty
        const float mm = fmaxf(m, o0);
        const float ll = l * ex2(m - mm) + o1 * ex2(o0 - mm);
        a.lse2[((size_t)bi * a.n_q_head + hq) * P + row_idx] = mm + log2f(ll);
      } else {
        a.acc_prompt[((size_t)bi * a.n_kv_head + hk) * P + row_idx] = colsum + o0;
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem_base) : "memory");
  }
  if (tid == 0 && *abort_flag) atomicOr(status, kStatusTimeout);
}

// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

namespace tc {
bool make_tile_map(CUtensorMap* tm, const void* base, long long rows, int d, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace tc

template <int D, int STAGES>
static cudaError_t launch_tc_t(const ScoreArgs& a, int* status, cudaStream_t s) {
  CUtensorMap tm_q, tm_k;
  const long long q_rows = (long long)a.batch * a.n_q_head * a.prompt, k_rows = (long long)a.batch * a.n_kv_head * a.prompt;
  if (q_rows + kTM > 0x7fffffffLL) return cudaErrorNotSupported;  // TMA coordinates are 32-bit
  if (!tc::make_tile_map(&tm_q, a.q, q_rows, D, kTM) || !tc::make_tile_map(&tm_k, a.k, k_rows, D, kTM)) return cudaErrorNotSupported;
  constexpr size_t smem = 1024 + (size_t)(1 + STAGES) * (D / 64) * kSubBytes + 8 * 16 + 16 + 2 * kTM * 4;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  const int n_tile = (a.prompt + kTM - 1) / kTM;
  auto k1 = prefill_scores_tc_kernel<D, STAGES, 1>;
  auto k2 = prefill_scores_tc_kernel<D, STAGES, 2>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  k1<<<dim3(a.n_q_head, a.batch, n_tile), kPrefillThreads, smem, s>>>(tm_q, tm_k, a, scale_log2, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  k2<<<dim3(a.n_kv_head, a.batch, n_tile), kPrefillThreads, smem, s>>>(tm_k, tm_q, a, scale_log2, status);
  return cudaGetLastError();
}

// Returns cudaErrorNotSupported when the shape or the driver cannot serve the tensor-core path.
cudaError_t launch_prefill_scores_tc(const ScoreArgs& a, int* status, cudaStream_t s) {
  if (a.n_q_head > 65535 || a.batch > 65535 || (a.prompt + kTM - 1) / kTM > 65535) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(a.q) | reinterpret_cast<uintptr_t>(a.k)) & 15u) return cudaErrorNotSupported;
  if (a.head_dim == 64) return launch_tc_t<64, 4>(a, status, s);
  if (a.head_dim == 128) return launch_tc_t<128, 2>(a, status, s);
  return cudaErrorNotSupported;
}

}  // namespace sq
