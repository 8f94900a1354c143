// Prefill side of Algorithm 1 (step 13 with the first compression of steps 16-18 applied at
// once): H2O prompt scores, C_seq selection over the prompt, and the gather of the kept K/V
// rows into the layer's cache region.
#include <cstdlib>
#include <cstring>

#include "sq_device.cuh"
#include "sq_internal.h"
#include "sq_select.cuh"

namespace sq {

// ---------------------------------------------------------------------------------------
// H2O prompt scores.  acc[t] = sum over the query heads sharing the KV head and over query
// rows r >= t of softmax_row_r(Q K^T / sqrt(d))[t] (causal).  Two passes over 64x64 score
// tiles: row log-sum-exp, then column sums of exp(s - lse).  Thread (tx, ty) of the 16x16
// block owns rows ty+16r and columns tx+16c of a tile (r, c in 0..3).
// ---------------------------------------------------------------------------------------
constexpr int TQ = 64, TK = 64, DC = 32;

template <typename T, int D>
__device__ __forceinline__ void score_tile(const T* __restrict__ qbase, const T* __restrict__ kbase, int q0, int k0,
                                           int P, float (*Qs)[DC + 1], float (*Ks)[DC + 1], float s[4][4]) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) s[r][c] = 0.f;
  for (int dc = 0; dc < D; dc += DC) {
    __syncthreads();
    for (int idx = tid; idx < TQ * DC; idx += 256) {
      int row = idx / DC, col = idx % DC;
      int qr = q0 + row, kr = k0 + row;
      Qs[row][col] = (qr < P) ? to_float<T>(qbase[(size_t)qr * D + dc + col]) : 0.f;
      Ks[row][col] = (kr < P) ? to_float<T>(kbase[(size_t)kr * D + dc + col]) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int dd = 0; dd < DC; ++dd) {
      float qv[4], kv[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) qv[r] = Qs[ty + 16 * r][dd];
#pragma unroll
      for (int c = 0; c < 4; ++c) kv[c] = Ks[tx + 16 * c][dd];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) s[r][c] = fmaf(qv[r], kv[c], s[r][c]);
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(256) prefill_row_lse_kernel(ScoreArgs a, float scale_log2) {
  __shared__ float Qs[TQ][DC + 1], Ks[TK][DC + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int qt = blockIdx.x, hq = blockIdx.y, bi = blockIdx.z;
  const int g = a.n_q_head / a.n_kv_head, P = a.prompt;
  const T* qbase = reinterpret_cast<const T*>(a.q) + ((size_t)bi * a.n_q_head + hq) * P * D;
  const T* kbase = reinterpret_cast<const T*>(a.k) + ((size_t)bi * a.n_kv_head + hq / g) * P * D;
  const int q0 = qt * TQ;
  float m[4], l[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    m[r] = -INFINITY;
    l[r] = 0.f;
  }
  for (int kt = 0; kt <= qt; ++kt) {
    const int k0 = kt * TK;
    float s[4][4];
    score_tile<T, D>(qbase, kbase, q0, k0, P, Qs, Ks, s);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int qr = q0 + ty + 16 * r;
      float tmax = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int kr = k0 + tx + 16 * c;
        s[r][c] = (kr <= qr && qr < P) ? s[r][c] * scale_log2 : -INFINITY;
        tmax = fmaxf(tmax, s[r][c]);
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      const float m_new = fmaxf(m[r], tmax);
      float psum = 0.f;
      if (m_new != -INFINITY) {
#pragma unroll
        for (int c = 0; c < 4; ++c) psum += exp2f(s[r][c] - m_new);
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
      if (m_new != -INFINITY) {
        l[r] = l[r] * exp2f(m[r] - m_new) + psum;
        m[r] = m_new;
      }
    }
  }
  if (tx == 0) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int qr = q0 + ty + 16 * r;
      if (qr < P) a.lse2[((size_t)bi * a.n_q_head + hq) * P + qr] = m[r] + log2f(l[r]);
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(256) prefill_col_sum_kernel(ScoreArgs a, float scale_log2) {
  __shared__ float Qs[TQ][DC + 1], Ks[TK][DC + 1];
  __shared__ float red[16][TK];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int kt = blockIdx.x, hk = blockIdx.y, bi = blockIdx.z;
  const int g = a.n_q_head / a.n_kv_head, P = a.prompt;
  const int n_tile = (P + TQ - 1) / TQ;
  const T* kbase = reinterpret_cast<const T*>(a.k) + ((size_t)bi * a.n_kv_head + hk) * P * D;
  const int k0 = kt * TK;
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  for (int h = 0; h < g; ++h) {
    const int hq = hk * g + h;
    const T* qbase = reinterpret_cast<const T*>(a.q) + ((size_t)bi * a.n_q_head + hq) * P * D;
    const float* lse = a.lse2 + ((size_t)bi * a.n_q_head + hq) * P;
    for (int qt = kt; qt < n_tile; ++qt) {
      const int q0 = qt * TQ;
      float s[4][4];
      score_tile<T, D>(qbase, kbase, q0, k0, P, Qs, Ks, s);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int qr = q0 + ty + 16 * r;
        if (qr >= P) continue;
        const float lr = lse[qr];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int kr = k0 + tx + 16 * c;
          if (kr <= qr) col[c] += exp2f(s[r][c] * scale_log2 - lr);
        }
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < 4; ++c) red[ty][tx + 16 * c] = col[c];
  __syncthreads();
  if (threadIdx.x < TK) {
    float sum = 0.f;
    for (int y = 0; y < 16; ++y) sum += red[y][threadIdx.x];
    const int kr = k0 + threadIdx.x;
    if (kr < P) a.acc_prompt[((size_t)bi * a.n_kv_head + hk) * P + kr] = sum;
  }
}

template <typename T, int D>
static cudaError_t launch_scores_t(const ScoreArgs& a, cudaStream_t s) {
  const int n_tile = (a.prompt + TQ - 1) / TQ;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  prefill_row_lse_kernel<T, D><<<dim3(n_tile, a.n_q_head, a.batch), 256, 0, s>>>(a, scale_log2);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  prefill_col_sum_kernel<T, D><<<dim3(n_tile, a.n_kv_head, a.batch), 256, 0, s>>>(a, scale_log2);
  return cudaGetLastError();
}

// fp32-pipe kernels (any dtype)
cudaError_t launch_prefill_scores_alu(const ScoreArgs& a, int dtype, cudaStream_t s) {
  if (dtype == SQ_F32) {
    return a.head_dim == 64 ? launch_scores_t<float, 64>(a, s) : launch_scores_t<float, 128>(a, s);
  }
  return a.head_dim == 64 ? launch_scores_t<__nv_bfloat16, 64>(a, s) : launch_scores_t<__nv_bfloat16, 128>(a, s);
}

// bf16 prompts go to the tcgen05 kernels; fp32 (and anything those cannot serve) stays on the
// fp32 pipes.
cudaError_t launch_prefill_scores(const ScoreArgs& a, int dtype, int* status, cudaStream_t s) {
  if (dtype == SQ_BF16) {
    cudaError_t e = launch_prefill_scores_tc(a, status, s);
    if (e != cudaErrorNotSupported) return e;
  }
  return launch_prefill_scores_alu(a, dtype, s);
}

// ---------------------------------------------------------------------------------------
// C_seq over the prompt for H2O (one block per unit): keeps the b_recent highest positions
// and, of the others, the b_heavy with the largest score (equal scores: lower position).
// Writes the kept positions in ascending order to the layer's position table.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads) select_prompt_kernel(const float* __restrict__ acc_prompt, int P,
                                                                    const LayerDesc* __restrict__ descs,
                                                                    int units_per_desc, char* pool) {
  __shared__ SelScratch sc;
  const int tid = threadIdx.x;
  const LayerDesc ld = descs[blockIdx.x / units_per_desc];  // the descriptor this unit belongs to
  const int unit = blockIdx.x % units_per_desc;             // its index within the descriptor
  const float* acc = acc_prompt + (size_t)blockIdx.x * P;
  int* pos_out = reinterpret_cast<int*>(pool + ld.pos_off) + (size_t)unit * ld.cap;
  if (P <= ld.b) {
    for (int i = tid; i < P; i += kSelThreads) pos_out[i] = i;
    return;
  }
  const int n_cand = P - ld.b_recent;  // positions [0, n_cand) compete for the heavy slots
  uint32_t thr = 0u;
  unsigned int n_at = 0u, ties = 0u;
  int pos_thr = -1;  // among entries with key == thr keep positions <= pos_thr
  if (ld.b_heavy > 0) {
    auto key = [&](int i) { return score_key(acc[i]); };
    auto all = [&](int) { return true; };
    thr = block_radix_select(sc, n_cand, (unsigned)ld.b_heavy, key, all, &n_at, &ties);
    if (ties == n_at) {
      pos_thr = P;
    } else {
      // the n_at lowest positions among the tied: select on the key (2^31-1 - position)
      auto pkey = [&](int i) { return 0x7fffffffu - (uint32_t)i; };
      auto tied = [&](int i) { return score_key(acc[i]) == thr; };
      unsigned int d0, d1;
      uint32_t pt = block_radix_select(sc, n_cand, n_at, pkey, tied, &d0, &d1);
      pos_thr = (int)(0x7fffffffu - pt);
    }
  }
  int written = 0;
  for (int i0 = 0; i0 < P; i0 += kSelThreads) {
    const int i = i0 + tid;
    bool keep = false;
    if (i < P) {
      if (i >= n_cand) {
        keep = true;
      } else if (ld.b_heavy > 0) {
        uint32_t kk = score_key(acc[i]);
        keep = (kk > thr) || (kk == thr && i <= pos_thr);
      }
    }
    int tot;
    int off = block_excl_count(sc, keep, &tot);
    if (keep && written + off < ld.b) pos_out[written + off] = i;
    written += tot;
  }
}

cudaError_t launch_select_prompt(const float* acc_prompt, int n_unit, int prompt, const LayerDesc* descs,
                                 int units_per_desc, char* pool, cudaStream_t s) {
  select_prompt_kernel<<<n_unit, kSelThreads, 0, s>>>(acc_prompt, prompt, descs, units_per_desc, pool);
  return cudaGetLastError();
}

// First victim of a full H2O cache (the token the next append will replace).
__global__ void __launch_bounds__(kSelThreads) pick_victim_kernel(char* pool, const LayerDesc* __restrict__ descs,
                                                                  int units_per_desc, int prompt, int next_pos) {
  __shared__ SelScratch sc;
  const LayerDesc ld = descs[blockIdx.x / units_per_desc];
  const int unit = blockIdx.x % units_per_desc;
  const int len = min(prompt, ld.b);
  if (len < ld.b) return;  // the cache still grows: the next token takes a fresh slot
  const int* pos = reinterpret_cast<const int*>(pool + ld.pos_off) + (size_t)unit * ld.cap;
  const float* acc = reinterpret_cast<const float*>(pool + ld.acc_off) + (size_t)unit * ld.cap;
  const int thr = next_pos - ld.b_recent;
  unsigned long long best = ~0ull;
  int slot = -1;
  for (int i = threadIdx.x; i < len; i += kSelThreads) {
    int p = pos[i];
    if (p <= thr) {
      unsigned long long r = victim_rank(acc[i], p);
      if (r < best) {
        best = r;
        slot = i;
      }
    }
  }
  slot = block_argmin(sc, best, slot);
  if (threadIdx.x == 0) reinterpret_cast<int*>(pool + ld.victim_off)[unit] = slot;
}

cudaError_t launch_pick_victim(char* pool, const LayerDesc* descs, int units_per_desc, int n_unit, int prompt,
                               int next_pos, cudaStream_t s) {
  pick_victim_kernel<<<n_unit, kSelThreads, 0, s>>>(pool, descs, units_per_desc, prompt, next_pos);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Gather: copies the kept prompt rows of K and V into the unit's slots (16-byte vectors) and
// fills the position (and, for H2O, score) tables.  Sliding Window / StreamingLLM compute the
// kept position of a slot in closed form; H2O reads it from the table the selection wrote.
// ---------------------------------------------------------------------------------------
constexpr int kGatherSlots = 16;

__global__ void __launch_bounds__(256) gather_kernel(GatherArgs a, int row_bytes) {
  const int ug = blockIdx.x, s0 = blockIdx.y * kGatherSlots;  // ug: unit of the batch (sequence, KV head)
  const LayerDesc ld = a.descs[ug / a.units_per_desc];
  const int unit = ug % a.units_per_desc;                     // its index within the descriptor
  const int n_keep = min(a.prompt, ld.b);
  if (s0 >= n_keep) return;                                   // the grid covers the longest descriptor
  const int vpr = row_bytes / 16;  // 16-byte vectors per row
  int* pos_tab = reinterpret_cast<int*>(a.pool + ld.pos_off) + (size_t)unit * ld.cap;
  float* acc_tab = reinterpret_cast<float*>(a.pool + ld.acc_off) + (size_t)unit * ld.cap;
  __shared__ int s_pos[kGatherSlots];
  if (threadIdx.x < kGatherSlots) {
    const int slot = s0 + threadIdx.x;
    int p = -1;
    if (slot < n_keep) {
      if (a.policy == SQ_POLICY_H2O) {
        p = pos_tab[slot];
        acc_tab[slot] = a.acc_prompt ? a.acc_prompt[(size_t)ug * a.prompt + p] : 0.f;
      } else {
        p = (slot < ld.ring_base) ? slot : ld.ring_origin + (slot - ld.ring_base);
        pos_tab[slot] = p;
      }
    }
    s_pos[threadIdx.x] = p;
  }
  __syncthreads();
  const uint4* ksrc = reinterpret_cast<const uint4*>(a.k_prompt) + (size_t)ug * a.prompt * vpr;
  const uint4* vsrc = reinterpret_cast<const uint4*>(a.v_prompt) + (size_t)ug * a.prompt * vpr;
  uint4* kdst = reinterpret_cast<uint4*>(a.pool + ld.k_off) + (size_t)unit * ld.cap * vpr;
  uint4* vdst = reinterpret_cast<uint4*>(a.pool + ld.v_off) + (size_t)unit * ld.cap * vpr;
  for (int idx = threadIdx.x; idx < kGatherSlots * vpr; idx += 256) {
    const int j = idx / vpr, v = idx % vpr;
    const int p = s_pos[j];
    if (p < 0) continue;
    const size_t so = (size_t)p * vpr + v, dofs = (size_t)(s0 + j) * vpr + v;
    kdst[dofs] = ld_stream(ksrc + so);
    vdst[dofs] = ld_stream(vsrc + so);
  }
}

cudaError_t launch_gather(const GatherArgs& a, int dtype, cudaStream_t s) {
  if (a.max_keep <= 0) return cudaSuccess;
  const int row_bytes = a.head_dim * (dtype == SQ_F32 ? 4 : 2);
  dim3 grid(a.n_unit, (a.max_keep + kGatherSlots - 1) / kGatherSlots);
  gather_kernel<<<grid, 256, 0, s>>>(a, row_bytes);
  return cudaGetLastError();
}

}  // namespace sq
