// Layer importance (Section 3 cosine-similarity equation; Algorithm 1, steps 1-4) and the
// layer-wise budget allocator (Algorithm 1, steps 5-12; Appendix A.2).
#include "sq_device.cuh"
#include "sq_internal.h"

namespace sq {

// One warp per token: streams the token's two hidden-state rows once, keeps the three sums
// (A.B, A.A, B.B) in fp32 registers, and adds the token's cosine to the warp's running sum.
// CTA sums go to cta_partial; the CTA that finishes last adds them up in index order (fp64),
// so the result does not depend on scheduling.
// FUSED: the rows are the residual stream (a) and the attention block's output (b); the kernel
// writes their sum, rounded to T, to sum_out and takes the cosine between a and that sum, i.e.
// between the hidden state before and after self-attention, in the pass that produces the latter.
template <typename T, bool FUSED>
__global__ void __launch_bounds__(256) cos_sim_reduce_kernel(ImportanceArgs a) {
  constexpr int EPV = Elem<T>::kPerVec;
  const int nvec = a.hidden / EPV;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long n_warp = (long long)gridDim.x * 8;
  float wsum = 0.f;
  for (long long row = (long long)blockIdx.x * 8 + warp; row < a.n_tok; row += n_warp) {
    const uint4* pa = reinterpret_cast<const uint4*>(a.a) + row * nvec;
    const uint4* pb = reinterpret_cast<const uint4*>(a.b) + row * nvec;
    uint4* po = FUSED ? reinterpret_cast<uint4*>(a.sum_out) + row * nvec : nullptr;
    float dot = 0.f, na = 0.f, nb = 0.f;
    for (int v0 = lane; v0 < nvec; v0 += 128) {
      uint4 va[4], vb[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int v = v0 + 32 * u;
        if (v < nvec) {
          va[u] = ld_stream(pa + v);
          vb[u] = ld_stream(pb + v);
        } else {
          va[u] = make_uint4(0, 0, 0, 0);
          vb[u] = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float fa[EPV], fb[EPV];
        widen<T>(va[u], fa);
        widen<T>(vb[u], fb);
        if (FUSED) {
          // the sum as it is stored: one fp32 addition, rounded to T
          T r[EPV];
#pragma unroll
          for (int e = 0; e < EPV; ++e) {
            r[e] = narrow<T>(fa[e] + fb[e]);
            fb[e] = to_float<T>(r[e]);
          }
          if (v0 + 32 * u < nvec) po[v0 + 32 * u] = *reinterpret_cast<const uint4*>(r);
        }
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
          dot = fmaf(fa[e], fb[e], dot);
          na = fmaf(fa[e], fa[e], na);
          nb = fmaf(fb[e], fb[e], nb);
        }
      }
    }
    dot = warp_sum(dot);
    na = warp_sum(na);
    nb = warp_sum(nb);
    float den = sqrtf(na) * sqrtf(nb);
    wsum += (den > 0.f) ? dot / den : 0.f;
  }
  __shared__ float s_w[8];
  __shared__ bool s_last;
  if (lane == 0) s_w[warp] = wsum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float c = 0.f;
    for (int i = 0; i < 8; ++i) c += s_w[i];
    a.cta_partial[blockIdx.x] = c;
    __threadfence();
    unsigned int t = atomicAdd(a.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (s_last && warp == 0) {
    __threadfence();
    double acc = 0.0;
    for (int i = lane; i < (int)gridDim.x; i += 32) acc += (double)__ldcg(a.cta_partial + i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      *a.cos_sum += acc;
      *a.ticket = 0u;
    }
  }
}

cudaError_t launch_importance(const ImportanceArgs& a, int dtype, int n_cta, cudaStream_t s) {
  if (a.sum_out) {
    if (dtype == SQ_F32) cos_sim_reduce_kernel<float, true><<<n_cta, 256, 0, s>>>(a);
    else cos_sim_reduce_kernel<__nv_bfloat16, true><<<n_cta, 256, 0, s>>>(a);
  } else {
    if (dtype == SQ_F32) cos_sim_reduce_kernel<float, false><<<n_cta, 256, 0, s>>>(a);
    else cos_sim_reduce_kernel<__nv_bfloat16, false><<<n_cta, 256, 0, s>>>(a);
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Budget allocator: one CTA.  The clustering is the exact optimum of one-dimensional k-means
// (optimal clusters of scalars are runs of the sorted values): every cut of the sorted list
// into k runs is costed in fp64 and the cheapest wins, the first in lexicographic order on
// equal cost.  A run's cost is evaluated in index order -- mean = (x0 + x1 + ...)/n, then
// (x0-mean)^2 + (x1-mean)^2 + ... -- with individually rounded operations, so the decision
// is reproducible on any IEEE machine.
// ---------------------------------------------------------------------------------------
__device__ double run_cost(const double* x, int lo, int hi) {
  double s = 0.0;
  for (int i = lo; i < hi; ++i) s = __dadd_rn(s, x[i]);
  double mean = __ddiv_rn(s, (double)(hi - lo));
  double c = 0.0;
  for (int i = lo; i < hi; ++i) {
    double d = __dsub_rn(x[i], mean);
    c = __dadd_rn(c, __dmul_rn(d, d));
  }
  return c;
}

__global__ void __launch_bounds__(256) allocate_budgets_kernel(AllocateArgs a) {
  __shared__ double s_x[kMaxLayers];         // sorted values
  __shared__ int s_idx[kMaxLayers];          // layer of each sorted value
  __shared__ double s_head[kMaxLayers + 1];  // cost of run [0, i)
  __shared__ double s_tail[kMaxLayers + 1];  // cost of run [i, n)
  __shared__ double s_best_cost[256];
  __shared__ int s_best_id[256];
  __shared__ int s_k, s_cut;
  const int n = a.n_layer, tid = threadIdx.x;
  const int st = a.stride, off = blockIdx.x;  // this CTA's budget vector: entries i * st + off

  // layer averages, rounded to fp32 (the value reported to the caller), ranked by (value, layer)
  for (int i = tid; i < n; i += blockDim.x) {
    long long cnt = a.tok_count[i * st + off];
    float c = cnt > 0 ? (float)(a.cos_sum[i * st + off] / (double)cnt) : 0.f;
    a.cos_sim[i * st + off] = c;
    s_head[i] = (double)c;  // scratch: unsorted values
  }
  __syncthreads();
  for (int i = tid; i < n; i += blockDim.x) {
    double v = s_head[i];
    int r = 0;
    for (int j = 0; j < n; ++j) {
      double w = s_head[j];
      r += (w < v) || (w == v && j < i);
    }
    s_x[r] = v;
    s_idx[r] = i;
  }
  __syncthreads();
  if (tid == 0) {
    int distinct = 1;
    for (int i = 1; i < n; ++i) distinct += (s_x[i] != s_x[i - 1]);
    s_k = min(a.n_cluster, distinct);
    s_cut = n;  // G3 = sorted ranks [cut, n)
  }
  __syncthreads();
  for (int i = tid; i <= n; i += blockDim.x) {
    s_head[i] = (i > 0) ? run_cost(s_x, 0, i) : 0.0;
    s_tail[i] = (i < n) ? run_cost(s_x, i, n) : 0.0;
  }
  __syncthreads();
  const int k = s_k;
  double best = 0.0;
  int best_id = -1;
  if (k == 2) {
    for (int i = 1 + tid; i < n; i += blockDim.x) {
      double c = __dadd_rn(s_head[i], s_tail[i]);
      if (best_id < 0 || c < best) {
        best = c;
        best_id = i;
      }
    }
  } else if (k == 3) {
    // candidate id = i * n + j, visited in increasing id per thread
    for (int id = tid; id < n * n; id += blockDim.x) {
      int i = id / n, j = id - i * n;
      if (i < 1 || i > n - 2 || j <= i || j > n - 1) continue;
      double c = __dadd_rn(__dadd_rn(s_head[i], run_cost(s_x, i, j)), s_tail[j]);
      if (best_id < 0 || c < best) {
        best = c;
        best_id = id;
      }
    }
  }
  s_best_cost[tid] = best;
  s_best_id[tid] = best_id;
  __syncthreads();
  if (tid == 0) {
    double bc = 0.0;
    int bi = -1;
    for (int t = 0; t < (int)blockDim.x; ++t) {
      int id = s_best_id[t];
      if (id < 0) continue;
      double c = s_best_cost[t];
      if (bi < 0 || c < bc || (c == bc && id < bi)) {
        bc = c;
        bi = id;
      }
    }
    if (k == 2 && bi >= 0) s_cut = bi;
    if (k == 3 && bi >= 0) s_cut = bi % n;
    // budgets (Algorithm 1, steps 6-12): G3 gets floor(b_init*p), the rest share what is left
    const int cut = s_cut;
    const int n3 = n - cut;
    for (int i = 0; i < n; ++i) {
      a.is_g3[i * st + off] = 0;
      a.budget[i * st + off] = (int)a.b_init;
    }
    if (n3 > 0 && n3 < n) {
      for (int r = cut; r < n; ++r) a.is_g3[s_idx[r] * st + off] = 1;
      long long b_low = (long long)floor(__dmul_rn((double)a.b_init, a.p));
      if (b_low < 1) b_low = 1;
      long long rest = (long long)n * a.b_init - (long long)n3 * b_low;
      long long m = n - n3;
      long long base = rest / m, extra = rest % m;
      long long seen = 0;
      for (int i = 0; i < n; ++i) {
        if (a.is_g3[i * st + off]) {
          a.budget[i * st + off] = (int)b_low;
        } else {
          a.budget[i * st + off] = (int)(base + (seen < extra ? 1 : 0));
          ++seen;
        }
      }
    }
  }
}

cudaError_t launch_allocate(const AllocateArgs& a, cudaStream_t s) {
  allocate_budgets_kernel<<<a.stride, 256, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace sq
