// Tensor-core decode attention for grouped / multi-query heads (bf16): with g query heads
// sharing a KV head the step is a dense [g x d] . [d x tokens] contraction (g flop per byte of
// K/V), too much for the fp32 pipes at HBM speed once g >= 4.  The g heads of a unit are
// padded to 16-row tiles and run through mma.sync m16n8k16 (bf16 in, fp32 accumulate):
//   S = Q K^T   (K tile in shared memory, B operand through ldmatrix)
//   O += P V    (P = exp2(S*scale - max) re-used from the S accumulators as the A operand,
//                V tile through ldmatrix.trans)
// K/V tiles of 64 tokens stream through a multi-stage cp.async pipeline (16-byte copies,
// XOR-swizzled rows so ldmatrix is bank-conflict free).  Warps split the tile's tokens (WN)
// and, for very wide groups, the head tiles (WM); partial results merge through shared memory.
#include "sq_decode_common.cuh"
#include "sq_device.cuh"
#include "sq_internal.h"

namespace sq {

namespace {

constexpr int kTile = 64;  // tokens per pipeline stage

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;  // 0: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// two floats -> packed bf16x2 (lo in the low half), and the values the packing kept
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi, float& lo_r, float& hi_r) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  uint32_t u = *reinterpret_cast<uint32_t*>(&v);
  lo_r = __uint_as_float(u << 16);
  hi_r = __uint_as_float(u & 0xffff0000u);
  return u;
}

template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  // byte offset of 16-byte chunk `chunk` of row `row` inside a [rows][D] bf16 tile
  return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

}  // namespace

template <int D, int MT, int WM, int WN, int STAGES>
__global__ void __launch_bounds__(32 * WM * WN) decode_attn_mma_kernel(DecodeArgs a) {
  constexpr int NT = 32 * WM * WN;
  constexpr int CH = D / 8;            // 16-byte chunks per row
  constexpr int KS = D / 16;           // k-steps of Q K^T / pairs of output n-blocks
  constexpr int NB = D / 8;            // output n-blocks of 8 columns
  constexpr int QROWS = WM * MT * 16;  // padded head rows
  constexpr int TILE_BYTES = kTile * D * 2;
  static_assert(kTile / WN == 16, "each warp owns 16 tokens of a tile");
  using bf16 = __nv_bfloat16;
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* q_s = smem;
  unsigned char* k_s = smem + QROWS * D * 2;
  unsigned char* v_s = k_s + STAGES * TILE_BYTES;

  ItemLoc it;
  if (!locate(a, blockIdx.x, it)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp / WN, wn = warp % WN;
  const int gq = lane >> 2, tq = lane & 3;
  const LayerDesc* ldp = a.layers + it.layer;
  const int b = ldp->b, cap = ldp->cap, G = a.group;
  const int unit = it.local / it.n_split, split = it.local - unit * it.n_split;
  const int len = min(a.n_tok + 1, b);
  const bool h2o = (a.policy == SQ_POLICY_H2O);
  int w;
  if (h2o) {
    w = (a.n_tok < b) ? a.n_tok : reinterpret_cast<const int*>(a.pool + ldp->victim_off)[unit];
    if (w < 0 || w >= b) {
      if (tid == 0) atomicOr(a.status, 2);
      w = 0;
    }
  } else {
    w = ring_slot(a.n_tok, b, ldp->ring_base, ldp->ring_origin);
  }
  const int t0 = split * a.split_tokens, t1 = min(len, t0 + a.split_tokens);
  const int seq = unit / a.n_kv_head, kvh = unit - seq * a.n_kv_head;
  const size_t tok = (size_t)(it.layer - a.layer_begin) * a.batch + seq;
  bf16* Kb = reinterpret_cast<bf16*>(a.pool + ldp->k_off) + (size_t)unit * cap * D;
  bf16* Vb = reinterpret_cast<bf16*>(a.pool + ldp->v_off) + (size_t)unit * cap * D;
  const bf16* qb = reinterpret_cast<const bf16*>(a.q) + (tok * a.n_q_head + (size_t)kvh * G) * D;
  const bf16* kn = reinterpret_cast<const bf16*>(a.k_new) + (tok * a.n_kv_head + kvh) * D;
  const bf16* vn = reinterpret_cast<const bf16*>(a.v_new) + (tok * a.n_kv_head + kvh) * D;
  bf16* ob = reinterpret_cast<bf16*>(a.out) + (tok * a.n_q_head + (size_t)kvh * G) * D;
  float* logit = a.logits + ldp->logit_off + (size_t)unit * cap * G;
  float* stat = a.part_stat + (size_t)blockIdx.x * G * kStatStride;
  float* po = a.part_o + (size_t)blockIdx.x * G * D;

  // the CTA whose range holds slot w stores the new token first, then reads it like any other
  if (w >= t0 && w < t1) {
    if (tid < 2 * CH) {
      const bool is_v = tid >= CH;
      const int c = is_v ? tid - CH : tid;
      const uint4 val = *reinterpret_cast<const uint4*>((is_v ? vn : kn) + c * 8);
      *reinterpret_cast<uint4*>((is_v ? Vb : Kb) + (size_t)w * D + c * 8) = val;
    }
    if (tid == 2 * CH) {
      reinterpret_cast<int*>(a.pool + ldp->pos_off)[(size_t)unit * cap + w] = a.n_tok;
      if (h2o) reinterpret_cast<float*>(a.pool + ldp->acc_off)[(size_t)unit * cap + w] = 0.f;
    }
    __threadfence_block();
  }
  // query rows (zero beyond the group) into shared memory
  for (int i = tid; i < QROWS * CH; i += NT) {
    const int row = i / CH, c = i - row * CH;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (row < G) val = *reinterpret_cast<const uint4*>(qb + (size_t)row * D + c * 8);
    *reinterpret_cast<uint4*>(q_s + swz<D>(row, c)) = val;
  }
  __syncthreads();

  const int n_tiles = (t1 - t0 + kTile - 1) / kTile;
  auto load_tile = [&](int tile) {
    if (tile < n_tiles) {
      const int stage = tile % STAGES;
      const int row0 = t0 + tile * kTile;
      const uint32_t kdst = smem_u32(k_s + stage * TILE_BYTES), vdst = smem_u32(v_s + stage * TILE_BYTES);
      for (int i = tid; i < kTile * CH; i += NT) {
        const int r = i / CH, c = i - r * CH;
        const bool ok = row0 + r < t1;
        const size_t src = (size_t)(ok ? row0 + r : t0) * D + c * 8;
        const uint32_t off = swz<D>(r, c);
        cp_async16(kdst + off, Kb + src, ok);
        cp_async16(vdst + off, Vb + src, ok);
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) load_tile(s);

  // A fragments of Q, kept for the whole item
  uint32_t qa[MT][KS][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int mi = lane >> 3, r = lane & 7;
    const int row = (wm * MT + mt) * 16 + (mi & 1) * 8 + r;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
      ldmatrix_x4(smem_u32(q_s + swz<D>(row, 2 * ks + (mi >> 1))), qa[mt][ks][0], qa[mt][ks][1], qa[mt][ks][2],
                  qa[mt][ks][3]);
  }
  float o[MT][NB][4];
  float m_run[MT][2], l_true[MT][2], l_w[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int j = 0; j < 4; ++j) o[mt][nb][j] = 0.f;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      m_run[mt][hf] = -INFINITY;
      l_true[mt][hf] = 0.f;
      l_w[mt][hf] = 0.f;
    }
  }

  for (int tile = 0; tile < n_tiles; ++tile) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    load_tile(tile + STAGES - 1);
    const int stage = tile % STAGES;
    const uint32_t kst = smem_u32(k_s + stage * TILE_BYTES), vst = smem_u32(v_s + stage * TILE_BYTES);
    const int tok0 = t0 + tile * kTile + wn * 16;  // first token of this warp's 16
    if (tok0 >= t1) continue;                      // warp-uniform: nothing of this tile is ours

    // ---- S = Q K^T over the warp's 16 tokens (two 8-token blocks) ----
    float s[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int j = 0; j < 4; ++j) s[mt][nb][j] = 0.f;
    {
      const int mi = lane >> 3, r = lane & 7;
      const int trow = wn * 16 + (mi >> 1) * 8 + r;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(kst + swz<D>(trow, 2 * ks + (mi & 1)), b0, b1, b2, b3);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if ((wm * MT + mt) * 16 < G) {
            mma_bf16(s[mt][0], qa[mt][ks], b0, b1);
            mma_bf16(s[mt][1], qa[mt][ks], b2, b3);
          }
        }
      }
    }
    // ---- online softmax in the log2 domain; P packed to bf16 as the next A operand ----
    uint32_t pa[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        float v[4];
#pragma unroll
        for (int nb = 0; nb < 2; ++nb)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int t = tok0 + nb * 8 + 2 * tq + j;
            v[nb * 2 + j] = (t < t1) ? s[mt][nb][hf * 2 + j] * a.scale_log2 : -INFINITY;
          }
        if (h2o) {
          const int h = (wm * MT + mt) * 16 + hf * 8 + gq;
          if (h < G) {
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                const int t = tok0 + nb * 8 + 2 * tq + j;
                if (t < t1) logit[(size_t)t * G + h] = v[nb * 2 + j];
              }
          }
        }
        float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
        const float m_new = fmaxf(m_run[mt][hf], mx);  // finite: token tok0 is valid
        const float corr = exp2f(m_run[mt][hf] - m_new);
        m_run[mt][hf] = m_new;
        float p[4], pr[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) p[j] = exp2f(v[j] - m_new);
        pa[mt][hf] = pack_bf16(p[0], p[1], pr[0], pr[1]);      // tokens 0-7 of the 16
        pa[mt][hf + 2] = pack_bf16(p[2], p[3], pr[2], pr[3]);  // tokens 8-15
        l_true[mt][hf] = l_true[mt][hf] * corr + ((p[0] + p[1]) + (p[2] + p[3]));
        l_w[mt][hf] = l_w[mt][hf] * corr + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          o[mt][nb][hf * 2] *= corr;
          o[mt][nb][hf * 2 + 1] *= corr;
        }
      }
    }
    // ---- O += P V ----
    {
      const int mi = lane >> 3, r = lane & 7;
      const int trow = wn * 16 + (mi & 1) * 8 + r;
#pragma unroll
      for (int nb2 = 0; nb2 < KS; ++nb2) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(vst + swz<D>(trow, 2 * nb2 + (mi >> 1)), b0, b1, b2, b3);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if ((wm * MT + mt) * 16 < G) {
            mma_bf16(o[mt][2 * nb2], pa[mt], b0, b1);
            mma_bf16(o[mt][2 * nb2 + 1], pa[mt], b2, b3);
          }
        }
      }
    }
  }
  cp_async_wait<0>();
  // sums over the four lanes that share a row
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      l_true[mt][hf] += __shfl_xor_sync(kFull, l_true[mt][hf], 1);
      l_true[mt][hf] += __shfl_xor_sync(kFull, l_true[mt][hf], 2);
      l_w[mt][hf] += __shfl_xor_sync(kFull, l_w[mt][hf], 1);
      l_w[mt][hf] += __shfl_xor_sync(kFull, l_w[mt][hf], 2);
    }
  __syncthreads();  // the pipeline buffers are free: reuse them for the merge

  // ---- merge the WN token groups (tree over shared memory) ----
  constexpr int SLOT_FLOATS = MT * 16 * (D + 4);
  float* mg = reinterpret_cast<float*>(k_s);
#pragma unroll
  for (int stride = WN / 2; stride >= 1; stride >>= 1) {
    float* slot = mg + (size_t)(wm * (WN / 2) + (wn % stride)) * SLOT_FLOATS;
    if (wn >= stride && wn < 2 * stride) {
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float* row = slot + (size_t)(mt * 16 + hf * 8 + gq) * (D + 4);
#pragma unroll
          for (int nb = 0; nb < NB; ++nb)
            *reinterpret_cast<float2*>(row + nb * 8 + 2 * tq) = make_float2(o[mt][nb][hf * 2], o[mt][nb][hf * 2 + 1]);
          if (tq == 0) {
            row[D] = m_run[mt][hf];
            row[D + 1] = l_true[mt][hf];
            row[D + 2] = l_w[mt][hf];
          }
        }
    }
    __syncthreads();
    if (wn < stride) {
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float* row = slot + (size_t)(mt * 16 + hf * 8 + gq) * (D + 4);
          const float m2 = row[D], m1 = m_run[mt][hf];
          const float mx = fmaxf(m1, m2);
          const float f1 = (m1 > -INFINITY) ? exp2f(m1 - mx) : 0.f;
          const float f2 = (m2 > -INFINITY) ? exp2f(m2 - mx) : 0.f;
          m_run[mt][hf] = mx;
          l_true[mt][hf] = l_true[mt][hf] * f1 + row[D + 1] * f2;
          l_w[mt][hf] = l_w[mt][hf] * f1 + row[D + 2] * f2;
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            const float2 o2 = *reinterpret_cast<const float2*>(row + nb * 8 + 2 * tq);
            o[mt][nb][hf * 2] = o[mt][nb][hf * 2] * f1 + o2.x * f2;
            o[mt][nb][hf * 2 + 1] = o[mt][nb][hf * 2 + 1] * f1 + o2.y * f2;
          }
        }
    }
    __syncthreads();
  }
  if (wn == 0) {
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int h = (wm * MT + mt) * 16 + hf * 8 + gq;
      if (h >= G) continue;
      if (it.n_split == 1) {
        const float inv = 1.f / l_w[mt][hf];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          *reinterpret_cast<__nv_bfloat162*>(ob + (size_t)h * D + nb * 8 + 2 * tq) =
              __floats2bfloat162_rn(o[mt][nb][hf * 2] * inv, o[mt][nb][hf * 2 + 1] * inv);
      } else {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          *reinterpret_cast<float2*>(po + (size_t)h * D + nb * 8 + 2 * tq) =
              make_float2(o[mt][nb][hf * 2], o[mt][nb][hf * 2 + 1]);
      }
      if (tq == 0) {
        stat[h * kStatStride] = m_run[mt][hf];
        stat[h * kStatStride + 1] = l_true[mt][hf];
        stat[h * kStatStride + 2] = l_w[mt][hf];
      }
    }
  }
  if (!h2o && it.n_split > 1) merge_if_last<bf16>(a, it, unit);
}

template <int D, int MT, int WM, int WN, int STAGES>
static cudaError_t launch_cfg(const DecodeArgs& a, int n_items, cudaStream_t s) {
  constexpr int QROWS = WM * MT * 16;
  constexpr size_t pipe = (size_t)2 * STAGES * kTile * D * 2;
  constexpr size_t merge = (size_t)WM * (WN / 2) * MT * 16 * (D + 4) * 4;
  static_assert(merge <= pipe, "the merge area reuses the pipeline stages");
  constexpr size_t smem = (size_t)QROWS * D * 2 + pipe;
  auto kern = decode_attn_mma_kernel<D, MT, WM, WN, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  kern<<<n_items, 32 * WM * WN, smem, s>>>(a);
  return cudaGetLastError();
}

// Returns cudaErrorNotSupported when no tensor-core configuration covers the shape.
cudaError_t launch_decode_attn_mma(const DecodeArgs& a, int n_items, cudaStream_t s) {
  const int G = a.group;
  if (a.head_dim == 128) {
    // Two stages of 32 KB let three CTAs share an SM, which wins once the launch has CTAs to
    // spare (measured: Mistral- and Llama-2-70B-shaped fused steps 5-9 % faster); a launch of
    // about one wave (one layer at a time) is better off with the deeper ring per CTA.
    static int n_sm = 0;
    if (n_sm == 0) {
      int dev = 0;
      if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        n_sm = 148;
    }
    const bool many = n_items >= 6 * n_sm;
    if (G <= 16) return many ? launch_cfg<128, 1, 1, 4, 2>(a, n_items, s) : launch_cfg<128, 1, 1, 4, 3>(a, n_items, s);
    if (G <= 32) return many ? launch_cfg<128, 2, 1, 4, 2>(a, n_items, s) : launch_cfg<128, 2, 1, 4, 3>(a, n_items, s);
  } else if (a.head_dim == 64) {
    if (G <= 16) return launch_cfg<64, 1, 1, 4, 4>(a, n_items, s);
    if (G <= 32) return launch_cfg<64, 2, 1, 4, 4>(a, n_items, s);
    if (G <= 96) return launch_cfg<64, 3, 2, 4, 4>(a, n_items, s);
  }
  return cudaErrorNotSupported;
}

}  // namespace sq
