// sq_prompt_scores_static: H2O prompt scores without any allocation, for callers that
// cannot obtain device memory of their own.  The intermediate the scoring kernels need (one
// log-sum-exp per query row) lives in a fixed array inside the library image.
#include <mutex>

#include "sq_internal.h"

namespace {

constexpr long long kMaxRows = SQ_STATIC_SCORE_MAX_ROWS;  // batch * n_q_head * prompt_len
constexpr int kMaxDevices = 64;

// Row log-sum-exp scratch.  Every GPU that loads the library holds these 4 MiB until the
// process exits.  The name below is only a handle in host code: the device address comes
// from cudaGetSymbolAddress.
static __device__ __align__(256) float g_row_lse_scratch[kMaxRows];

std::mutex g_mu;
float* g_scratch_ptr[kMaxDevices] = {nullptr};

}  // namespace

extern "C" int sq_prompt_scores_static(const void* q_prompt, const void* k_prompt, int32_t batch, int32_t n_q_head,
                                       int32_t n_kv_head, int32_t prompt_len, int32_t head_dim, int32_t dtype,
                                       float* acc_out, void* stream) {
  if (!q_prompt || !k_prompt || !acc_out) return SQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_prompt) | reinterpret_cast<uintptr_t>(k_prompt)) & 15u) return SQ_ERR_INVALID_ARG;
  if (batch < 1 || n_q_head < 1 || n_kv_head < 1 || prompt_len < 1 || n_q_head % n_kv_head) return SQ_ERR_INVALID_ARG;
  if (batch > 65535 || n_q_head > 65535) return SQ_ERR_INVALID_ARG;
  if (dtype != SQ_F32 && dtype != SQ_BF16) return SQ_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return SQ_ERR_UNSUPPORTED;
  if ((long long)batch * n_q_head * prompt_len > kMaxRows) return SQ_ERR_CAPACITY;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SQ_ERR_CUDA;
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
      // set-up, once per device, with that device current
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_row_lse_scratch) != cudaSuccess || !p) return SQ_ERR_CUDA;
      g_scratch_ptr[dev] = static_cast<float*>(p);
    }
    scratch = g_scratch_ptr[dev];
  }
  sq::ScoreArgs a;
  a.q = q_prompt;
  a.k = k_prompt;
  a.lse2 = scratch;
  a.acc_prompt = acc_out;
  a.batch = batch;
  a.n_q_head = n_q_head;
  a.n_kv_head = n_kv_head;
  a.prompt = prompt_len;
  a.head_dim = head_dim;
  if (sq::launch_prefill_scores_alu(a, dtype, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SQ_ERR_CUDA;
  return SQ_OK;
}
