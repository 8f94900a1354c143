// Internal declarations shared by the libsq translation units (host context + kernel launchers).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sq.h"

namespace sq {

constexpr int kMaxLayers = 256;
constexpr int kMaxGroup = 128;          // query heads per KV head
constexpr int kTargetItems = 148 * 16;  // room for split-K pieces beyond one per (layer, unit)

// Per-layer cache geometry, resident in device memory once the budgets are known.
// k/v/pos/acc/victim offsets are BYTES from the pool base; logit_off and lse_off count floats from the
// start of the logits area of the workspace.
struct LayerDesc {
  long long k_off, v_off, pos_off, acc_off, victim_off, logit_off;
  long long lse_off;      // H2O: [unit][group] row log-sum-exps for the score pass of wide groups
  int b;                  // budget: tokens kept per unit
  int cap;                // slots per unit (b rounded up to page_tokens)
  int b_heavy, b_recent;  // H2O split of b
  int ring_base;          // Sliding Window 0, StreamingLLM n_sink: slots below it never rotate
  int ring_origin;        // the position that maps to slot ring_base
};

// Slot of position x in a ring-managed (Sliding Window / StreamingLLM) cache.
__host__ __device__ inline int ring_slot(int x, int b, int base, int origin) {
  if (x < base) return x;
  return base + (x - origin) % (b - base);
}

struct ImportanceArgs {
  const void* a;
  const void* b;
  void* sum_out;         // fused form: receives a + b (rounded to the dtype), which then plays the part of b; else null
  long long n_tok;
  int hidden;
  float* cta_partial;    // [n_cta]
  unsigned int* ticket;  // zero on entry, zero again on exit
  double* cos_sum;       // += sum over tokens of the cosine
};

struct AllocateArgs {  // entry of layer i: [i * stride + blockIdx.x] (one CTA per budget vector)
  const double* cos_sum;
  const long long* tok_count;
  int n_layer, n_cluster, stride;
  long long b_init;
  double p;
  float* cos_sim;
  int* budget;
  unsigned char* is_g3;
};

struct GatherArgs {  // prompt rows -> cache slots of one layer (all its descriptors in one launch)
  const void* k_prompt;
  const void* v_prompt;
  const float* acc_prompt;  // H2O, else null
  char* pool;
  const LayerDesc* descs;   // the layer's descriptors (device); unit u belongs to descs[u / units_per_desc]
  int units_per_desc;
  int n_unit, prompt, max_keep, policy, head_dim;
};

struct ScoreArgs {  // H2O prompt scores of one layer
  const void* q;
  const void* k;
  float* lse2;        // [B, Hq, P]  log2-domain row log-sum-exp
  float* acc_prompt;  // [B, Hkv, P]
  int batch, n_q_head, n_kv_head, prompt, head_dim;
};

// "Layer" below means one cache descriptor: a layer of the whole batch, or, with per-sequence
// budgets, a (layer, sequence) pair holding that sequence's n_kv_head units (batch = 1 then).
struct DecodeArgsBase {
  const LayerDesc* layers;
  const int* order;  // the launch's descriptors, n_layer_total of them, in launch order (largest budget first)
  char* pool;
  float* logits;
  float* part_stat;  // [item][group][4]   (max, sum, sum of rounded weights, pad) in the log2 domain
  float* part_o;     // [item][group][head_dim]
  const void* q;
  const void* k_new;
  const void* v_new;
  void* out;
  int* status;
  int* tickets;  // [n_layer_total][n_unit] arrival counters of the split-K pieces, zero between launches
  int n_layer_total, layer_begin, layer_end;
  int n_tok;  // tokens seen before this step == position of the new token
  int batch, n_q_head, n_kv_head, head_dim, group;
  int n_unit;  // batch * n_kv_head
  int split_tokens, policy;
  int uniform;  // every descriptor of the launch has n_unit items (no split-K): items are found in O(1)
  int has_logits;  // H2O: the workspace holds the per-slot logits the kernels other than the tcgen05 pair need
  float scale_log2;  // log2(e) / sqrt(head_dim)
};
// With split-K: items before the k-th descriptor of the launch (k <= n_layer_total <= kMaxLayers).
// Rides in the kernel parameters, so a lookup is a binary search in constant memory; the kernel
// build for launches without split-K takes the base only (1 KB less to pass per launch).
struct DecodeArgs : DecodeArgsBase {
  int cum[kMaxLayers + 1];
};

struct EvictLayer {  // one layer of an explicit eviction
  LayerDesc ld_old, ld_new;
  int len, n_tok;
};

struct EvictArgs {
  char* pool;
  const EvictLayer* tab;  // [n_layers] in device memory
  int n_layers, max_cap;
  int n_unit, policy, n_sink, row_bytes;
  int* status;
};

// Launchers: each returns the cudaError_t of its launches.
cudaError_t launch_importance(const ImportanceArgs& a, int dtype, int n_cta, cudaStream_t s);
cudaError_t launch_allocate(const AllocateArgs& a, cudaStream_t s);
cudaError_t launch_gather(const GatherArgs& a, int dtype, cudaStream_t s);
cudaError_t launch_prefill_scores(const ScoreArgs& a, int dtype, int* status, cudaStream_t s);
cudaError_t launch_prefill_scores_alu(const ScoreArgs& a, int dtype, cudaStream_t s);
cudaError_t launch_prefill_scores_tc(const ScoreArgs& a, int* status, cudaStream_t s);
cudaError_t launch_select_prompt(const float* acc_prompt, int n_unit, int prompt, const LayerDesc* descs,
                                 int units_per_desc, char* pool, cudaStream_t s);
cudaError_t launch_pick_victim(char* pool, const LayerDesc* descs, int units_per_desc, int n_unit, int prompt,
                               int next_pos, cudaStream_t s);
// desc_tiles: per descriptor of the launch (launch order) the 128-token tiles of one unit
cudaError_t launch_decode(const DecodeArgs& a, int dtype, int n_items, bool need_combine, size_t pool_bytes,
                          size_t q_rows, const int* desc_tiles, cudaStream_t s);
cudaError_t launch_decode_attn_tc(const DecodeArgs& a, int n_items, size_t pool_bytes, size_t q_rows, cudaStream_t s);
cudaError_t launch_decode_attn_tc_stream(const DecodeArgs& a, const int* desc_tiles, size_t pool_bytes, size_t q_rows,
                                         cudaStream_t s);
cudaError_t launch_h2o_gain_tc(const DecodeArgs& a, int n_items, size_t pool_bytes, size_t q_rows, cudaStream_t s);
cudaError_t launch_decode_attn_mma(const DecodeArgs& a, int n_items, cudaStream_t s);
cudaError_t launch_evict(const EvictArgs& a, cudaStream_t s);

}  // namespace sq
