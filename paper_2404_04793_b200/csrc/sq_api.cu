// Host side of libsq: context, memory layout of the caller's pool and workspace, argument
// validation, call-order checks and kernel launches.  See include/sq.h for the contract.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "sq_internal.h"

using namespace sq;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int elem_bytes(int dtype) { return dtype == SQ_F32 ? 4 : 2; }
constexpr int kMaxImportanceCtas = 4096;

struct WsLayout {
  size_t cos_sum, tok_count, cta_partial, ticket, cos_sim, budget, is_g3, status, tickets, layers, order, order_by_layer,
      evict_tab;
  size_t part_stat, part_o, logits, acc_prompt, lse2, total;
  size_t items_cap, logits_floats, lse_floats, n_desc_cap;
};

// Pinned staging for the small host <-> device tables.  "desc" = one cache descriptor: a layer
// of the whole batch, or with per-sequence budgets a (layer, sequence) pair; arrays hold
// n_desc_cap entries, entry of (layer, group) = layer * n_grp + group.
struct HostStage {
  int32_t* budget;
  uint8_t* is_g3;
  float* cos_sim;
  long long* tok_count;
  LayerDesc* layers;
  int* order;           // all descriptors, largest budget first
  int* order_by_layer;  // per layer its descriptors, largest budget first
  EvictLayer* evict_tab;
  void* block;
};

}  // namespace

struct sq_ctx {
  sq_config cfg;
  int64_t b_init_cap;
  char* pool;
  size_t pool_bytes;
  char* ws;
  size_t ws_bytes;
  WsLayout wl;
  HostStage hs;
  cudaEvent_t ev;
  int n_sm;
  int batch, prompt;
  bool per_seq;    // one budget vector per sequence instead of one per batch
  int n_grp;       // descriptors per layer: batch with per-sequence budgets, else 1
  int desc_units;  // units (sequence, KV head) per descriptor
  int n_desc;      // n_layer * n_grp
  bool begun;
  int budget_state;  // 0 none, 1 computed on device (copy in flight), 2 on host, laid out
  int n_tok[kMaxLayers];
  long long imp_tokens[kMaxLayers];  // tokens of a layer seen by sq_layer_importance so far
  bool prefilled[kMaxLayers];
  bool importance_seen[kMaxLayers];
  std::string err;
};

namespace {

int fail(sq_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  return code;
}

int check_config(const sq_config* c, std::string* why) {
  auto bad = [&](const char* m) {
    if (why) *why = m;
    return (int)SQ_ERR_INVALID_ARG;
  };
  if (!c) return bad("config is NULL");
  if (c->n_layer < 1 || c->n_layer > kMaxLayers) return bad("n_layer must be in 1..256");
  if (c->n_kv_head < 1 || c->n_q_head < 1 || c->n_q_head % c->n_kv_head) return bad("n_q_head must be a multiple of n_kv_head");
  if (c->n_q_head / c->n_kv_head > kMaxGroup) return bad("more than 128 query heads per KV head");
  if (c->head_dim != 64 && c->head_dim != 128) {
    if (why) *why = "head_dim must be 64 or 128";
    return (int)SQ_ERR_UNSUPPORTED;
  }
  if (c->hidden < 8 || c->hidden % 8) return bad("hidden must be a positive multiple of 8");
  if (c->max_batch < 1 || c->max_prompt < 1 || c->max_new_tokens < 0) return bad("max_batch/max_prompt/max_new_tokens");
  if (c->dtype != SQ_F32 && c->dtype != SQ_BF16) return bad("dtype");
  if (c->policy < SQ_POLICY_SLIDING_WINDOW || c->policy > SQ_POLICY_H2O) return bad("policy");
  if (c->policy == SQ_POLICY_STREAMING_LLM && c->n_sink < 0) return bad("n_sink");
  if (c->policy == SQ_POLICY_H2O && (c->heavy_den < 1 || c->heavy_num < 0 || c->heavy_num >= c->heavy_den))
    return bad("H2O needs 0 <= heavy_num < heavy_den");
  if (c->n_cluster != 2 && c->n_cluster != 3) return bad("n_cluster must be 2 or 3");
  if (c->page_tokens < 1) return bad("page_tokens must be >= 1");
  if (c->per_sequence_budgets != 0 && c->per_sequence_budgets != 1) return bad("per_sequence_budgets must be 0 or 1");
  return SQ_OK;
}

// H2O decode of 33..128 bf16 query heads per KV head at head_dim 64 runs on the tcgen05 attention
// + score-pass pair, which keeps no per-slot logits.
bool wide_h2o_pair(const sq_config& c) {
  const int G = c.n_q_head / c.n_kv_head;
  return c.policy == SQ_POLICY_H2O && c.dtype == SQ_BF16 && c.head_dim == 64 && G > 32 && G <= kMaxGroup;
}

size_t pool_bytes_for(const sq_config& c, int64_t b_init) {
  const size_t U = (size_t)c.max_batch * c.n_kv_head;
  const size_t tokens = (size_t)c.n_layer * (size_t)b_init + (size_t)c.n_layer * (c.page_tokens - 1);
  size_t per_tok = 2 * (size_t)c.head_dim * elem_bytes(c.dtype) + 4 + (c.policy == SQ_POLICY_H2O ? 4 : 0);
  const size_t n_desc = (size_t)c.n_layer * (c.per_sequence_budgets ? c.max_batch : 1);
  return U * tokens * per_tok + (size_t)c.n_layer * U * 4 + n_desc * 6 * kAlign;
}

WsLayout ws_layout(const sq_config& c, int64_t b_init) {
  WsLayout w{};
  const size_t L = c.n_layer, U = (size_t)c.max_batch * c.n_kv_head, G = c.n_q_head / c.n_kv_head;
  const size_t ND = L * (c.per_sequence_budgets ? (size_t)c.max_batch : 1);
  w.n_desc_cap = ND;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes);
    return o;
  };
  w.cos_sum = take(8 * ND);
  w.tok_count = take(8 * ND);
  w.cta_partial = take(4 * (size_t)kMaxImportanceCtas);
  w.ticket = take(4);
  w.cos_sim = take(4 * ND);
  w.budget = take(4 * ND);
  w.is_g3 = take(ND);
  w.status = take(4);
  w.tickets = take(4 * L * U);
  w.layers = take(sizeof(LayerDesc) * ND);
  w.order = take(4 * ND);
  w.order_by_layer = take(4 * ND);
  w.evict_tab = take(sizeof(EvictLayer) * ND);
  w.items_cap = (size_t)kTargetItems + U * L;
  w.part_stat = take(w.items_cap * G * 4 * 4);
  w.part_o = take(w.items_cap * G * c.head_dim * 4);
  const bool h2o = c.policy == SQ_POLICY_H2O;
  // H2O: row log-sum-exps [unit][group] per layer, then (unless the shape is served by the
  // tcgen05 pair, which recomputes the logits) the logits of every slot
  w.lse_floats = h2o ? U * G * L : 0;
  w.logits_floats = (h2o && !wide_h2o_pair(c)) ? U * G * (L * (size_t)b_init + L * (c.page_tokens - 1)) : 0;
  w.logits = take((w.lse_floats + w.logits_floats) * 4);
  w.acc_prompt = take(h2o ? U * (size_t)c.max_prompt * 4 : 0);
  w.lse2 = take(h2o ? (size_t)c.max_batch * c.n_q_head * c.max_prompt * 4 : 0);
  w.total = off;
  return w;
}

template <typename T>
T* ws_ptr(sq_ctx* c, size_t off) {
  return reinterpret_cast<T*>(c->ws + off);
}

#define SQ_CUDA(c, expr)                                                                         \
  do {                                                                                           \
    cudaError_t e__ = (expr);                                                                    \
    if (e__ != cudaSuccess)                                                                      \
      return fail((c), SQ_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__));        \
  } while (0)

// Launch orders: all descriptors by budget (the fused launch starts the longest first), and
// the same within each layer (launches over a sub-range of layers).
void sort_orders(sq_ctx* c) {
  const int nd = c->n_desc, ng = c->n_grp;
  std::vector<int> ord(nd);
  for (int d = 0; d < nd; ++d) ord[d] = d;
  auto by_budget = [&](int x, int y) { return c->hs.budget[x] > c->hs.budget[y]; };
  std::stable_sort(ord.begin(), ord.end(), by_budget);
  std::copy(ord.begin(), ord.end(), c->hs.order);
  for (int d = 0; d < nd; ++d) ord[d] = d;
  for (int l = 0; l < c->cfg.n_layer; ++l) std::stable_sort(ord.begin() + l * ng, ord.begin() + (l + 1) * ng, by_budget);
  std::copy(ord.begin(), ord.end(), c->hs.order_by_layer);
}

// Computes the cache geometry for the budgets in hs.budget and uploads it.
int build_layout(sq_ctx* c, cudaStream_t st) {
  const sq_config& cfg = c->cfg;
  const size_t U = (size_t)c->desc_units, G = cfg.n_q_head / cfg.n_kv_head;
  const size_t row = (size_t)cfg.head_dim * elem_bytes(cfg.dtype);
  const bool h2o = cfg.policy == SQ_POLICY_H2O;
  size_t off = 0, lfl = 0, lse = 0;
  const bool slot_logits = h2o && !wide_h2o_pair(cfg);
  for (int d = 0; d < c->n_desc; ++d) {
    LayerDesc& ld = c->hs.layers[d];
    const int b = c->hs.budget[d];
    if (b < 1) return fail(c, SQ_ERR_INVALID_ARG, "a layer budget is below 1");
    if (cfg.policy == SQ_POLICY_STREAMING_LLM && b <= cfg.n_sink)
      return fail(c, SQ_ERR_INVALID_ARG, "StreamingLLM needs every layer budget above n_sink");
    ld.b = b;
    ld.cap = (b + cfg.page_tokens - 1) / cfg.page_tokens * cfg.page_tokens;
    ld.b_heavy = h2o ? (int)(((long long)b * cfg.heavy_num) / cfg.heavy_den) : 0;
    ld.b_recent = b - ld.b_heavy;
    ld.ring_base = (cfg.policy == SQ_POLICY_STREAMING_LLM) ? cfg.n_sink : 0;
    ld.ring_origin = std::max(ld.ring_base, c->prompt - (b - ld.ring_base));
    ld.k_off = (long long)off;
    off = align_up(off + U * ld.cap * row);
    ld.v_off = (long long)off;
    off = align_up(off + U * ld.cap * row);
    ld.pos_off = (long long)off;
    off = align_up(off + U * ld.cap * 4);
    ld.acc_off = (long long)off;
    if (h2o) off = align_up(off + U * ld.cap * 4);
    ld.victim_off = (long long)off;
    off = align_up(off + U * 4);
    ld.lse_off = (long long)lse;
    if (h2o) lse += U * G;
    ld.logit_off = (long long)(c->wl.lse_floats + lfl);
    if (slot_logits) lfl += U * ld.cap * G;
  }
  if (off > c->pool_bytes) return fail(c, SQ_ERR_CAPACITY, "budgets do not fit the cache pool");
  if (lfl > c->wl.logits_floats) return fail(c, SQ_ERR_CAPACITY, "budgets do not fit the workspace");
  sort_orders(c);
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<LayerDesc>(c, c->wl.layers), c->hs.layers, sizeof(LayerDesc) * c->n_desc,
                             cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.order), c->hs.order, 4 * c->n_desc, cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.order_by_layer), c->hs.order_by_layer, 4 * c->n_desc,
                             cudaMemcpyHostToDevice, st));
  // the staging block is reused by later calls: make sure the copies have left it
  SQ_CUDA(c, cudaStreamSynchronize(st));
  c->budget_state = 2;
  return SQ_OK;
}

int ensure_budgets(sq_ctx* c, cudaStream_t st) {
  if (c->budget_state == 2) return SQ_OK;
  if (c->budget_state == 0) return fail(c, SQ_ERR_STATE, "budgets not set: call sq_allocate_budgets or sq_set_budgets first");
  SQ_CUDA(c, cudaEventSynchronize(c->ev));
  return build_layout(c, st);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// User-facing arrays are [n_layer] (one budget vector per batch) or [batch][n_layer]
// (per-sequence budgets); internally entry (layer, group) sits at layer * n_grp + group.
inline int user_index(const sq_ctx* c, int layer, int grp) { return grp * c->cfg.n_layer + layer; }

}  // namespace

extern "C" {

int sq_query_sizes(const sq_config* cfg, int64_t b_init, size_t* pool_bytes, size_t* workspace_bytes) {
  int rc = check_config(cfg, nullptr);
  if (rc != SQ_OK) return rc;
  if (b_init < 1 || !pool_bytes || !workspace_bytes) return SQ_ERR_INVALID_ARG;
  *pool_bytes = pool_bytes_for(*cfg, b_init);
  *workspace_bytes = ws_layout(*cfg, b_init).total;
  return SQ_OK;
}

int sq_ctx_create(const sq_config* cfg, int64_t b_init, void* pool, size_t pool_bytes, void* workspace,
                  size_t workspace_bytes, sq_ctx** out) {
  if (!out) return SQ_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_config(cfg, nullptr);
  if (rc != SQ_OK) return rc;
  if (b_init < 1 || !pool || !workspace) return SQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(pool) % kAlign) || (reinterpret_cast<uintptr_t>(workspace) % kAlign))
    return SQ_ERR_INVALID_ARG;
  if (pool_bytes < pool_bytes_for(*cfg, b_init)) return SQ_ERR_CAPACITY;
  WsLayout wl = ws_layout(*cfg, b_init);
  if (workspace_bytes < wl.total) return SQ_ERR_CAPACITY;
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SQ_ERR_CUDA;
  if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SQ_ERR_CUDA;
  sq_ctx* c = new (std::nothrow) sq_ctx();
  if (!c) return SQ_ERR_CAPACITY;
  c->cfg = *cfg;
  c->b_init_cap = b_init;
  c->pool = static_cast<char*>(pool);
  c->pool_bytes = pool_bytes;
  c->ws = static_cast<char*>(workspace);
  c->ws_bytes = workspace_bytes;
  c->wl = wl;
  c->n_sm = n_sm;
  c->per_seq = cfg->per_sequence_budgets != 0;
  c->begun = false;
  c->budget_state = 0;
  // one pinned block, carved into the staging arrays (largest alignment first)
  const size_t nd = wl.n_desc_cap;
  const size_t bytes = nd * (sizeof(LayerDesc) + sizeof(EvictLayer) + 8 + 4 + 4 + 4 + 4 + 1) + 64;
  void* blk = nullptr;
  if (cudaHostAlloc(&blk, bytes, cudaHostAllocDefault) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev, cudaEventDisableTiming) != cudaSuccess) {
    if (blk) cudaFreeHost(blk);
    delete c;
    return SQ_ERR_CUDA;
  }
  std::memset(blk, 0, bytes);
  char* p = static_cast<char*>(blk);
  c->hs.block = blk;
  c->hs.layers = reinterpret_cast<LayerDesc*>(p);
  p += nd * sizeof(LayerDesc);
  c->hs.evict_tab = reinterpret_cast<EvictLayer*>(p);
  p += nd * sizeof(EvictLayer);
  c->hs.tok_count = reinterpret_cast<long long*>(p);
  p += nd * 8;
  c->hs.budget = reinterpret_cast<int32_t*>(p);
  p += nd * 4;
  c->hs.cos_sim = reinterpret_cast<float*>(p);
  p += nd * 4;
  c->hs.order = reinterpret_cast<int*>(p);
  p += nd * 4;
  c->hs.order_by_layer = reinterpret_cast<int*>(p);
  p += nd * 4;
  c->hs.is_g3 = reinterpret_cast<uint8_t*>(p);
  *out = c;
  return SQ_OK;
}

int sq_ctx_destroy(sq_ctx* c) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaEventDestroy(c->ev);
  cudaFreeHost(c->hs.block);
  delete c;
  return SQ_OK;
}

const char* sq_last_error(sq_ctx* c) { return c ? c->err.c_str() : "context is NULL"; }

int sq_begin_sequence_batch(sq_ctx* c, int32_t batch, int32_t prompt_len, void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (batch < 1 || batch > c->cfg.max_batch) return fail(c, SQ_ERR_INVALID_ARG, "batch out of range");
  if (prompt_len < 1 || prompt_len > c->cfg.max_prompt) return fail(c, SQ_ERR_INVALID_ARG, "prompt_len out of range");
  c->batch = batch;
  c->prompt = prompt_len;
  c->n_grp = c->per_seq ? batch : 1;
  c->desc_units = c->per_seq ? c->cfg.n_kv_head : batch * c->cfg.n_kv_head;
  c->n_desc = c->cfg.n_layer * c->n_grp;
  c->begun = true;
  c->budget_state = 0;
  for (int l = 0; l < c->cfg.n_layer; ++l) {
    c->n_tok[l] = 0;
    c->imp_tokens[l] = 0;
    c->prefilled[l] = false;
    c->importance_seen[l] = false;
  }
  for (int d = 0; d < c->n_desc; ++d) c->hs.tok_count[d] = 0;
  // everything up to the layer table: statistics, ticket, budgets, status
  SQ_CUDA(c, cudaMemsetAsync(c->ws, 0, c->wl.layers, st));
  return SQ_OK;
}

// Shared body of sq_layer_importance (sum_out null) and sq_layer_importance_fused.
static int importance_rows(sq_ctx* c, int32_t layer, const void* row_a, const void* row_b, void* sum_out, int64_t n_tok_total,
                           void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (layer < 0 || layer >= c->cfg.n_layer) return fail(c, SQ_ERR_INVALID_ARG, "layer out of range");
  if (!row_a || !row_b || !aligned16(row_a) || !aligned16(row_b) || !aligned16(sum_out))
    return fail(c, SQ_ERR_INVALID_ARG, "hidden state pointers must be non-NULL and 16-byte aligned");
  if (n_tok_total < 0) return fail(c, SQ_ERR_INVALID_ARG, "n_tok_total is negative");
  if (n_tok_total == 0) return SQ_OK;
  if (c->per_seq && c->imp_tokens[layer] + n_tok_total > (long long)c->batch * c->prompt)
    return fail(c, SQ_ERR_INVALID_ARG, "more tokens than batch * prompt_len for this layer");
  const size_t row = (size_t)c->cfg.hidden * elem_bytes(c->cfg.dtype);
  long long done = 0;
  while (done < n_tok_total) {
    // with per-sequence budgets the rows are taken sequence by sequence, prompt_len rows each:
    // a call is cut at the sequence boundaries it spans
    long long n = n_tok_total - done;
    int grp = 0;
    if (c->per_seq) {
      const long long t = c->imp_tokens[layer] + done;
      grp = (int)(t / c->prompt);
      n = std::min<long long>(n, (long long)(grp + 1) * c->prompt - t);
    }
    const int d = layer * c->n_grp + grp;
    ImportanceArgs a;
    a.a = static_cast<const char*>(row_a) + (size_t)done * row;
    a.b = static_cast<const char*>(row_b) + (size_t)done * row;
    a.sum_out = sum_out ? static_cast<char*>(sum_out) + (size_t)done * row : nullptr;
    a.n_tok = n;
    a.hidden = c->cfg.hidden;
    a.cta_partial = ws_ptr<float>(c, c->wl.cta_partial);
    a.ticket = ws_ptr<unsigned int>(c, c->wl.ticket);
    a.cos_sum = ws_ptr<double>(c, c->wl.cos_sum) + d;
    long long want = (n + 7) / 8;
    int n_cta = (int)std::min<long long>(want, std::min(kMaxImportanceCtas, c->n_sm * 8));
    SQ_CUDA(c, launch_importance(a, c->cfg.dtype, n_cta, static_cast<cudaStream_t>(stream)));
    c->hs.tok_count[d] += n;
    done += n;
  }
  c->imp_tokens[layer] += n_tok_total;
  c->importance_seen[layer] = true;
  return SQ_OK;
}

int sq_layer_importance(sq_ctx* c, int32_t layer, const void* hidden_in, const void* hidden_out, int64_t n_tok_total,
                        void* stream) {
  return importance_rows(c, layer, hidden_in, hidden_out, nullptr, n_tok_total, stream);
}

int sq_layer_importance_fused(sq_ctx* c, int32_t layer, const void* resid, const void* attn_out, void* hidden_out,
                              int64_t n_tok_total, void* stream) {
  if (c && !hidden_out) return fail(c, SQ_ERR_INVALID_ARG, "hidden_out is NULL");
  return importance_rows(c, layer, resid, attn_out, hidden_out, n_tok_total, stream);
}

int sq_allocate_budgets(sq_ctx* c, int64_t b_init, double p, void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (!(p > 0.0 && p <= 1.0)) return fail(c, SQ_ERR_INVALID_ARG, "p must satisfy 0 < p <= 1");
  if (b_init < 1 || b_init > c->b_init_cap) return fail(c, SQ_ERR_INVALID_ARG, "b_init must be in 1..the context's b_init");
  for (int l = 0; l < c->cfg.n_layer; ++l) {
    if (!c->importance_seen[l]) return fail(c, SQ_ERR_STATE, "sq_layer_importance has not been called for every layer");
    if (c->per_seq && c->imp_tokens[l] != (long long)c->batch * c->prompt)
      return fail(c, SQ_ERR_STATE, "per-sequence budgets need the hidden states of every prompt token of every layer");
  }
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<long long>(c, c->wl.tok_count), c->hs.tok_count, 8 * c->n_desc, cudaMemcpyHostToDevice,
                             st));
  AllocateArgs a;
  a.cos_sum = ws_ptr<double>(c, c->wl.cos_sum);
  a.tok_count = ws_ptr<long long>(c, c->wl.tok_count);
  a.n_layer = c->cfg.n_layer;
  a.n_cluster = c->cfg.n_cluster;
  a.stride = c->n_grp;
  a.b_init = b_init;
  a.p = p;
  a.cos_sim = ws_ptr<float>(c, c->wl.cos_sim);
  a.budget = ws_ptr<int>(c, c->wl.budget);
  a.is_g3 = ws_ptr<unsigned char>(c, c->wl.is_g3);
  SQ_CUDA(c, launch_allocate(a, st));
  SQ_CUDA(c, cudaMemcpyAsync(c->hs.budget, a.budget, 4 * c->n_desc, cudaMemcpyDeviceToHost, st));
  SQ_CUDA(c, cudaMemcpyAsync(c->hs.is_g3, a.is_g3, c->n_desc, cudaMemcpyDeviceToHost, st));
  SQ_CUDA(c, cudaMemcpyAsync(c->hs.cos_sim, a.cos_sim, 4 * c->n_desc, cudaMemcpyDeviceToHost, st));
  SQ_CUDA(c, cudaEventRecord(c->ev, st));
  c->budget_state = 1;
  for (int l = 0; l < c->cfg.n_layer; ++l) c->prefilled[l] = false;
  return SQ_OK;
}

int sq_set_budgets(sq_ctx* c, const int32_t* budgets_host, void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (!budgets_host) return fail(c, SQ_ERR_INVALID_ARG, "budgets_host is NULL");
  if (c->budget_state == 1) SQ_CUDA(c, cudaEventSynchronize(c->ev));
  for (int l = 0; l < c->cfg.n_layer; ++l) {
    for (int g = 0; g < c->n_grp; ++g) {
      c->hs.budget[l * c->n_grp + g] = budgets_host[user_index(c, l, g)];
      c->hs.is_g3[l * c->n_grp + g] = 0;
    }
    c->prefilled[l] = false;
  }
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.budget), c->hs.budget, 4 * c->n_desc, cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemsetAsync(ws_ptr<unsigned char>(c, c->wl.is_g3), 0, c->n_desc, st));
  c->budget_state = 0;
  int rc = build_layout(c, st);
  return rc;
}

int sq_prefill_compress(sq_ctx* c, int32_t layer, const void* k_prompt, const void* v_prompt, const void* q_prompt,
                        const float* acc_prompt, void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (layer < 0 || layer >= c->cfg.n_layer) return fail(c, SQ_ERR_INVALID_ARG, "layer out of range");
  if (!k_prompt || !v_prompt || !aligned16(k_prompt) || !aligned16(v_prompt))
    return fail(c, SQ_ERR_INVALID_ARG, "k_prompt/v_prompt must be non-NULL and 16-byte aligned");
  const bool h2o = c->cfg.policy == SQ_POLICY_H2O;
  if (h2o && !q_prompt && !acc_prompt) return fail(c, SQ_ERR_INVALID_ARG, "H2O needs q_prompt or acc_prompt");
  int rc = ensure_budgets(c, st);
  if (rc != SQ_OK) return rc;
  const int P = c->prompt, U = c->desc_units;
  const float* acc = nullptr;
  if (h2o) {
    if (acc_prompt) {
      acc = acc_prompt;
    } else {
      // the scores do not depend on the budgets: one pass for the whole batch
      ScoreArgs s;
      s.q = q_prompt;
      s.k = k_prompt;
      s.lse2 = ws_ptr<float>(c, c->wl.lse2);
      s.acc_prompt = ws_ptr<float>(c, c->wl.acc_prompt);
      s.batch = c->batch;
      s.n_q_head = c->cfg.n_q_head;
      s.n_kv_head = c->cfg.n_kv_head;
      s.prompt = P;
      s.head_dim = c->cfg.head_dim;
      SQ_CUDA(c, launch_prefill_scores(s, c->cfg.dtype, ws_ptr<int>(c, c->wl.status), st));
      acc = s.acc_prompt;
    }
  }
  // selection, gather and first victim: one launch each over all descriptors of the layer
  const LayerDesc* descs_dev = ws_ptr<LayerDesc>(c, c->wl.layers) + layer * c->n_grp;
  const int n_unit = c->batch * c->cfg.n_kv_head;
  int max_keep = 0;
  bool any_full = false;
  for (int g = 0; g < c->n_grp; ++g) {
    const LayerDesc& ld = c->hs.layers[layer * c->n_grp + g];
    max_keep = std::max(max_keep, std::min(P, ld.b));
    any_full |= P >= ld.b;
  }
  if (h2o) SQ_CUDA(c, launch_select_prompt(acc, n_unit, P, descs_dev, U, c->pool, st));
  GatherArgs ga;
  ga.k_prompt = k_prompt;
  ga.v_prompt = v_prompt;
  ga.acc_prompt = acc;
  ga.pool = c->pool;
  ga.descs = descs_dev;
  ga.units_per_desc = U;
  ga.n_unit = n_unit;
  ga.prompt = P;
  ga.max_keep = max_keep;
  ga.policy = c->cfg.policy;
  ga.head_dim = c->cfg.head_dim;
  SQ_CUDA(c, launch_gather(ga, c->cfg.dtype, st));
  if (h2o && any_full) SQ_CUDA(c, launch_pick_victim(c->pool, descs_dev, U, n_unit, P, P, st));
  c->n_tok[layer] = P;
  c->prefilled[layer] = true;
  return SQ_OK;
}

int sq_decode_step(sq_ctx* c, int32_t layer_begin, int32_t layer_end, const void* q, const void* k_new,
                   const void* v_new, void* out, void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (layer_begin < 0 || layer_end > c->cfg.n_layer || layer_begin >= layer_end)
    return fail(c, SQ_ERR_INVALID_ARG, "layer range");
  if (!q || !k_new || !v_new || !out || !aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out))
    return fail(c, SQ_ERR_INVALID_ARG, "q/k_new/v_new/out must be non-NULL and 16-byte aligned");
  int rc = ensure_budgets(c, st);
  if (rc != SQ_OK) return rc;
  const sq_config& cfg = c->cfg;
  for (int l = layer_begin; l < layer_end; ++l) {
    if (!c->prefilled[l]) return fail(c, SQ_ERR_STATE, "sq_prefill_compress has not been called for a layer in the range");
    if (c->n_tok[l] >= cfg.max_prompt + cfg.max_new_tokens) return fail(c, SQ_ERR_CAPACITY, "max_new_tokens exceeded");
  }
  const int U = c->desc_units, G = cfg.n_q_head / cfg.n_kv_head, ng = c->n_grp;
  const size_t eb = elem_bytes(cfg.dtype);
  const size_t q_layer = (size_t)c->batch * cfg.n_q_head * cfg.head_dim * eb;
  const size_t kv_layer = (size_t)c->batch * cfg.n_kv_head * cfg.head_dim * eb;
  int s = layer_begin;
  while (s < layer_end) {
    int e = s + 1;
    while (e < layer_end && c->n_tok[e] == c->n_tok[s]) ++e;
    const int n_tok = c->n_tok[s];
    const int d0 = s * ng, d1 = e * ng;  // descriptors of the launch
    // Split-K plan.  A piece costs a fixed set-up plus its tiles, and pieces run in waves of
    // as many CTAs as fit the GPU at once; among the piece lengths that are whole tiles, take
    // the one with the smallest estimated time.  What a tile, a set-up (in tiles; fitted to
    // measured step times, it includes writing and merging the partial results) and a wave are
    // depends on the kernel the shape is served by.  The running item counts of a split launch
    // travel in the kernel parameters, which hold kMaxLayers descriptors: larger launches (many
    // sequences with per-sequence budgets) are not split; they have units to spare anyway.
    const bool bf16 = cfg.dtype == SQ_BF16;
    int tile, setup, per_sm;
    if (bf16 && cfg.head_dim == 64 && G > 32) {  // tcgen05 kernel: 128-token tiles, 2 CTAs per SM
      tile = 128, setup = 8, per_sm = 2;
    } else if (bf16 && G > 1) {                  // mma.sync kernel: 64-token tiles
      tile = 64, setup = 12, per_sm = cfg.head_dim == 64 && G <= 32 ? 3 : 2;
    } else {                                     // fp32-pipe kernel
      tile = 128, setup = 1, per_sm = G == 1 ? 7 : 2;
    }
    const long long slots = (long long)per_sm * c->n_sm;
    int max_len = 1;
    for (int d = d0; d < d1; ++d) max_len = std::max(max_len, std::min(n_tok + 1, c->hs.layers[d].b));
    int split = 0;
    double best_cost = 0.0;
    int prev = -1;
    for (int pieces = 1; pieces <= (d1 - d0 > kMaxLayers ? 1 : 64); ++pieces) {
      int cand = ((max_len + pieces - 1) / pieces + tile - 1) / tile * tile;
      if (pieces > 1 && cand < 2 * tile) break;  // a piece is never shorter than two tiles
      if (cand == prev) continue;
      prev = cand;
      long long items = 0, work = 0;
      for (int d = d0; d < d1; ++d) {
        const int len = std::min(n_tok + 1, c->hs.layers[d].b);
        const int ns = (len + cand - 1) / cand;
        items += (long long)U * ns;
        work += (long long)U * ((long long)ns * setup + (len + tile - 1) / tile);
      }
      if ((size_t)items > c->wl.items_cap) break;
      // CTAs start in item order, longest layers first: the makespan is about the evenly spread
      // work, but never below the longest piece, and whole waves when there are only a few
      const long long waves = (items + slots - 1) / slots;
      const double t_max = setup + (double)std::min(cand, max_len) / tile;
      const double spread = (double)work / (double)slots + 0.5 * t_max;
      const double cost = items <= slots ? t_max : std::max(t_max, std::min(spread, (double)waves * t_max));
      if (split == 0 || cost < best_cost * 0.90) {  // more pieces only for a clear gain
        best_cost = cost;
        split = cand;
      }
    }
    // the launch's descriptors in launch order: the global order for the whole stack, else layer by layer
    const bool all = (s == 0 && e == cfg.n_layer);
    const int* order_host = all ? c->hs.order : c->hs.order_by_layer + d0;
    DecodeArgs a;
    long long n_items = 0;
    bool any_split = false;
    for (int k = 0; k < d1 - d0; ++k) {
      const int len = std::min(n_tok + 1, c->hs.layers[order_host[k]].b);
      const int ns = (len + split - 1) / split;
      any_split |= ns > 1;
      if (k <= kMaxLayers) a.cum[std::min(k, kMaxLayers)] = (int)n_items;
      n_items += (long long)U * ns;
    }
    if (d1 - d0 <= kMaxLayers) a.cum[d1 - d0] = (int)n_items;
    if ((size_t)n_items > c->wl.items_cap) return fail(c, SQ_ERR_CAPACITY, "workspace too small for the split plan");
    a.layers = ws_ptr<LayerDesc>(c, c->wl.layers);
    a.pool = c->pool;
    a.logits = ws_ptr<float>(c, c->wl.logits);
    a.has_logits = c->wl.logits_floats > 0 ? 1 : 0;
    a.part_stat = ws_ptr<float>(c, c->wl.part_stat);
    a.part_o = ws_ptr<float>(c, c->wl.part_o);
    a.q = static_cast<const char*>(q) + (size_t)(s - layer_begin) * q_layer;
    a.k_new = static_cast<const char*>(k_new) + (size_t)(s - layer_begin) * kv_layer;
    a.v_new = static_cast<const char*>(v_new) + (size_t)(s - layer_begin) * kv_layer;
    a.out = static_cast<char*>(out) + (size_t)(s - layer_begin) * q_layer;
    a.status = ws_ptr<int>(c, c->wl.status);
    a.tickets = ws_ptr<int>(c, c->wl.tickets);
    // without split-K every descriptor has exactly U items and an item is found in O(1)
    a.uniform = any_split ? 0 : 1;
    a.order = all ? ws_ptr<int>(c, c->wl.order) : ws_ptr<int>(c, c->wl.order_by_layer) + d0;
    a.n_layer_total = d1 - d0;
    a.layer_begin = d0;
    a.layer_end = d1;
    a.n_tok = n_tok;
    a.batch = c->per_seq ? 1 : c->batch;
    a.n_q_head = cfg.n_q_head;
    a.n_kv_head = cfg.n_kv_head;
    a.head_dim = cfg.head_dim;
    a.group = G;
    a.n_unit = U;
    a.split_tokens = split;
    a.policy = cfg.policy;
    a.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)cfg.head_dim));
    const bool combine = cfg.policy == SQ_POLICY_H2O;  // other policies merge split-K pieces in the last piece
    // 128-token tiles per unit of every descriptor, in launch order (the wide-group kernel deals
    // the launch's tiles out evenly over the SMs)
    std::vector<int> desc_tiles(d1 - d0);
    for (int k = 0; k < d1 - d0; ++k)
      desc_tiles[k] = (std::min(n_tok + 1, c->hs.layers[order_host[k]].b) + 127) / 128;
    SQ_CUDA(c, launch_decode(a, cfg.dtype, (int)n_items, combine, c->pool_bytes,
                             (size_t)(e - s) * c->batch * cfg.n_q_head, desc_tiles.data(), st));
    for (int l = s; l < e; ++l) c->n_tok[l] += 1;
    s = e;
  }
  return SQ_OK;
}

int sq_evict(sq_ctx* c, int32_t layer_begin, int32_t layer_end, const int32_t* new_budgets_host, void* stream) {
  if (!c) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (layer_begin < 0 || layer_end > c->cfg.n_layer || layer_begin >= layer_end || !new_budgets_host)
    return fail(c, SQ_ERR_INVALID_ARG, "layer range / budgets");
  int rc = ensure_budgets(c, st);
  if (rc != SQ_OK) return rc;
  const sq_config& cfg = c->cfg;
  const int ng = c->n_grp, nl = layer_end - layer_begin;
  // new_budgets_host: [layer_end - layer_begin], or [batch][layer_end - layer_begin] with per-sequence budgets
  auto new_budget = [&](int l, int g) { return new_budgets_host[g * nl + (l - layer_begin)]; };
  for (int l = layer_begin; l < layer_end; ++l) {
    if (!c->prefilled[l]) return fail(c, SQ_ERR_STATE, "sq_prefill_compress has not been called for a layer in the range");
    for (int g = 0; g < ng; ++g) {
      const int nb = new_budget(l, g);
      if (nb < 1 || nb > c->hs.layers[l * ng + g].b) return fail(c, SQ_ERR_INVALID_ARG, "new budget must be in 1..current budget");
      if (cfg.policy == SQ_POLICY_STREAMING_LLM && nb <= cfg.n_sink)
        return fail(c, SQ_ERR_INVALID_ARG, "StreamingLLM needs every layer budget above n_sink");
    }
  }
  int n_active = 0, max_cap = 0;
  for (int l = layer_begin; l < layer_end; ++l) {
    for (int g = 0; g < ng; ++g) {
      const int d = l * ng + g;
      const int nb = new_budget(l, g);
      LayerDesc old = c->hs.layers[d];
      if (nb == old.b) continue;
      LayerDesc nw = old;
      nw.b = nb;
      nw.b_heavy = cfg.policy == SQ_POLICY_H2O ? (int)(((long long)nb * cfg.heavy_num) / cfg.heavy_den) : 0;
      nw.b_recent = nb - nw.b_heavy;
      const int n_tok = c->n_tok[l];
      const int len = std::min(n_tok, old.b);
      if (cfg.policy != SQ_POLICY_H2O) {
        // the compaction keeps slot order, so the ring stays a rotation: find its new phase
        const int base = old.ring_base, r_old = old.b - base, r_new = nb - base;
        if (n_tok <= nb) {
          nw.ring_origin = base;
        } else {
          const int x0 = n_tok - r_new;
          const int r0 = (x0 - old.ring_origin) % r_old;
          const int h = (r0 + r_new <= r_old) ? 0 : r0 + r_new - r_old;
          nw.ring_origin = x0 - h;
        }
      }
      // a cache the new budget makes exactly full has nothing to drop, but under H2O the kernel
      // still has to choose the slot its next append replaces
      if (len > nb || (len == nb && cfg.policy == SQ_POLICY_H2O)) {
        EvictLayer& ev = c->hs.evict_tab[n_active++];
        ev.ld_old = old;
        ev.ld_new = nw;
        ev.len = len;
        ev.n_tok = n_tok;
        max_cap = std::max(max_cap, old.cap);
      }
      c->hs.layers[d] = nw;
      c->hs.budget[d] = nb;
    }
  }
  if (n_active > 0) {
    // all descriptors of the call in one launch, the longest caches first (their CTAs run longest)
    std::stable_sort(c->hs.evict_tab, c->hs.evict_tab + n_active,
                     [](const EvictLayer& x, const EvictLayer& y) { return x.len > y.len; });
    EvictArgs a;
    a.pool = c->pool;
    a.tab = ws_ptr<EvictLayer>(c, c->wl.evict_tab);
    a.n_layers = n_active;
    a.max_cap = max_cap;
    a.n_unit = c->desc_units;
    a.policy = cfg.policy;
    a.n_sink = cfg.n_sink;
    a.row_bytes = cfg.head_dim * elem_bytes(cfg.dtype);
    a.status = ws_ptr<int>(c, c->wl.status);
    SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<EvictLayer>(c, c->wl.evict_tab), c->hs.evict_tab, sizeof(EvictLayer) * n_active,
                               cudaMemcpyHostToDevice, st));
    SQ_CUDA(c, launch_evict(a, st));
  }
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<LayerDesc>(c, c->wl.layers) + layer_begin * ng, &c->hs.layers[layer_begin * ng],
                             sizeof(LayerDesc) * nl * ng, cudaMemcpyHostToDevice, st));
  // the launch orders (largest budget first) may have changed
  sort_orders(c);
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.order), c->hs.order, 4 * c->n_desc, cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.order_by_layer), c->hs.order_by_layer, 4 * c->n_desc,
                             cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.budget), c->hs.budget, 4 * c->n_desc, cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaStreamSynchronize(st));
  return SQ_OK;
}

int sq_get_importance_state(sq_ctx* c, double* cos_sum_host, int64_t* n_tok_host) {
  if (!c || !cos_sum_host || !n_tok_host) return SQ_ERR_INVALID_ARG;
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (c->per_seq) return fail(c, SQ_ERR_UNSUPPORTED, "per-sequence budgets have no state to exchange");
  SQ_CUDA(c, cudaDeviceSynchronize());
  SQ_CUDA(c, cudaMemcpy(cos_sum_host, ws_ptr<double>(c, c->wl.cos_sum), 8 * c->cfg.n_layer, cudaMemcpyDeviceToHost));
  for (int l = 0; l < c->cfg.n_layer; ++l) n_tok_host[l] = c->hs.tok_count[l];
  return SQ_OK;
}

int sq_set_importance_state(sq_ctx* c, const double* cos_sum_host, const int64_t* n_tok_host, void* stream) {
  if (!c || !cos_sum_host || !n_tok_host) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (c->per_seq) return fail(c, SQ_ERR_UNSUPPORTED, "per-sequence budgets have no state to exchange");
  for (int l = 0; l < c->cfg.n_layer; ++l)
    if (n_tok_host[l] < 1) return fail(c, SQ_ERR_INVALID_ARG, "a layer's token count is below 1");
  // pageable source: the copy has left the caller's array when the call returns
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<double>(c, c->wl.cos_sum), cos_sum_host, 8 * c->cfg.n_layer, cudaMemcpyHostToDevice, st));
  for (int l = 0; l < c->cfg.n_layer; ++l) {
    c->hs.tok_count[l] = n_tok_host[l];
    c->importance_seen[l] = true;
  }
  return SQ_OK;
}

int sq_get_cos_sim(sq_ctx* c, float* cos_sim_host) {
  if (!c || !cos_sim_host) return SQ_ERR_INVALID_ARG;
  if (c->budget_state == 0) return fail(c, SQ_ERR_STATE, "sq_allocate_budgets has not been called");
  SQ_CUDA(c, cudaDeviceSynchronize());
  std::vector<float> tmp(c->n_desc);
  SQ_CUDA(c, cudaMemcpy(tmp.data(), ws_ptr<float>(c, c->wl.cos_sim), 4 * c->n_desc, cudaMemcpyDeviceToHost));
  for (int l = 0; l < c->cfg.n_layer; ++l)
    for (int g = 0; g < c->n_grp; ++g) cos_sim_host[user_index(c, l, g)] = tmp[l * c->n_grp + g];
  return SQ_OK;
}

int sq_get_budgets(sq_ctx* c, int32_t* budgets_host, uint8_t* is_g3_host) {
  if (!c || !budgets_host) return SQ_ERR_INVALID_ARG;
  if (c->budget_state == 0) return fail(c, SQ_ERR_STATE, "budgets not set");
  SQ_CUDA(c, cudaDeviceSynchronize());
  std::vector<int32_t> tb(c->n_desc);
  std::vector<uint8_t> tg(c->n_desc);
  SQ_CUDA(c, cudaMemcpy(tb.data(), ws_ptr<int>(c, c->wl.budget), 4 * c->n_desc, cudaMemcpyDeviceToHost));
  SQ_CUDA(c, cudaMemcpy(tg.data(), ws_ptr<unsigned char>(c, c->wl.is_g3), c->n_desc, cudaMemcpyDeviceToHost));
  for (int l = 0; l < c->cfg.n_layer; ++l)
    for (int g = 0; g < c->n_grp; ++g) {
      budgets_host[user_index(c, l, g)] = tb[l * c->n_grp + g];
      if (is_g3_host) is_g3_host[user_index(c, l, g)] = tg[l * c->n_grp + g];
    }
  return SQ_OK;
}

// Where a unit lives: its descriptor and its index within it.
static const LayerDesc& unit_desc(sq_ctx* c, int layer, int seq, int kv_head, size_t* unit) {
  *unit = c->per_seq ? (size_t)kv_head : (size_t)seq * c->cfg.n_kv_head + kv_head;
  return c->hs.layers[layer * c->n_grp + (c->per_seq ? seq : 0)];
}

static int unit_order(sq_ctx* c, int layer, int seq, int kv_head, std::vector<int>& pos, std::vector<int>& order) {
  if (layer < 0 || layer >= c->cfg.n_layer || seq < 0 || seq >= c->batch || kv_head < 0 || kv_head >= c->cfg.n_kv_head)
    return fail(c, SQ_ERR_INVALID_ARG, "layer/seq/kv_head out of range");
  if (c->budget_state != 2 || !c->prefilled[layer]) return fail(c, SQ_ERR_STATE, "layer has no cache yet");
  SQ_CUDA(c, cudaDeviceSynchronize());
  size_t unit;
  const LayerDesc& ld = unit_desc(c, layer, seq, kv_head, &unit);
  const int len = std::min(c->n_tok[layer], ld.b);
  pos.resize(len);
  SQ_CUDA(c, cudaMemcpy(pos.data(), c->pool + ld.pos_off + unit * ld.cap * 4, (size_t)len * 4, cudaMemcpyDeviceToHost));
  order.resize(len);
  for (int i = 0; i < len; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](int x, int y) { return pos[x] < pos[y]; });
  return SQ_OK;
}

int sq_get_kept(sq_ctx* c, int32_t layer, int32_t seq, int32_t kv_head, int32_t* pos_host, float* acc_host, int32_t* n) {
  if (!c || !pos_host || !n) return SQ_ERR_INVALID_ARG;
  std::vector<int> pos, order;
  int rc = unit_order(c, layer, seq, kv_head, pos, order);
  if (rc != SQ_OK) return rc;
  size_t unit;
  const LayerDesc& ld = unit_desc(c, layer, seq, kv_head, &unit);
  const int len = (int)pos.size();
  std::vector<float> acc(len, 0.f);
  if (c->cfg.policy == SQ_POLICY_H2O && len > 0)
    SQ_CUDA(c, cudaMemcpy(acc.data(), c->pool + ld.acc_off + unit * ld.cap * 4, (size_t)len * 4, cudaMemcpyDeviceToHost));
  for (int i = 0; i < len; ++i) {
    pos_host[i] = pos[order[i]];
    if (acc_host) acc_host[i] = acc[order[i]];
  }
  *n = len;
  return SQ_OK;
}

int sq_get_kv(sq_ctx* c, int32_t layer, int32_t seq, int32_t kv_head, void* k_host, void* v_host) {
  if (!c || !k_host || !v_host) return SQ_ERR_INVALID_ARG;
  std::vector<int> pos, order;
  int rc = unit_order(c, layer, seq, kv_head, pos, order);
  if (rc != SQ_OK) return rc;
  size_t unit;
  const LayerDesc& ld = unit_desc(c, layer, seq, kv_head, &unit);
  const int len = (int)pos.size();
  const size_t row = (size_t)c->cfg.head_dim * elem_bytes(c->cfg.dtype);
  std::vector<char> kb(len * row), vb(len * row);
  if (len > 0) {
    SQ_CUDA(c, cudaMemcpy(kb.data(), c->pool + ld.k_off + unit * ld.cap * row, len * row, cudaMemcpyDeviceToHost));
    SQ_CUDA(c, cudaMemcpy(vb.data(), c->pool + ld.v_off + unit * ld.cap * row, len * row, cudaMemcpyDeviceToHost));
  }
  for (int i = 0; i < len; ++i) {
    std::memcpy(static_cast<char*>(k_host) + i * row, kb.data() + order[i] * row, row);
    std::memcpy(static_cast<char*>(v_host) + i * row, vb.data() + order[i] * row, row);
  }
  return SQ_OK;
}

int sq_get_len(sq_ctx* c, int32_t layer, int32_t* len) {
  if (!c || !len) return SQ_ERR_INVALID_ARG;
  if (layer < 0 || layer >= c->cfg.n_layer) return fail(c, SQ_ERR_INVALID_ARG, "layer out of range");
  if (c->budget_state != 2 || !c->prefilled[layer]) return fail(c, SQ_ERR_STATE, "layer has no cache yet");
  int longest = 0;  // with per-sequence budgets: the longest of the layer's sequences
  for (int g = 0; g < c->n_grp; ++g) longest = std::max(longest, std::min(c->n_tok[layer], c->hs.layers[layer * c->n_grp + g].b));
  *len = longest;
  return SQ_OK;
}

int sq_status(sq_ctx* c, int32_t* device_status) {
  if (!c || !device_status) return SQ_ERR_INVALID_ARG;
  SQ_CUDA(c, cudaDeviceSynchronize());
  SQ_CUDA(c, cudaMemcpy(device_status, ws_ptr<int>(c, c->wl.status), 4, cudaMemcpyDeviceToHost));
  return SQ_OK;
}

int sq_ctx_export_layout(sq_ctx* c, sq_layer_layout* out) {
  if (!c || !out) return SQ_ERR_INVALID_ARG;
  if (c->budget_state != 2) return fail(c, SQ_ERR_STATE, "budgets not laid out yet");
  SQ_CUDA(c, cudaDeviceSynchronize());
  for (int l = 0; l < c->cfg.n_layer; ++l)
    for (int g = 0; g < c->n_grp; ++g) {
      const LayerDesc& ld = c->hs.layers[l * c->n_grp + g];
      sq_layer_layout& o = out[user_index(c, l, g)];
      o.k_off = ld.k_off;
      o.v_off = ld.v_off;
      o.pos_off = ld.pos_off;
      o.acc_off = ld.acc_off;
      o.victim_off = ld.victim_off;
      o.budget = ld.b;
      o.cap = ld.cap;
      o.b_heavy = ld.b_heavy;
      o.ring_base = ld.ring_base;
      o.ring_origin = ld.ring_origin;
      o.n_tok = c->prefilled[l] ? c->n_tok[l] : -1;
      o.n_unit = c->desc_units;
      o.reserved = 0;
    }
  return SQ_OK;
}

int sq_ctx_import_layout(sq_ctx* c, const sq_layer_layout* in, void* stream) {
  if (!c || !in) return SQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const sq_config& cfg = c->cfg;
  if (!c->begun) return fail(c, SQ_ERR_STATE, "sq_begin_sequence_batch has not been called");
  if (c->budget_state == 1) SQ_CUDA(c, cudaEventSynchronize(c->ev));
  // The geometry follows the slots a layer was laid out with, not its present budget (an explicit
  // eviction lowers the budget and leaves the slots where they are): lay the pool out by the
  // exported capacities, then put the budgets back.
  for (int l = 0; l < cfg.n_layer; ++l)
    for (int g = 0; g < c->n_grp; ++g) {
      const sq_layer_layout& e = in[user_index(c, l, g)];
      if (e.n_unit != c->desc_units) return fail(c, SQ_ERR_INVALID_ARG, "layout was exported for another batch shape");
      if (e.n_tok != in[user_index(c, l, 0)].n_tok) return fail(c, SQ_ERR_INVALID_ARG, "sequences of a layer disagree on n_tok");
      if (e.n_tok > cfg.max_prompt + cfg.max_new_tokens) return fail(c, SQ_ERR_INVALID_ARG, "n_tok beyond the context's limits");
      if (e.cap < 1 || e.cap % cfg.page_tokens != 0 || e.budget < 1 || e.budget > e.cap)
        return fail(c, SQ_ERR_INVALID_ARG, "layout: budget / cap");
      if (cfg.policy == SQ_POLICY_STREAMING_LLM && e.budget <= cfg.n_sink)
        return fail(c, SQ_ERR_INVALID_ARG, "StreamingLLM needs every layer budget above n_sink");
      c->hs.budget[l * c->n_grp + g] = e.cap;
      c->hs.is_g3[l * c->n_grp + g] = 0;
    }
  c->budget_state = 0;
  int rc = build_layout(c, st);
  if (rc != SQ_OK) return rc;
  c->budget_state = 0;  // until the descriptors below are in place
  for (int l = 0; l < cfg.n_layer; ++l) {
    for (int g = 0; g < c->n_grp; ++g) {
      const sq_layer_layout& e = in[user_index(c, l, g)];
      const int d = l * c->n_grp + g;
      LayerDesc& ld = c->hs.layers[d];
      const int b_heavy = cfg.policy == SQ_POLICY_H2O ? (int)(((long long)e.budget * cfg.heavy_num) / cfg.heavy_den) : 0;
      if (e.k_off != ld.k_off || e.v_off != ld.v_off || e.pos_off != ld.pos_off || e.acc_off != ld.acc_off ||
          e.victim_off != ld.victim_off || e.cap != ld.cap || e.b_heavy != b_heavy || e.ring_base != ld.ring_base)
        return fail(c, SQ_ERR_INVALID_ARG, "layout does not match this context's config or pool");
      if (e.ring_origin < ld.ring_base) return fail(c, SQ_ERR_INVALID_ARG, "layout: ring_origin");
      ld.b = e.budget;
      ld.b_heavy = b_heavy;
      ld.b_recent = e.budget - b_heavy;
      ld.ring_origin = e.ring_origin;  // moved by explicit evictions
      c->hs.budget[d] = e.budget;
    }
    const int n_tok = in[user_index(c, l, 0)].n_tok;
    c->prefilled[l] = n_tok >= 0;
    c->n_tok[l] = n_tok >= 0 ? n_tok : 0;
  }
  sort_orders(c);
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<LayerDesc>(c, c->wl.layers), c->hs.layers, sizeof(LayerDesc) * c->n_desc,
                             cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.order), c->hs.order, 4 * c->n_desc, cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.order_by_layer), c->hs.order_by_layer, 4 * c->n_desc,
                             cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemcpyAsync(ws_ptr<int>(c, c->wl.budget), c->hs.budget, 4 * c->n_desc, cudaMemcpyHostToDevice, st));
  SQ_CUDA(c, cudaMemsetAsync(ws_ptr<unsigned char>(c, c->wl.is_g3), 0, c->n_desc, st));
  SQ_CUDA(c, cudaStreamSynchronize(st));
  c->budget_state = 2;
  return SQ_OK;
}

int sq_kv_bytes_per_step(sq_ctx* c, int32_t layer_begin, int32_t layer_end, int64_t* bytes) {
  if (!c || !bytes) return SQ_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end > c->cfg.n_layer || layer_begin >= layer_end)
    return fail(c, SQ_ERR_INVALID_ARG, "layer range");
  if (c->budget_state != 2) return fail(c, SQ_ERR_STATE, "budgets not on the host yet");
  const int64_t U = c->desc_units;
  const int64_t row = (int64_t)c->cfg.head_dim * elem_bytes(c->cfg.dtype);
  int64_t total = 0;
  for (int l = layer_begin; l < layer_end; ++l)
    for (int g = 0; g < c->n_grp; ++g)
      total += U * std::min(c->n_tok[l] + 1, c->hs.layers[l * c->n_grp + g].b) * 2 * row;
  *bytes = total;
  return SQ_OK;
}

}  // extern "C"
