/*
 * sq.h -- C ABI of libsq: SqueezeAttention's data-parallel hot path on one GPU (sm_100a).
 *
 * The library follows Algorithm 1 of "SqueezeAttention: 2D Management of KV-Cache in LLM
 * Inference via Layer-wise Optimal Budget" (arXiv 2404.04793):
 *
 *   prefill : per layer, cosine similarity of every prompt token's hidden state before and
 *             after self-attention, averaged over the prompt        -> sq_layer_importance
 *             KMeans of the layer averages, budget of the least important group scaled by p,
 *             freed slots handed to the other layers                -> sq_allocate_budgets
 *             the prompt's K/V enters the cache under each layer's own budget
 *                                                                   -> sq_prefill_compress
 *   decode  : per generated token and layer: append K/V, compress with the sequence-wise
 *             policy C_seq if the layer is over its budget, self-attention over what is
 *             left                                                  -> sq_decode_step
 *   C_seq on its own, to a tighter budget, in place                 -> sq_evict
 *
 * Conventions
 *   - Every call returns an sq_status_t (SQ_OK == 0).  Nothing throws, aborts or traps;
 *     sq_last_error() returns a message for the last failing call on that context.
 *   - All tensor arguments are CALLER-OWNED DEVICE pointers, dense row-major, 16-byte
 *     aligned, of the context's dtype unless stated.  "host" pointers are marked.
 *   - The library allocates no device memory.  The caller provides one cache pool and one
 *     workspace (sizes from sq_query_sizes); both must stay valid until sq_ctx_destroy and
 *     must not be touched by the caller in between.  sq_ctx_create allocates one small block of
 *     page-locked HOST memory (staging of the budget and layout tables, a few KB per layer) and
 *     one CUDA event; sq_ctx_destroy frees them.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued on it and calls return without waiting, except the sq_get_* calls and
 *     sq_status, which synchronise the device, and the first call after sq_allocate_budgets
 *     that needs the budgets on the host (sq_prefill_compress / sq_decode_step / sq_evict),
 *     which waits for that one small kernel.
 *     All calls of one context must use the same stream or be ordered by the caller.
 *   - A sequence batch has `batch` sequences of the same prompt length.  A *unit* is one
 *     (sequence, KV head) pair of a layer; unit index = seq * n_kv_head + kv_head.
 *   - Scores must be finite (no NaN).
 *   - There is no CPU fallback: a missing device or a failed launch is an error.
 */
#ifndef SQ_H_
#define SQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sq_ctx sq_ctx;

typedef enum {
  SQ_OK = 0,
  SQ_ERR_INVALID_ARG = 1, /* bad pointer, size, range or alignment                         */
  SQ_ERR_STATE = 2,       /* call order violated (e.g. decode before prefill)              */
  SQ_ERR_CAPACITY = 3,    /* pool or workspace too small for the requested budgets         */
  SQ_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed                          */
  SQ_ERR_UNSUPPORTED = 5  /* shape outside what the kernels are built for                  */
} sq_status_t;

/* Sequence-wise compressor C_seq (Sections 2.2 and 5.1). */
typedef enum {
  SQ_POLICY_SLIDING_WINDOW = 0, /* keep the most recent tokens                              */
  SQ_POLICY_STREAMING_LLM = 1,  /* first n_sink tokens + the most recent                    */
  SQ_POLICY_H2O = 2             /* heavy hitters by accumulated attention + the most recent */
} sq_policy;

typedef enum { SQ_F32 = 0, SQ_BF16 = 1 } sq_dtype;

typedef struct sq_config {
  int32_t n_layer;        /* 1..256                                                         */
  int32_t n_q_head;       /* multiple of n_kv_head; n_q_head / n_kv_head <= 128             */
  int32_t n_kv_head;
  int32_t head_dim;       /* 64 or 128                                                      */
  int32_t hidden;         /* d_model of the hidden states; multiple of 8                    */
  int32_t max_batch;
  int32_t max_prompt;
  int32_t max_new_tokens;
  int32_t dtype;          /* sq_dtype of hidden states, Q, K, V and outputs                 */
  int32_t policy;         /* sq_policy                                                      */
  int32_t n_sink;         /* StreamingLLM sinks; the paper uses 4 (Section 5.1)             */
  int32_t heavy_num;      /* H2O: floor(b * heavy_num / heavy_den) slots of a layer's       */
  int32_t heavy_den;      /*      budget b go to heavy hitters, the rest to recent tokens   */
  int32_t n_cluster;      /* 3 (Algorithm 1, step 5) or 2                                   */
  int32_t page_tokens;    /* per-unit slot ranges are rounded up to this many tokens (>= 1) */
  int32_t per_sequence_budgets; /* 0: one budget vector for the batch, from the cosine averaged over
                                      all its prompts (the default);  1: one budget vector per
                                      prompt (Section 4.1 allocates "for the given prompt"): every
                                      sequence is clustered on its own averages and gets its own
                                      per-layer budgets, each summing to n_layer * b_init.  Then the
                                      per-layer arrays of sq_set_budgets, sq_get_cos_sim,
                                      sq_get_budgets and sq_evict are [batch][n_layer] (sequence
                                      first), sq_layer_importance takes the rows sequence by
                                      sequence (prompt_len rows each, all of them before
                                      sq_allocate_budgets) */
} sq_config;

/* Bytes of cache pool and workspace a context needs when the per-layer budgets sum to at most
 * n_layer * b_init (which sq_allocate_budgets guarantees).  Host-only, no CUDA call. */
int sq_query_sizes(const sq_config* cfg, int64_t b_init, size_t* pool_bytes, size_t* workspace_bytes);

/* Creates a context on the current device over caller-provided device memory (256-byte
 * aligned).  The context remembers b_init as the capacity it was sized for. */
int sq_ctx_create(const sq_config* cfg, int64_t b_init, void* pool, size_t pool_bytes, void* workspace,
                  size_t workspace_bytes, sq_ctx** out);
int sq_ctx_destroy(sq_ctx* ctx);

/* Starts a new batch of `batch` prompts of `prompt_len` tokens: clears the layer statistics,
 * budgets and cache state. */
int sq_begin_sequence_batch(sq_ctx* ctx, int32_t batch, int32_t prompt_len, void* stream);

/* Section 3 (cosine-similarity equation) and Algorithm 1, steps 1-4.
 * hidden_in / hidden_out: [n_tok_total, hidden], the hidden state of each prompt token before
 * and after this layer's self-attention block (any flattening of [batch, tokens]).  Adds the
 * sum of the per-token cosine similarities to the layer's statistic; may be called several
 * times per layer (chunks of the prompt).  A token with a zero-norm vector contributes 0. */
int sq_layer_importance(sq_ctx* ctx, int32_t layer, const void* hidden_in, const void* hidden_out,
                        int64_t n_tok_total, void* stream);

/* The same statistic taken where the hidden state after self-attention is made (Section 4.1:
 * the similarities are collected "whenever the self-attention is conducted"; Table 4 prices the
 * separate pass at +6.3 % of prefill).  resid: the residual stream entering the layer's
 * attention block = the hidden state before self-attention; attn_out: the attention block's
 * output; both [n_tok_total, hidden].  Writes hidden_out = resid + attn_out (one fp32 addition
 * per element, rounded to the context's dtype) and adds the cosine between resid and that stored
 * sum, token by token, to the layer's statistic: per token it reads 2 rows and writes 1, where a
 * producer's own addition followed by sq_layer_importance reads 4 and writes 1.  hidden_out may
 * be resid or attn_out itself (every element is read before it is written).  Chunking, call order
 * and errors as for sq_layer_importance; the two calls may be mixed between layers. */
int sq_layer_importance_fused(sq_ctx* ctx, int32_t layer, const void* resid, const void* attn_out, void* hidden_out,
                              int64_t n_tok_total, void* stream);

/* Algorithm 1, steps 5-12, and Appendix A.2.  Averages each layer's statistic, clusters the
 * n_layer averages (exact one-dimensional k-means with n_cluster groups; the group with the
 * largest average is the least important, G3), sets G3's budget to max(1, floor(b_init * p))
 * and splits the rest of n_layer * b_init evenly over the other layers, remainder to the
 * lowest-indexed ones, so the budgets sum to n_layer * b_init exactly.  0 < p <= 1;
 * 1 <= b_init <= the b_init of sq_ctx_create.  Runs on the device. */
int sq_allocate_budgets(sq_ctx* ctx, int64_t b_init, double p, void* stream);

/* Sets the per-layer budgets directly (host array [n_layer]; [batch][n_layer] with
 * per_sequence_budgets), bypassing importance and clustering.  SQ_ERR_CAPACITY if they do not
 * fit the pool. */
int sq_set_budgets(sq_ctx* ctx, const int32_t* budgets_host, void* stream);

/* Algorithm 1, step 13, with the first compression (steps 16-18) applied at once: caches the
 * prompt's K/V of one layer, keeping min(prompt_len, budget[layer]) tokens per unit as C_seq
 * selects them.
 *   k_prompt, v_prompt : [batch, n_kv_head, prompt_len, head_dim]
 *   q_prompt           : [batch, n_q_head, prompt_len, head_dim]; H2O only (else NULL): the
 *                        prompt's accumulated attention is the column sums of the causal
 *                        softmax(Q K^T / sqrt(head_dim)), summed over the query heads that
 *                        share the KV head
 *   acc_prompt         : optional fp32 [batch, n_kv_head, prompt_len]; H2O only: use these
 *                        scores instead of computing them from q_prompt
 * Equal scores keep the lower position. */
int sq_prefill_compress(sq_ctx* ctx, int32_t layer, const void* k_prompt, const void* v_prompt,
                        const void* q_prompt, const float* acc_prompt, void* stream);

/* Algorithm 1, steps 15-22, for layers [layer_begin, layer_end) and one new token per
 * sequence: append k_new/v_new at the next position; if the layer is then over its budget,
 * C_seq drops one token (its slot is reused); every query head attends over the kept tokens
 * (softmax(q K^T / sqrt(head_dim)) V); for H2O each kept token's score grows by the
 * probability it received, summed over the query heads sharing its KV head.
 *   q            : [layer_end-layer_begin, batch, n_q_head, head_dim]
 *   k_new, v_new : [layer_end-layer_begin, batch, n_kv_head, head_dim]
 *   out          : same shape and dtype as q */
int sq_decode_step(sq_ctx* ctx, int32_t layer_begin, int32_t layer_end, const void* q, const void* k_new,
                   const void* v_new, void* out, void* stream);

/* C_seq(K, b) on its own (Section 4.1): lowers the budgets of layers [layer_begin, layer_end)
 * to new_budgets_host[i] (host array [layer_end-layer_begin], or [batch][layer_end-layer_begin]
 * with per_sequence_budgets; each <= the current budget, >= 1) and compresses their caches in
 * place to at most that many tokens.  One kernel launch serves all layers of the call. */
int sq_evict(sq_ctx* ctx, int32_t layer_begin, int32_t layer_end, const int32_t* new_budgets_host,
             void* stream);

/* One batch sharded over several GPUs (each rank holds some of its sequences and their whole
 * cache): with one budget vector for the batch, the layer averages of Section 3's cosine run over
 * the tokens of all ranks, so the ranks exchange, once, after the last sq_layer_importance and
 * before sq_allocate_budgets, the per-layer sums of cosines and token counts (2 * n_layer numbers;
 * summed over the ranks by the caller, e.g. one all-reduce) and every rank then runs the same
 * deterministic allocation.  sq_get_importance_state reads this context's sums (synchronises);
 * sq_set_importance_state replaces them (host arrays [n_layer]; asynchronous on `stream`).  Not
 * available with per_sequence_budgets (nothing to exchange there): SQ_ERR_UNSUPPORTED. */
int sq_get_importance_state(sq_ctx* ctx, double* cos_sum_host /* [n_layer] */, int64_t* n_tok_host /* [n_layer] */);
int sq_set_importance_state(sq_ctx* ctx, const double* cos_sum_host, const int64_t* n_tok_host, void* stream);

/* Read-back (host outputs; these synchronise). */
int sq_get_cos_sim(sq_ctx* ctx, float* cos_sim_host /* [n_layer]; [batch][n_layer] with per_sequence_budgets */);
int sq_get_budgets(sq_ctx* ctx, int32_t* budgets_host /* same shape */, uint8_t* is_g3_host /* same shape, or NULL */);
/* Kept tokens of one unit, sorted by position: positions and (H2O; else zeros) scores.
 * Arrays must hold the unit's budget (sq_get_len(layer) entries always suffice); *n receives
 * the count. */
int sq_get_kept(sq_ctx* ctx, int32_t layer, int32_t seq, int32_t kv_head, int32_t* pos_host, float* acc_host,
                int32_t* n);
/* Cached K and V rows of one unit in the same (position) order as sq_get_kept, as raw
 * elements of the context's dtype: [n, head_dim] each (host buffers). */
int sq_get_kv(sq_ctx* ctx, int32_t layer, int32_t seq, int32_t kv_head, void* k_host, void* v_host);
/* Number of cached tokens per unit of a layer (with per_sequence_budgets: of its longest unit). */
int sq_get_len(sq_ctx* ctx, int32_t layer, int32_t* len);
/* Device-side status word: 0 = clean; non-zero = a kernel detected an inconsistency. */
int sq_status(sq_ctx* ctx, int32_t* device_status);
const char* sq_last_error(sq_ctx* ctx);

/* Checkpoint / resume.  The cache state of a batch is the caller's pool plus this table: one
 * entry per layer (per (sequence, layer), sequence first, with per_sequence_budgets).  Offsets
 * are bytes from the pool base; a unit's slots are rows [unit * cap, unit * cap + min(n_tok,
 * budget)) of each region (K, V rows of head_dim elements; pos int32; acc fp32, H2O only; victim
 * int32 per unit, H2O only).  To resume: copy the pool's bytes back (or keep the pool), create a
 * context with the same config and b_init, sq_begin_sequence_batch with the same batch and
 * prompt_len, then sq_ctx_import_layout with the exported table; decoding continues with the
 * next token as if it had not stopped.  Export synchronises the device; import is host work plus
 * small asynchronous copies on `stream` and one wait for them.  Import lays the pool out by the
 * table's capacities and returns SQ_ERR_INVALID_ARG, changing nothing the caller can decode
 * from, when the table's offsets are not the ones this context gives those capacities. */
typedef struct sq_layer_layout {
  int64_t k_off, v_off, pos_off, acc_off, victim_off;
  int32_t budget;      /* tokens kept per unit                                              */
  int32_t cap;         /* slots per unit: the budget the layer was laid out with, rounded
                          up to page_tokens (an explicit eviction lowers budget, not cap)   */
  int32_t b_heavy;     /* H2O: slots of the budget held for heavy hitters                   */
  int32_t ring_base;   /* Sliding Window 0, StreamingLLM n_sink: slots below it never move  */
  int32_t ring_origin; /* the position stored in slot ring_base                             */
  int32_t n_tok;       /* tokens seen so far (prompt + generated); -1: layer not prefilled  */
  int32_t n_unit;      /* units that share this entry                                       */
  int32_t reserved;
} sq_layer_layout;
int sq_ctx_export_layout(sq_ctx* ctx, sq_layer_layout* layout_host /* [n_layer]; [batch][n_layer] with per_sequence_budgets */);
int sq_ctx_import_layout(sq_ctx* ctx, const sq_layer_layout* layout_host, void* stream);

/* Bytes of K+V the decode kernel reads per step for the given layer range at the current
 * fill level (for bandwidth accounting). */
int sq_kv_bytes_per_step(sq_ctx* ctx, int32_t layer_begin, int32_t layer_end, int64_t* bytes);

/* H2O prompt scores for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the scoring step inside
 * sq_prefill_compress.)  Some hosts of this library run where cudaMalloc is off limits:
 * inside a memory pool that was sized and handed out up front, in a plugin whose embedding
 * runtime owns every allocation, or in a service that forbids allocation after start-up so
 * that a request can never fail for lack of memory.  sq_prefill_compress needs a workspace
 * from the caller for the per-row log-sum-exp of the causal score matrix; this call keeps
 * that intermediate in a fixed array that is part of the library image instead, so the
 * caller passes only inputs and the output:
 *   q_prompt [batch, n_q_head, prompt_len, head_dim], k_prompt [batch, n_kv_head, prompt_len,
 *   head_dim] (dtype sq_dtype), acc_out fp32 [batch, n_kv_head, prompt_len]; all device
 *   pointers, 16-byte aligned.  acc_out[b, h, t] = sum over the query heads sharing KV head h
 *   and over rows r >= t of softmax_row_r(Q K^T / sqrt(head_dim))[t], the quantity
 *   sq_prefill_compress computes from q_prompt (bf16 inputs take the fp32-pipe kernels here, so the
 *   two agree to rounding, not bit for bit).
 * Limits and rules:
 *   - batch * n_q_head * prompt_len <= SQ_STATIC_SCORE_MAX_ROWS (the array holds one float
 *     per query row: 4 MiB, resident on every GPU that loads the library until the process
 *     exits); larger requests return SQ_ERR_CAPACITY and launch nothing.
 *   - The first call on each device looks up the array's device address (no allocation);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (every
 *     entry a call reads was written by that call first), but two calls that overlap on the
 *     GPU (different streams, or different host threads without ordering) race on it: order
 *     them on one stream or with events.
 *   - Calls no cudaMalloc/cudaFree and no allocating library routine; needs no sq_ctx. */
#define SQ_STATIC_SCORE_MAX_ROWS (1 << 20)
int sq_prompt_scores_static(const void* q_prompt, const void* k_prompt, int32_t batch, int32_t n_q_head,
                            int32_t n_kv_head, int32_t prompt_len, int32_t head_dim, int32_t dtype, float* acc_out,
                            void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SQ_H_ */
