"""CPU oracle for SqueezeAttention (arXiv 2404.04793) -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the paper's method computes, one
function per step of Algorithm 1.  It exists to check the CUDA library and is
never part of the product path: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  It imports nothing from the CUDA
package and shares no code, tables or helpers with it.

Every function takes numpy arrays (any float dtype; converted exactly to
float64) and works on the smallest independent unit of the method, so a reader
can follow it against the paper by eye:

  layer_importance     Section 3 cosine-similarity equation, Algorithm 1 steps 1-4
  cluster_layers       Algorithm 1 step 5 (KMeans into groups, G3 = largest mean)
  allocate_budgets     Algorithm 1 steps 6-12, Appendix A.2 worked example
  c_seq                the sequence-wise compressor C_seq(K, b), Sections 2.2 / 5.1
  prefill_scores       accumulated attention of the prompt (H2O ranking signal)
  UnitCache            Algorithm 1 steps 13-22 for one (sequence, layer, KV head)

Parity pins: every function here is pinned by tests/test_oracle_pins.py
(closed forms, the paper's worked example, library routines, brute force).
Nothing in this file is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

SLIDING_WINDOW = 0
STREAMING_LLM = 1
H2O = 2


def _f64(x):
    return np.asarray(x, dtype=np.float64)


# --------------------------------------------------------------------------
# Section 3, cosine-similarity equation; Algorithm 1 steps 1-4
# --------------------------------------------------------------------------
def token_cosine(a, b):
    """cos(A, B) = (sum_i A_i B_i) / (sqrt(sum_i A_i^2) * sqrt(sum_i B_i^2)) for
    one token's hidden state before (A) and after (B) self-attention.
    The equation has no epsilon; a token whose product of norms is zero
    contributes 0 (reading: the quotient is undefined there)."""
    a = _f64(a)
    b = _f64(b)
    dot = float(np.sum(a * b))
    na = math.sqrt(float(np.sum(a * a)))
    nb = math.sqrt(float(np.sum(b * b)))
    if na * nb == 0.0:
        return 0.0
    return dot / (na * nb)


def layer_importance(hidden_in, hidden_out):
    """cos_sim^(i): the mean over all prompt tokens (all sequences of the
    batch) of the per-token cosine similarity.  hidden_* are [n_tokens, d_model]
    (leading dims are flattened)."""
    a = _f64(hidden_in)
    b = _f64(hidden_out)
    a = a.reshape(-1, a.shape[-1])
    b = b.reshape(-1, b.shape[-1])
    total = 0.0
    for j in range(a.shape[0]):
        total += token_cosine(a[j], b[j])
    return total / a.shape[0]


# --------------------------------------------------------------------------
# Algorithm 1 step 5: KMeans of n_layer scalars into groups
# --------------------------------------------------------------------------
def _run_cost(x):
    """Within-run sum of squared deviations, evaluated in index order:
    mean = (x_0 + x_1 + ...)/n, cost = (x_0-mean)^2 + (x_1-mean)^2 + ..."""
    s = 0.0
    for v in x:
        s = s + v
    mean = s / len(x)
    c = 0.0
    for v in x:
        dlt = v - mean
        c = c + dlt * dlt
    return c


def cluster_layers(cos_sim, n_cluster=3):
    """The exact optimum of 1-D k-means (the paper leaves KMeans' seed and
    iteration count open; the global optimum is the deterministic fixed point
    every run of it approximates).  In one dimension the optimal clusters are
    contiguous runs of the sorted values, so the optimum is found by trying
    every way to cut the sorted list into k non-empty runs.

    Details fixed by this reading: values are sorted ascending with ties in
    layer order; k is lowered to the number of distinct values if there are
    fewer; candidate cuts are visited in lexicographic order and a candidate
    replaces the incumbent only if its cost is strictly smaller; the cost of a
    candidate is cost(run_1) + cost(run_2) (+ cost(run_3)) added in that order.

    Returns is_g3[n_layer] (bool): membership of the group with the largest
    values -- the paper's G3, the least important layers.  With a single
    distinct value there is no G3."""
    c = [float(v) for v in np.asarray(cos_sim, dtype=np.float64)]
    n = len(c)
    order = sorted(range(n), key=lambda i: (c[i], i))
    x = [c[i] for i in order]
    k = min(n_cluster, len(set(x)))
    is_g3 = np.zeros(n, dtype=bool)
    if k <= 1:
        return is_g3
    best_cost = None
    best_last_cut = None
    if k == 2:
        for i in range(1, n):
            cost = _run_cost(x[:i]) + _run_cost(x[i:])
            if best_cost is None or cost < best_cost:
                best_cost, best_last_cut = cost, i
    elif k == 3:
        for i in range(1, n - 1):
            for j in range(i + 1, n):
                cost = _run_cost(x[:i]) + _run_cost(x[i:j]) + _run_cost(x[j:])
                if best_cost is None or cost < best_cost:
                    best_cost, best_last_cut = cost, j
    else:
        raise ValueError("n_cluster must be 2 or 3")
    for r in range(best_last_cut, n):
        is_g3[order[r]] = True
    return is_g3


# --------------------------------------------------------------------------
# Algorithm 1 steps 6-12; Appendix A.2
# --------------------------------------------------------------------------
def allocate_budgets(cos_sim, b_init, p, n_cluster=3):
    """b^(i) = b_init * p for i in G3; the other layers share
    n_layer*b_init - |G3|*b_init*p equally.

    Token budgets are integers and the paper states the total is unchanged, so:
    b_low = max(1, floor(b_init * p)) (one fp64 product); the remainder
    R = n_layer*b_init - |G3|*b_low is split over the m other layers as
    floor(R/m), with the R mod m lowest-indexed of them getting one more.
    G3 empty or G3 = all layers: nothing to move, every layer keeps b_init.

    Returns (budgets int64[n_layer], is_g3 bool[n_layer])."""
    is_g3 = cluster_layers(cos_sim, n_cluster)
    n = len(is_g3)
    n3 = int(is_g3.sum())
    budgets = np.full(n, int(b_init), dtype=np.int64)
    if n3 == 0 or n3 == n:
        return budgets, np.zeros(n, dtype=bool)
    b_low = max(1, int(math.floor(float(b_init) * float(p))))
    rest = n * int(b_init) - n3 * b_low
    m = n - n3
    base, extra = divmod(rest, m)
    seen = 0
    for i in range(n):
        if is_g3[i]:
            budgets[i] = b_low
        else:
            budgets[i] = base + (1 if seen < extra else 0)
            seen += 1
    return budgets, is_g3


# --------------------------------------------------------------------------
# C_seq(K, b): Sections 2.2 and 5.1 (Sliding Window, StreamingLLM, H2O)
# --------------------------------------------------------------------------
def c_seq(policy, pos, acc, b, n_sink=4, heavy_num=1, heavy_den=2):
    """Indices (into pos/acc) of the tokens C_seq keeps, ordered by position.

    pos: distinct integer token positions held by the cache; acc: accumulated
    attention score per token (H2O only).  len(pos) <= b: nothing is dropped
    (Algorithm 1 compresses only when len(K) > b).  Otherwise exactly b stay:
      Sliding Window : the b most recent positions.
      StreamingLLM   : the first min(n_sink, b) positions plus the most recent.
      H2O            : b_r = b - floor(b*heavy_num/heavy_den) most recent, and of
                       the rest the floor(b*heavy_num/heavy_den) with the largest
                       accumulated score; equal scores keep the lower position.
    """
    pos = [int(v) for v in pos]
    n = len(pos)
    by_pos = sorted(range(n), key=lambda i: pos[i])
    if n <= b:
        return by_pos
    if policy == SLIDING_WINDOW:
        keep = by_pos[n - b:]
    elif policy == STREAMING_LLM:
        s = min(n_sink, b)
        keep = by_pos[:s] + by_pos[n - (b - s):] if b - s > 0 else by_pos[:s]
    elif policy == H2O:
        b_h = (b * heavy_num) // heavy_den
        b_r = b - b_h
        recent = by_pos[n - b_r:] if b_r > 0 else []
        others = by_pos[:n - b_r]
        a = [float(v) for v in np.asarray(acc, dtype=np.float64)]
        ranked = sorted(others, key=lambda i: (-a[i], pos[i]))
        keep = ranked[:b_h] + recent
    else:
        raise ValueError("unknown policy")
    return sorted(keep, key=lambda i: pos[i])


# --------------------------------------------------------------------------
# Self-attention (Section 2.1; textbook scaled dot-product, scale 1/sqrt(d))
# --------------------------------------------------------------------------
def _softmax(s):
    m = np.max(s)
    e = np.exp(s - m)
    return e / np.sum(e)


def prefill_scores(q_prompt, k_prompt):
    """Accumulated attention each prompt token receives during prefill:
    acc[t] = sum over the query heads sharing this KV head, and over query rows
    r >= t, of softmax_row_r(Q K^T / sqrt(d))[t]  (causal mask).
    q_prompt [g, P, d], k_prompt [P, d]  ->  acc [P]."""
    q = _f64(q_prompt)
    k = _f64(k_prompt)
    g, P, d = q.shape
    acc = np.zeros(P, dtype=np.float64)
    for h in range(g):
        s = (q[h] @ k.T) / math.sqrt(d)
        for r in range(P):
            acc[: r + 1] += _softmax(s[r, : r + 1])
    return acc


class UnitCache:
    """The KV cache of one (sequence, layer, KV head) through Algorithm 1's
    steps 13-22: the prompt's K/V is cached, then per generated token the new
    K/V is appended, the cache is compressed by C_seq if it exceeds this layer's
    budget b, and the g query heads sharing the KV head attend over what is
    left.  For H2O every kept token's score then grows by the attention
    probability it just received (summed over the g heads)."""

    def __init__(self, policy, b, n_sink=4, heavy_num=1, heavy_den=2):
        self.policy = policy
        self.b = int(b)
        self.n_sink = n_sink
        self.heavy_num = heavy_num
        self.heavy_den = heavy_den
        self.pos = []          # token positions, ascending
        self.acc = []          # accumulated scores (fp64)
        self.K = []            # rows, fp64
        self.V = []
        self.next_pos = 0

    def _compress(self):
        if len(self.pos) > self.b:
            keep = c_seq(self.policy, self.pos, self.acc, self.b, self.n_sink,
                         self.heavy_num, self.heavy_den)
            self.pos = [self.pos[i] for i in keep]
            self.acc = [self.acc[i] for i in keep]
            self.K = [self.K[i] for i in keep]
            self.V = [self.V[i] for i in keep]

    def prefill(self, k_prompt, v_prompt, q_prompt=None, acc_prompt=None, compress=True):
        """Cache the prompt's K/V ([P, d] each).  For H2O the prompt's scores
        come from q_prompt [g, P, d] (or are given as acc_prompt [P]).
        compress=True applies C_seq right away; Algorithm 1 defers it to the
        first decode step, which keeps the same set (see the pin test)."""
        k = _f64(k_prompt)
        v = _f64(v_prompt)
        P = k.shape[0]
        if acc_prompt is not None:
            acc = [float(x) for x in np.asarray(acc_prompt, dtype=np.float64)]
        elif self.policy == H2O and q_prompt is not None:
            acc = [float(x) for x in prefill_scores(q_prompt, k)]
        else:
            acc = [0.0] * P
        self.pos = list(range(P))
        self.acc = acc
        self.K = [k[t] for t in range(P)]
        self.V = [v[t] for t in range(P)]
        self.next_pos = P
        if compress:
            self._compress()

    def decode_step(self, q, k_new, v_new):
        """q [g, d], k_new [d], v_new [d] -> out [g, d].
        Order within the step (Algorithm 1): append, compress if over budget,
        attend, then (H2O) accumulate the probabilities."""
        q = _f64(q)
        g, d = q.shape
        self.pos.append(self.next_pos)
        self.acc.append(0.0)
        self.K.append(_f64(k_new))
        self.V.append(_f64(v_new))
        self.next_pos += 1
        self._compress()
        K = np.stack(self.K)
        V = np.stack(self.V)
        out = np.zeros((g, d), dtype=np.float64)
        gain = np.zeros(len(self.pos), dtype=np.float64)
        for h in range(g):
            prob = _softmax((K @ q[h]) / math.sqrt(d))
            out[h] = prob @ V
            gain += prob
        if self.policy == H2O:
            self.acc = [a + float(x) for a, x in zip(self.acc, gain)]
        return out

    def kept_positions(self):
        return list(self.pos)


def kv_bytes_per_token(n_layer, d_model, elem_bytes):
    """Section 2.1: the cache holds 2 * d_model * n_layer values per token."""
    return 2 * d_model * n_layer * elem_bytes
