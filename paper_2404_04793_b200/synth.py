"""Seeded synthetic workloads shaped like the models the paper evaluates.

This module only *draws inputs*: hidden states, prompt Q/K/V and decode-time
q/k/v tensors with the shapes, dtypes and structure of the paper's workloads
(layer/head counts of Llama-2-7B/70B, Mistral-7B, Falcon-7B; a few key positions
that attract most of the attention; per-layer hidden-state drift that gives the
"few special layers / important first half / unimportant rest" pattern of
Sections 3 and 4.2.2).  It contains none of the method's arithmetic and is used
to feed the same bits to the CUDA library and to the CPU oracle.

All draws come from torch.Generator objects seeded from (workload id, tensor
family, layer, step), on whichever device is asked for, in fp32, and are then
rounded to the workload's dtype.
"""
from __future__ import annotations

import dataclasses
import math

import torch

SLIDING_WINDOW = 0
STREAMING_LLM = 1
H2O = 2
POLICY_NAMES = {SLIDING_WINDOW: "sliding_window", STREAMING_LLM: "streaming_llm", H2O: "h2o"}

_BASE_SEED = 20240404


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    wid: int                 # enters every seed
    n_layer: int
    n_q_head: int
    n_kv_head: int
    head_dim: int
    hidden: int
    batch: int
    prompt: int
    steps: int               # decode steps
    dtype: torch.dtype
    policy: int
    budget_pct: float        # total budget as % of prompt length
    p: float
    n_sink: int = 4
    heavy_num: int = 1
    heavy_den: int = 2
    heavy_mode: str = "none"  # "uniform4" | "zipf" | "none"
    budget_tokens: int = 0    # > 0: the initial per-layer budget in absolute tokens (budget_pct is then unused)

    @property
    def b_init(self) -> int:
        if self.budget_tokens > 0:
            return int(self.budget_tokens)
        return int(math.floor(self.budget_pct * self.prompt / 100.0))

    @property
    def group(self) -> int:
        return self.n_q_head // self.n_kv_head

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def tiny() -> Workload:
    return Workload("tiny_h2o_fp32", 1, 4, 2, 2, 64, 128, 1, 256, 16, torch.float32,
                    H2O, 40.0, 0.3, heavy_mode="uniform4")


def llama2_7b() -> Workload:
    return Workload("llama2_7b_sw_bf16", 2, 32, 32, 32, 128, 4096, 8, 2048, 128, torch.bfloat16,
                    SLIDING_WINDOW, 20.0, 0.3)


def mistral_7b() -> Workload:
    return Workload("mistral_7b_h2o_bf16", 3, 32, 32, 8, 128, 4096, 16, 4096, 256, torch.bfloat16,
                    H2O, 20.0, 0.35, heavy_mode="zipf")


def llama2_70b() -> Workload:
    return Workload("llama2_70b_streaming_bf16", 4, 80, 64, 8, 128, 8192, 32, 4096, 128, torch.bfloat16,
                    STREAMING_LLM, 30.0, 0.3)


def falcon_7b(batch=32, prompt=2048, budget_pct=20.0, policy=SLIDING_WINDOW) -> Workload:
    return Workload(f"falcon_7b_{POLICY_NAMES[policy]}_b{batch}_p{prompt}_{int(budget_pct)}pct", 5,
                    32, 71, 1, 64, 4544, batch, prompt, 128, torch.bfloat16, policy, budget_pct, 0.3,
                    heavy_mode="zipf" if policy == H2O else "none")


def mistral_7b_long_generation(batch=32) -> Workload:
    """Mistral-7B-shaped, the paper's throughput shape (prompt 512, 1024 generated tokens, Sliding
    Window), with the budget given in absolute tokens, above the prompt length: 600 per layer.
    The important layers' caches (about 1040 tokens) keep growing for some 530 steps before
    their first eviction; the others (210 tokens) are compressed already at prefill."""
    return Workload(f"mistral_7b_sw_p512_t1024_abs600_b{batch}", 6, 32, 32, 8, 128, 4096, batch, 512, 1024,
                    torch.bfloat16, SLIDING_WINDOW, 0.0, 0.35, budget_tokens=600)


def falcon_7b_max(policy=SLIDING_WINDOW) -> Workload:
    """The largest cell of the Falcon-shaped sweep: batch 224, prompt 16384, budget 50 %."""
    return falcon_7b(224, 16384, 50.0, policy)


WORKLOADS = {"tiny": tiny, "llama2_7b": llama2_7b, "mistral_7b": mistral_7b,
             "llama2_70b": llama2_70b, "falcon_7b": falcon_7b, "falcon_7b_max": falcon_7b_max,
             "mistral_7b_long_generation": mistral_7b_long_generation}


def _gen(w: Workload, family: int, a: int = 0, b: int = 0, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_BASE_SEED + 1000 * w.wid + family + 7919 * (a + 1) + 104729 * (b + 1))
    return g


def cos_targets(n_layer: int):
    """Target per-layer cosine similarity: a few special layers (first two and
    the last; for deep stacks first three and last two) near 0.60-0.66, the rest
    of the first ~45% near 0.80-0.86, the remainder near 0.95-0.99."""
    L = n_layer
    if L == 4:
        return [0.60, 0.82, 0.97, 0.99]
    if L >= 64:
        special = [0, 1, 2, L - 2, L - 1]
        n_mid = max(1, int(round(0.175 * L)))
    else:
        special = [0, 1, L - 1] if L >= 3 else [0]
        n_mid = max(1, int(round(0.45 * L)) - 2)
    rest = [i for i in range(L) if i not in special]
    mid = rest[:n_mid]
    low = rest[n_mid:]
    c = [0.0] * L
    for j, i in enumerate(special):
        c[i] = 0.60 + 0.06 * j / max(1, len(special) - 1)
    for j, i in enumerate(mid):
        c[i] = 0.80 + 0.06 * j / max(1, len(mid) - 1)
    for j, i in enumerate(low):
        c[i] = 0.95 + 0.04 * j / max(1, len(low) - 1)
    return c


def hidden_pair(w: Workload, layer: int, device="cpu", batch=None, n_tok=None, chunk=0):
    """(hidden_in, hidden_out), each [B, P, hidden]: the state before and after
    self-attention.  hidden_out = hidden_in + alpha_l * noise with alpha_l set
    from the layer's target similarity.  Large batches can be drawn in pieces:
    `batch` sequences per call, `chunk` numbering the pieces."""
    B = w.batch if batch is None else batch
    P = w.prompt if n_tok is None else n_tok
    c = cos_targets(w.n_layer)[layer]
    alpha = math.sqrt(1.0 / (c * c) - 1.0)
    g = _gen(w, 0, layer, chunk, device=device)
    a = torch.randn(B, P, w.hidden, generator=g, device=device, dtype=torch.float32)
    n = torch.randn(B, P, w.hidden, generator=g, device=device, dtype=torch.float32)
    b = a + alpha * n
    return a.to(w.dtype), b.to(w.dtype)


def heavy_dirs(w: Workload, device="cpu"):
    """Unit direction per (layer, KV head) that heavy-hitter keys and all
    queries lean towards: [L, H_kv, d] fp32."""
    g = _gen(w, 5, device=device)
    u = torch.randn(w.n_layer, w.n_kv_head, w.head_dim, generator=g, device=device, dtype=torch.float32)
    return u / u.norm(dim=-1, keepdim=True)


def heavy_positions(w: Workload, layer: int):
    """Prompt positions of the heavy-hitter keys, one 1-D LongTensor per KV head
    (shared by all sequences of the batch)."""
    out = []
    for h in range(w.n_kv_head):
        g = _gen(w, 6, layer, h, device="cpu")
        if w.heavy_mode == "uniform4":
            hi = max(4, w.prompt // 2)
            pos = torch.randperm(hi, generator=g)[:4]
        elif w.heavy_mode == "zipf":
            r = torch.arange(1, w.prompt + 1, dtype=torch.float64)
            prob = r.pow(-1.1)
            draws = torch.multinomial(prob / prob.sum(), 64, replacement=True, generator=g)
            pos = torch.unique(draws)
        else:
            pos = torch.zeros(0, dtype=torch.long)
        out.append(pos.sort().values)
    return out


def _mu(w: Workload) -> float:
    # shifts a heavy key's logit q.k/sqrt(d) by +3 (three standard deviations)
    return math.sqrt(3.0 * math.sqrt(w.head_dim))


def prompt_qkv(w: Workload, layer: int, device="cpu", need_q=True):
    """Prompt tensors of one layer: Q [B, H_q, P, d] (or None), K, V [B, H_kv, P, d]."""
    B, P, d = w.batch, w.prompt, w.head_dim
    heavy = w.heavy_mode != "none"
    u = heavy_dirs(w, device)[layer] if heavy else None         # [H_kv, d]
    mu = _mu(w)
    q = None
    if need_q:
        g = _gen(w, 1, layer, device=device)
        q = torch.randn(B, w.n_q_head, P, d, generator=g, device=device, dtype=torch.float32)
        if heavy:
            q = q + mu * u.repeat_interleave(w.group, dim=0)[None, :, None, :]
        q = q.to(w.dtype)
    g = _gen(w, 2, layer, device=device)
    k = torch.randn(B, w.n_kv_head, P, d, generator=g, device=device, dtype=torch.float32)
    if heavy:
        for h, pos in enumerate(heavy_positions(w, layer)):
            if pos.numel():
                k[:, h, pos.to(device), :] += mu * u[h]
    k = k.to(w.dtype)
    g = _gen(w, 3, layer, device=device)
    v = torch.randn(B, w.n_kv_head, P, d, generator=g, device=device, dtype=torch.float32).to(w.dtype)
    return q, k, v


def prompt_scores_standin(w: Workload, layer: int, device="cpu"):
    """Stand-in for a layer's accumulated prompt attention, fp32 [B, H_kv, P], for runs that fill
    a cache without paying for the quadratic scoring pass: uniform draws scaled to the number of
    query heads, with the heavy-hitter positions lifted well above the rest."""
    g = _gen(w, 7, layer, device=device)
    acc = torch.rand(w.batch, w.n_kv_head, w.prompt, generator=g, device=device, dtype=torch.float32) * w.group
    for h, pos in enumerate(heavy_positions(w, layer)):
        if pos.numel():
            acc[:, h, pos.to(device)] += 50.0 * w.group
    return acc


def decode_qkv(w: Workload, step: int, device="cpu"):
    """Decode-time tensors of one step for all layers:
    q [L, B, H_q, d], k_new, v_new [L, B, H_kv, d]."""
    L, B, d = w.n_layer, w.batch, w.head_dim
    g = _gen(w, 4, step, device=device)
    q = torch.randn(L, B, w.n_q_head, d, generator=g, device=device, dtype=torch.float32)
    k = torch.randn(L, B, w.n_kv_head, d, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(L, B, w.n_kv_head, d, generator=g, device=device, dtype=torch.float32)
    if w.heavy_mode != "none":
        u = heavy_dirs(w, device)                                 # [L, H_kv, d]
        q = q + _mu(w) * u.repeat_interleave(w.group, dim=1)[:, None, :, :]
    return q.to(w.dtype), k.to(w.dtype), v.to(w.dtype)
