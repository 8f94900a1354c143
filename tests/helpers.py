"""Shared plumbing of the GPU parity tests: drives the CUDA library and the CPU oracle with
the same seeded inputs.  Holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np
import torch

from oracle import sq_oracle as O
from paper_2404_04793_b200 import binding as B
from paper_2404_04793_b200 import synth

TOL_OUT = {torch.float32: 1e-5, torch.bfloat16: 1e-2}   # max-abs error on attention outputs / cosines
RTOL_ACC = {torch.float32: 2e-5, torch.bfloat16: 1e-4}  # relative error on H2O scores (fp32 accumulators)


def f64(t):
    return t.detach().to("cpu").to(torch.float64).numpy()


def make_ctx(w: synth.Workload, b_init=None, **over):
    cfg = B.make_config(n_layer=w.n_layer, n_q_head=w.n_q_head, n_kv_head=w.n_kv_head, head_dim=w.head_dim,
                        hidden=w.hidden, max_batch=w.batch, max_prompt=w.prompt, max_new_tokens=max(w.steps, 1),
                        dtype=w.dtype, policy=w.policy, n_sink=w.n_sink, heavy_num=w.heavy_num,
                        heavy_den=w.heavy_den, **over)
    return B.Context(cfg, w.b_init if b_init is None else b_init)


def run_importance_and_allocate(ctx, w, device="cuda", chunks=1, b_init=None, p=None):
    """Feeds every layer's hidden states (optionally in chunks) and allocates budgets.
    Returns the oracle's per-layer cosine similarity."""
    want = feed_importance(ctx, w, device, chunks)
    ctx.allocate_budgets(w.b_init if b_init is None else b_init, w.p if p is None else p)
    return want


def feed_importance(ctx, w, device="cuda", chunks=1):
    ctx.begin_sequence_batch(w.batch, w.prompt)
    want = []
    for l in range(w.n_layer):
        a, b = synth.hidden_pair(w, l, device)
        a2 = a.reshape(-1, w.hidden)
        b2 = b.reshape(-1, w.hidden)
        n = a2.shape[0]
        edges = [round(i * n / chunks) for i in range(chunks + 1)]
        for i in range(chunks):
            if edges[i + 1] > edges[i]:
                ctx.layer_importance(l, a2[edges[i]:edges[i + 1]].contiguous(), b2[edges[i]:edges[i + 1]].contiguous())
        want.append(O.layer_importance(f64(a2), f64(b2)))
    return np.array(want)


def prefill_all(ctx, w, device="cuda", keep_inputs=True):
    """Runs sq_prefill_compress on every layer; returns the prompt tensors (CPU) per layer."""
    kept = []
    for l in range(w.n_layer):
        q, k, v = synth.prompt_qkv(w, l, device, need_q=(w.policy == synth.H2O))
        ctx.prefill_compress(l, k, v, q)
        if keep_inputs:
            kept.append((None if q is None else q.cpu(), k.cpu(), v.cpu()))
    torch.cuda.synchronize()
    return kept


def oracle_unit(w, budgets, prompt_cpu, layer, seq, kvh):
    q, k, v = prompt_cpu[layer]
    g = w.group
    u = O.UnitCache(w.policy, budgets[layer], w.n_sink, w.heavy_num, w.heavy_den)
    qq = None if q is None else f64(q[seq, kvh * g:(kvh + 1) * g])
    u.prefill(f64(k[seq, kvh]), f64(v[seq, kvh]), qq)
    return u


def all_units(w):
    return [(l, s, h) for l in range(w.n_layer) for s in range(w.batch) for h in range(w.n_kv_head)]


def sample_units(w, n, seed=0, every_layer=True):
    """Seeded sample of (layer, sequence, KV head) units: always the first and the last unit and,
    with every_layer, every layer of one sequence and head (so at least n_layer + 2 units)."""
    units = all_units(w)
    if len(units) <= n:
        return units
    rng = np.random.default_rng(seed)
    pick = {0, len(units) - 1}
    s0, h0 = int(rng.integers(w.batch)), int(rng.integers(w.n_kv_head))
    if every_layer:
        for l in range(w.n_layer):
            pick.add((l * w.batch + s0) * w.n_kv_head + h0)
    while len(pick) < n:
        pick.add(int(rng.integers(len(units))))
    return [units[i] for i in sorted(pick)]
