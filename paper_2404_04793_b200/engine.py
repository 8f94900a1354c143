"""Drives one whole pass of Algorithm 1 over a synthetic workload through the C ABI:
layer importance for every layer, budget allocation, prefill compression of every layer,
then the decode steps.  Pure orchestration: every step runs in the library's kernels."""
from __future__ import annotations

import torch

from . import binding as B
from . import synth


def context_for(w: synth.Workload, device, **over) -> B.Context:
    cfg = B.make_config(n_layer=w.n_layer, n_q_head=w.n_q_head, n_kv_head=w.n_kv_head, head_dim=w.head_dim,
                        hidden=w.hidden, max_batch=w.batch, max_prompt=w.prompt, max_new_tokens=max(w.steps, 1),
                        dtype=w.dtype, policy=w.policy, n_sink=w.n_sink, heavy_num=w.heavy_num,
                        heavy_den=w.heavy_den, **over)
    return B.Context(cfg, w.b_init, device)


def _empty(shape, dtype, device):
    if str(device) == "cpu":
        return torch.empty(shape, dtype=dtype, pin_memory=True)   # page-locked: copies can be asynchronous
    return torch.empty(shape, dtype=dtype, device=device)


class ResidentInputs:
    """All inputs of one job, drawn once on `gen_device` and kept on `device` ("cuda:N", or "cpu":
    page-locked host memory).

    hidden_seqs: the hidden states of a layer are drawn for this many distinct sequences; the
    batch is made of batch / hidden_seqs repeats of them (the importance reduction still reads
    every token's bytes: a layer's chunk is fed that many times).  Default: the whole batch.
    prompt_layers: distinct layers of prompt tensors kept (layer l uses l % prompt_layers);
    default all.
    standin_scores: H2O only: keep stand-in prompt scores (synth.prompt_scores_standin) instead of
    the prompt's queries, so that filling the cache skips the quadratic scoring pass."""

    def __init__(self, w: synth.Workload, device, gen_device=None, hidden_seqs=None, prompt_layers=None,
                 standin_scores=False):
        self.w = w
        gen_device = gen_device or device
        self.hidden_seqs = w.batch if hidden_seqs is None else int(hidden_seqs)
        if w.batch % self.hidden_seqs:
            raise ValueError("hidden_seqs must divide the batch")
        self.hidden_repeat = w.batch // self.hidden_seqs
        n_pl = w.n_layer if prompt_layers is None else max(1, min(int(prompt_layers), w.n_layer))
        need_q = w.policy == synth.H2O and not standin_scores
        self.acc = None

        def place(t):
            out = _empty(t.shape, t.dtype, device)
            out.copy_(t)
            return out

        self.hidden, self._prompt = [], []
        for l in range(w.n_layer):
            a, b = synth.hidden_pair(w, l, gen_device, batch=self.hidden_seqs)
            self.hidden.append((place(a), place(b)))
            del a, b
        for l in range(n_pl):
            q, k, v = synth.prompt_qkv(w, l, gen_device, need_q=need_q)
            self._prompt.append((None if q is None else place(q), place(k), place(v)))
            del q, k, v
        if w.policy == synth.H2O and standin_scores:
            self.acc = [place(synth.prompt_scores_standin(w, l, gen_device)) for l in range(n_pl)]
        L, Bt, d = w.n_layer, w.batch, w.head_dim
        self.q = _empty((w.steps, L, Bt, w.n_q_head, d), w.dtype, device)
        self.k_new = _empty((w.steps, L, Bt, w.n_kv_head, d), w.dtype, device)
        self.v_new = _empty((w.steps, L, Bt, w.n_kv_head, d), w.dtype, device)
        for t in range(w.steps):
            q, k, v = synth.decode_qkv(w, t, gen_device)
            self.q[t].copy_(q); self.k_new[t].copy_(k); self.v_new[t].copy_(v)
            del q, k, v

    def prompt(self, layer):
        return self._prompt[layer % len(self._prompt)]

    def scores(self, layer):
        return None if self.acc is None else self.acc[layer % len(self.acc)]

    def bytes_per_pass(self):
        """Bytes a pass fed from here moves: every distinct tensor once (a layer's hidden chunk is
        sent once and then read hidden_repeat times on the device)."""
        w = self.w
        n = self.q.numel() * self.q.element_size() + 2 * self.k_new.numel() * self.k_new.element_size()
        for a, b in self.hidden:
            n += 2 * a.numel() * a.element_size()
        for l in range(w.n_layer):
            q, k, v = self.prompt(l)
            n += 2 * k.numel() * k.element_size() + (0 if q is None else q.numel() * q.element_size())
        return n


class Job:
    """One context and the launch sequence of a whole pass."""

    def __init__(self, w: synth.Workload, device, per_layer_decode=False, keep_steps=None, exchange=None):
        self.w = w
        self.exchange = exchange  # called with the context after the importance pass (one batch sharded over ranks)
        self.device = torch.device(device)
        self.ctx = context_for(w, device)
        self.per_layer_decode = per_layer_decode
        n_out = w.steps if keep_steps is None else keep_steps     # outputs of step t land in slot t % n_out
        self.out = torch.empty(n_out, w.n_layer, w.batch, w.n_q_head, w.head_dim, dtype=w.dtype, device=device)

    # ---- phases over device-resident inputs ----
    def prefill(self, inp: ResidentInputs):
        w, ctx = self.w, self.ctx
        ctx.begin_sequence_batch(w.batch, w.prompt)
        for l in range(w.n_layer):
            a, b = inp.hidden[l]
            for _ in range(inp.hidden_repeat):
                ctx.layer_importance(l, a, b)
        if self.exchange is not None:
            self.exchange(ctx)  # a batch sharded over ranks: the layer sums of all ranks, once, before the allocation
        ctx.allocate_budgets(w.b_init, w.p)
        for l in range(w.n_layer):
            q, k, v = inp.prompt(l)
            ctx.prefill_compress(l, k, v, q, inp.scores(l))

    def decode(self, inp: ResidentInputs, steps=None):
        w, ctx = self.w, self.ctx
        n_out = self.out.shape[0]
        for t in range(w.steps if steps is None else steps):
            o = self.out[t % n_out]
            if self.per_layer_decode:
                for l in range(w.n_layer):
                    ctx.decode_step(l, l + 1, inp.q[t, l], inp.k_new[t, l], inp.v_new[t, l], o[l])
            else:
                ctx.decode_step(0, w.n_layer, inp.q[t], inp.k_new[t], inp.v_new[t], o)

    def run(self, inp: ResidentInputs):
        self.prefill(inp)
        self.decode(inp)

    def capture_decode(self, inp: ResidentInputs, per_layer: bool, steps=None):
        """Captures the decode steps of a pass (one launch per layer if per_layer, else one per
        step) into a CUDA graph.  Call right after prefill(inp): the kernel arguments, among
        them each step's token position, are frozen at capture, so the graph replays exactly
        the steps that follow a prefill of this workload.  The library's host-side step counter
        advances during capture and not during replay: use replays for timing, and the plain
        calls when the cache is inspected afterwards."""
        saved = self.per_layer_decode
        self.per_layer_decode = per_layer
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.decode(inp, steps)
        self.per_layer_decode = saved
        return graph

    def kernel_launches_per_pass(self, inp: ResidentInputs, per_layer_decode=None) -> int:
        """Kernels of the library launched by one pass: importance per layer and chunk feed, one
        allocator, prefill kernels per layer, decode kernels per step."""
        w = self.w
        per_layer = self.per_layer_decode if per_layer_decode is None else per_layer_decode
        h2o = w.policy == synth.H2O
        # H2O: two scoring sweeps (unless stand-in scores are given), selection, gather, first victim
        per_layer_prefill = ((0 if inp.acc is not None else 2) + 1 + 1 + 1) if h2o else 1
        groups = w.n_layer if per_layer else 1
        per_step = groups * (2 if h2o else 1)
        return w.n_layer * inp.hidden_repeat + 1 + w.n_layer * per_layer_prefill + w.steps * per_step

    # ---- the same pass fed from page-locked host memory ----
    def run_from_host(self, host: ResidentInputs, out_host: torch.Tensor):
        """Every input crosses PCIe inside the call (double-buffered device staging, copies on
        a side stream overlapped with the kernels) and every step's output is copied back into
        out_host[t % len(out_host)]."""
        w, ctx, dev = self.w, self.ctx, self.device
        if host.acc is not None:
            raise ValueError("run_from_host computes the prompt scores from the prompt's queries")
        if not hasattr(self, "_stage"):
            a, b = host.hidden[0]
            q, k, v = host.prompt(0)
            mk = lambda t: None if t is None else torch.empty_like(t, device=dev)
            self._stage = [dict(a=mk(a), b=mk(b), q=mk(q), k=mk(k), v=mk(v)) for _ in range(2)]
            self._dq = [torch.empty_like(host.q[0], device=dev) for _ in range(2)]
            self._dk = [torch.empty_like(host.k_new[0], device=dev) for _ in range(2)]
            self._dv = [torch.empty_like(host.v_new[0], device=dev) for _ in range(2)]
            self._copy = torch.cuda.Stream(device=dev)
        main = torch.cuda.current_stream(dev)
        cp = self._copy
        ready = [torch.cuda.Event() for _ in range(2)]
        freed = [torch.cuda.Event() for _ in range(2)]
        for e in freed:
            e.record(main)

        def pipeline(n, load, use):
            # load(i, slot) on the copy stream, use(i, slot) on the main stream, two slots
            for i in range(n + 1):
                if i < n:
                    s = i % 2
                    cp.wait_event(freed[s])
                    with torch.cuda.stream(cp):
                        load(i, s)
                        ready[s].record(cp)
                if i >= 1:
                    s = (i - 1) % 2
                    main.wait_event(ready[s])
                    use(i - 1, s)
                    freed[s].record(main)

        ctx.begin_sequence_batch(w.batch, w.prompt)

        def load_h(l, s):
            self._stage[s]["a"].copy_(host.hidden[l][0], non_blocking=True)
            self._stage[s]["b"].copy_(host.hidden[l][1], non_blocking=True)

        def use_h(l, s):
            for _ in range(host.hidden_repeat):
                ctx.layer_importance(l, self._stage[s]["a"], self._stage[s]["b"])

        pipeline(w.n_layer, load_h, use_h)
        ctx.allocate_budgets(w.b_init, w.p)

        def load_p(l, s):
            q, k, v = host.prompt(l)
            if q is not None:
                self._stage[s]["q"].copy_(q, non_blocking=True)
            self._stage[s]["k"].copy_(k, non_blocking=True)
            self._stage[s]["v"].copy_(v, non_blocking=True)

        pipeline(w.n_layer, load_p,
                 lambda l, s: ctx.prefill_compress(l, self._stage[s]["k"], self._stage[s]["v"], self._stage[s]["q"]))

        n_out, n_host = self.out.shape[0], out_host.shape[0]

        def load_d(t, s):
            self._dq[s].copy_(host.q[t], non_blocking=True)
            self._dk[s].copy_(host.k_new[t], non_blocking=True)
            self._dv[s].copy_(host.v_new[t], non_blocking=True)

        def use_d(t, s):
            o = self.out[t % n_out]
            if self.per_layer_decode:
                for l in range(w.n_layer):
                    ctx.decode_step(l, l + 1, self._dq[s][l], self._dk[s][l], self._dv[s][l], o[l])
            else:
                ctx.decode_step(0, w.n_layer, self._dq[s], self._dk[s], self._dv[s], o)
            out_host[t % n_host].copy_(self.out[t % n_out], non_blocking=True)

        pipeline(w.steps, load_d, use_d)
