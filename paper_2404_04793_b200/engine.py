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


class ResidentInputs:
    """All inputs of one job, generated once on `device` ("cuda:N" or "cpu"; CPU tensors are
    pinned so they can be copied asynchronously)."""

    def __init__(self, w: synth.Workload, device, gen_device=None):
        self.w = w
        gen_device = gen_device or device
        pin = (str(device) == "cpu")

        def place(t):
            t = t.to(device)
            return t.pin_memory() if pin else t

        need_q = w.policy == synth.H2O
        self.hidden, self.prompt = [], []
        for l in range(w.n_layer):
            a, b = synth.hidden_pair(w, l, gen_device)
            self.hidden.append((place(a), place(b)))
            q, k, v = synth.prompt_qkv(w, l, gen_device, need_q=need_q)
            self.prompt.append((None if q is None else place(q), place(k), place(v)))
        qs, ks, vs = [], [], []
        for t in range(w.steps):
            q, k, v = synth.decode_qkv(w, t, gen_device)
            qs.append(q); ks.append(k); vs.append(v)
        self.q = place(torch.stack(qs))
        self.k_new = place(torch.stack(ks))
        self.v_new = place(torch.stack(vs))

    def bytes(self):
        n = self.q.numel() * self.q.element_size() + 2 * self.k_new.numel() * self.k_new.element_size()
        for a, b in self.hidden:
            n += 2 * a.numel() * a.element_size()
        for q, k, v in self.prompt:
            n += 2 * k.numel() * k.element_size() + (0 if q is None else q.numel() * q.element_size())
        return n


class Job:
    """One context and the launch sequence of a whole pass."""

    def __init__(self, w: synth.Workload, device, per_layer_decode=False):
        self.w = w
        self.device = torch.device(device)
        self.ctx = context_for(w, device)
        self.per_layer_decode = per_layer_decode
        self.out = torch.empty(w.steps, w.n_layer, w.batch, w.n_q_head, w.head_dim, dtype=w.dtype, device=device)

    # ---- phases over device-resident inputs ----
    def prefill(self, inp: ResidentInputs):
        w, ctx = self.w, self.ctx
        ctx.begin_sequence_batch(w.batch, w.prompt)
        for l in range(w.n_layer):
            a, b = inp.hidden[l]
            ctx.layer_importance(l, a, b)
        ctx.allocate_budgets(w.b_init, w.p)
        for l in range(w.n_layer):
            q, k, v = inp.prompt[l]
            ctx.prefill_compress(l, k, v, q)

    def decode(self, inp: ResidentInputs, steps=None):
        w, ctx = self.w, self.ctx
        for t in range(w.steps if steps is None else steps):
            if self.per_layer_decode:
                for l in range(w.n_layer):
                    ctx.decode_step(l, l + 1, inp.q[t, l], inp.k_new[t, l], inp.v_new[t, l], self.out[t, l])
            else:
                ctx.decode_step(0, w.n_layer, inp.q[t], inp.k_new[t], inp.v_new[t], self.out[t])

    def run(self, inp: ResidentInputs):
        self.prefill(inp)
        self.decode(inp)

    def capture_decode(self, inp: ResidentInputs, per_layer: bool):
        """Captures all decode steps of a pass (one launch per layer if per_layer, else one per
        step) into a CUDA graph.  Call right after prefill(inp): the kernel arguments, among
        them each step's token position, are frozen at capture, so the graph replays exactly
        the steps that follow a prefill of this workload.  The library's host-side step counter
        advances during capture and not during replay: use replays for timing, and the plain
        calls when the cache is inspected afterwards."""
        saved = self.per_layer_decode
        self.per_layer_decode = per_layer
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.decode(inp)
        self.per_layer_decode = saved
        return graph

    def kernel_launches_per_pass(self) -> int:
        """Kernels of the library launched by one run(): importance per layer, one allocator,
        prefill kernels per layer, decode kernels per step."""
        w = self.w
        h2o = w.policy == synth.H2O
        per_layer_prefill = (2 + 1 + 1 + 1) if h2o else 1   # scores x2, select, gather, first victim
        groups = w.n_layer if self.per_layer_decode else 1
        per_step = groups * (2 if h2o else 1)
        return w.n_layer + 1 + w.n_layer * per_layer_prefill + w.steps * per_step

    # ---- the same pass fed from pinned host memory ----
    def run_from_host(self, host: ResidentInputs, out_host: torch.Tensor):
        """Every input crosses PCIe inside the call (double-buffered device staging, copies on
        a side stream overlapped with the kernels) and every step's output is copied back."""
        w, ctx, dev = self.w, self.ctx, self.device
        if not hasattr(self, "_stage"):
            a, b = host.hidden[0]
            q, k, v = host.prompt[0]
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

        pipeline(w.n_layer, load_h, lambda l, s: ctx.layer_importance(l, self._stage[s]["a"], self._stage[s]["b"]))
        ctx.allocate_budgets(w.b_init, w.p)

        def load_p(l, s):
            q, k, v = host.prompt[l]
            if q is not None:
                self._stage[s]["q"].copy_(q, non_blocking=True)
            self._stage[s]["k"].copy_(k, non_blocking=True)
            self._stage[s]["v"].copy_(v, non_blocking=True)

        pipeline(w.n_layer, load_p,
                 lambda l, s: ctx.prefill_compress(l, self._stage[s]["k"], self._stage[s]["v"], self._stage[s]["q"]))

        def load_d(t, s):
            self._dq[s].copy_(host.q[t], non_blocking=True)
            self._dk[s].copy_(host.k_new[t], non_blocking=True)
            self._dv[s].copy_(host.v_new[t], non_blocking=True)

        def use_d(t, s):
            ctx.decode_step(0, w.n_layer, self._dq[s], self._dk[s], self._dv[s], self.out[t])
            out_host[t].copy_(self.out[t], non_blocking=True)

        pipeline(w.steps, load_d, use_d)
