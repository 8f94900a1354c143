"""Decode-step micro-benchmark: times sq_decode_step alone on any workload shape.

    python microbench.py --workload falcon_7b --batch 32 --prompt 8192 \
        --budget-pct 30 --policy sliding_window --steps 12 [--per-layer]

The cache is filled through the regular calls (importance on a 256-token slice per layer,
allocation, prefill compression of one random prompt reused for every layer; H2O prompts get
random scores), so only the decode inputs are large.  Prints one JSON line with the step time
and the achieved K/V bandwidth.
"""
from __future__ import annotations

import argparse
import json

import torch

import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2404_04793_b200 import engine, synth  # noqa: E402

POLICIES = {"sliding_window": synth.SLIDING_WINDOW, "streaming_llm": synth.STREAMING_LLM, "h2o": synth.H2O}


def build_workload(args) -> synth.Workload:
    if args.workload == "falcon_7b":
        w = synth.falcon_7b(args.batch or 32, args.prompt or 2048, args.budget_pct or 20.0,
                            POLICIES[args.policy] if args.policy else synth.SLIDING_WINDOW)
    else:
        w = synth.WORKLOADS[args.workload]()
        kw = {}
        if args.batch:
            kw["batch"] = args.batch
        if args.prompt:
            kw["prompt"] = args.prompt
        if args.budget_pct:
            kw["budget_pct"] = args.budget_pct
        if args.policy:
            kw["policy"] = POLICIES[args.policy]
        if kw:
            w = w.replace(**kw)
    return w


def decode_step_time(w: synth.Workload, steps=12, warmup=3, per_layer=False, device="cuda:0", per_sequence=False,
                     sample_clocks=False):
    job = engine.Job(w.replace(steps=steps + warmup), device)
    ctx = job.ctx
    ctx.begin_sequence_batch(w.batch, w.prompt)
    for l in range(w.n_layer):
        a, b = synth.hidden_pair(w, l, device, batch=1, n_tok=256)
        ctx.layer_importance(l, a, b)
    ctx.allocate_budgets(w.b_init, w.p)
    budgets, _ = ctx.get_budgets()
    if per_sequence:
        # same budget vector rotated by one layer per sequence: every sequence has its own
        # budgets (equal totals), as the per-sequence allocation would produce on unlike prompts
        ctx.close()
        ctx = job.ctx = engine.context_for(job.w, device, per_sequence_budgets=1)
        ctx.begin_sequence_batch(w.batch, w.prompt)
        rows = [budgets[s % w.n_layer:] + budgets[:s % w.n_layer] for s in range(w.batch)]
        ctx.set_budgets(rows)
        budgets = [sum(r[l] for r in rows) / w.batch for l in range(w.n_layer)]   # mean per layer, for the byte count
    g = torch.Generator(device=device).manual_seed(1)
    shape_kv = (w.batch, w.n_kv_head, w.prompt, w.head_dim)
    k = torch.randn(shape_kv, generator=g, device=device).to(w.dtype)
    v = torch.randn(shape_kv, generator=g, device=device).to(w.dtype)
    acc = torch.rand(w.batch, w.n_kv_head, w.prompt, generator=g, device=device) if w.policy == synth.H2O else None
    for l in range(w.n_layer):
        ctx.prefill_compress(l, k, v, None, acc)
    q = torch.randn(w.n_layer, w.batch, w.n_q_head, w.head_dim, generator=g, device=device).to(w.dtype)
    kn = torch.randn(w.n_layer, w.batch, w.n_kv_head, w.head_dim, generator=g, device=device).to(w.dtype)
    vn = torch.randn(w.n_layer, w.batch, w.n_kv_head, w.head_dim, generator=g, device=device).to(w.dtype)
    out = torch.empty_like(q)

    def step():
        if per_layer:
            for l in range(w.n_layer):
                ctx.decode_step(l, l + 1, q[l], kn[l], vn[l], out[l])
        else:
            ctx.decode_step(0, w.n_layer, q, kn, vn, out)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = None
    if sample_clocks:
        # SM clock, power and throttle reasons while the timed steps run (a run of a second or
        # more reaches the board's power limit; a few steps do not)
        import time
        from bench import ClockSampler
        sampler = ClockSampler(torch.cuda.current_device())
        sampler.start()
        time.sleep(0.3)
        t_begin = time.time()
    if per_layer:
        # one launch per layer is CPU-bound when issued from Python: time a CUDA-graph replay of
        # the same launches instead (kernel arguments frozen at capture; the caches are full, so
        # every replay does the same work)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(steps):
                step()
        if w.policy != synth.H2O:
            graph.replay()
        # (H2O: the captured steps carry their token positions, so a second replay would hand the
        # score pass positions that run backwards; the first replay is the one that is timed)
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
    else:
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop(t_begin, time.time()) if sampler else None
    ms = e0.elapsed_time(e1) / steps
    e = 2 if w.dtype == torch.bfloat16 else 4
    kv = int(w.batch * w.n_kv_head * sum(min(w.prompt + 1, b) for b in budgets) * 2 * w.head_dim * e)
    io = w.batch * w.n_layer * (2 * w.n_q_head + 2 * w.n_kv_head) * w.head_dim * e
    extra = int(w.batch * w.n_kv_head * sum(budgets) * 8) if w.policy == synth.H2O else 0
    gbs = (kv + io + extra) / ms / 1e6
    return dict(workload=w.name, per_layer=per_layer, per_sequence_budgets=per_sequence, ms_per_step=round(ms, 4), GBs=round(gbs, 1),
                kv_GB=round(kv / 1e9, 3), algorithmic_bytes=kv + io + extra, tokens_per_s=round(w.batch / ms * 1e3),
                flops=int(4 * w.n_q_head * w.head_dim * w.batch * sum(budgets)), device_status=ctx.status(),
                **({"clocks": clocks} if clocks else {}))


def prefill_compress_time(w: synth.Workload, reps=3, device="cuda:0"):
    """Times sq_prefill_compress of one layer (for H2O: prompt scores on the tensor cores,
    selection, gather, first victim)."""
    job = engine.Job(w.replace(steps=1), device)
    ctx = job.ctx
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets([w.b_init] * w.n_layer)
    q, k, v = synth.prompt_qkv(w, 0, device, need_q=(w.policy == synth.H2O))
    ctx.prefill_compress(0, k, v, q)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        ctx.prefill_compress(0, k, v, q)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    flops = 2 * w.batch * w.n_q_head * w.prompt * w.prompt * w.head_dim if w.policy == synth.H2O else 0
    return dict(workload=w.name, what="prefill_compress, one layer", ms=round(ms, 3),
                causal_score_flops=flops, tflops=round(flops / ms / 1e9, 1), device_status=ctx.status())


def touch_all_kernels(w: synth.Workload, device="cuda:0"):
    """One short pass that launches every kernel of the library on a workload (importance,
    allocator, prefill scoring / selection / gather, decode steps, explicit eviction to half the
    budgets): the command behind the per-kernel profiler summaries."""
    job = engine.Job(w, device)
    ctx = job.ctx
    ctx.begin_sequence_batch(w.batch, w.prompt)
    for l in range(w.n_layer):
        a, b = synth.hidden_pair(w, l, device)
        ctx.layer_importance(l, a, b)
        del a, b
    ctx.allocate_budgets(w.b_init, w.p)
    budgets, _ = ctx.get_budgets()
    for l in range(w.n_layer):
        q, k, v = synth.prompt_qkv(w, l, device, need_q=(w.policy == synth.H2O))
        ctx.prefill_compress(l, k, v, q)
        del q, k, v
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, device)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
    floor = (w.n_sink + 1) if w.policy == synth.STREAMING_LLM else 1
    ctx.evict(0, w.n_layer, [max(floor, b // 2) for b in budgets])
    torch.cuda.synchronize()
    return dict(workload=w.name, what="every kernel once", budgets=budgets, device_status=ctx.status())


def evict_time(w: synth.Workload, reps=3, device="cuda:0"):
    """Times one explicit eviction (sq_evict over all layers, budgets halved) on caches filled to
    their budgets; the context is refilled before every repetition, since an eviction is not
    repeatable.  Algorithmic bytes: the rows that stay, read and written once each (K and V,
    positions, and scores for H2O)."""
    job = engine.Job(w.replace(steps=1), device)
    ctx = job.ctx
    g = torch.Generator(device=device).manual_seed(1)
    shape_kv = (w.batch, w.n_kv_head, w.prompt, w.head_dim)
    k = torch.randn(shape_kv, generator=g, device=device).to(w.dtype)
    v = torch.randn(shape_kv, generator=g, device=device).to(w.dtype)
    acc = torch.rand(w.batch, w.n_kv_head, w.prompt, generator=g, device=device) if w.policy == synth.H2O else None
    floor = (w.n_sink + 1) if w.policy == synth.STREAMING_LLM else 1
    times = []
    for _ in range(reps + 1):
        ctx.begin_sequence_batch(w.batch, w.prompt)
        for l in range(w.n_layer):
            a, b = synth.hidden_pair(w, l, device, batch=1, n_tok=256)
            ctx.layer_importance(l, a, b)
        ctx.allocate_budgets(w.b_init, w.p)
        budgets, _ = ctx.get_budgets()
        for l in range(w.n_layer):
            ctx.prefill_compress(l, k, v, None, acc)
        new = [max(floor, b // 2) for b in budgets]
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.evict(0, w.n_layer, new)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = min(times[1:])
    e = 2 if w.dtype == torch.bfloat16 else 4
    per_row = 2 * w.head_dim * e + 4 + (4 if w.policy == synth.H2O else 0)
    moved = 2 * w.batch * w.n_kv_head * sum(min(n, min(w.prompt, b)) for n, b in zip(new, budgets)) * per_row
    return dict(workload=w.name, what="sq_evict, all layers, budgets halved", ms=round(ms, 4), all_ms=[round(t, 4) for t in times],
                algorithmic_bytes=moved, GBs=round(moved / ms / 1e6, 1), device_status=ctx.status())


def generation_throughput(w: synth.Workload, device="cuda:0"):
    """Decode tokens/s of the attention + eviction path over a whole generation: cache filled
    from a prompt of w.prompt tokens, then w.steps fused decode steps, all timed together."""
    job = engine.Job(w, device)
    ctx = job.ctx
    ctx.begin_sequence_batch(w.batch, w.prompt)
    for l in range(w.n_layer):
        a, b = synth.hidden_pair(w, l, device, batch=1, n_tok=min(256, w.prompt))
        ctx.layer_importance(l, a, b)
    ctx.allocate_budgets(w.b_init, w.p)
    budgets, _ = ctx.get_budgets()
    g = torch.Generator(device=device).manual_seed(1)
    shape_kv = (w.batch, w.n_kv_head, w.prompt, w.head_dim)
    k = torch.randn(shape_kv, generator=g, device=device).to(w.dtype)
    v = torch.randn(shape_kv, generator=g, device=device).to(w.dtype)
    acc = torch.rand(w.batch, w.n_kv_head, w.prompt, generator=g, device=device) if w.policy == synth.H2O else None
    q = torch.randn(w.n_layer, w.batch, w.n_q_head, w.head_dim, generator=g, device=device).to(w.dtype)
    kn = torch.randn(w.n_layer, w.batch, w.n_kv_head, w.head_dim, generator=g, device=device).to(w.dtype)
    vn = torch.randn(w.n_layer, w.batch, w.n_kv_head, w.head_dim, generator=g, device=device).to(w.dtype)
    out = torch.empty_like(q)

    def one_generation():
        for l in range(w.n_layer):
            ctx.prefill_compress(l, k, v, None, acc)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(w.steps):
            ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    one_generation()
    ms = one_generation()
    e = 2 if w.dtype == torch.bfloat16 else 4
    cache_gb = w.batch * w.n_kv_head * sum(min(w.prompt + w.steps, b) for b in budgets) * 2 * w.head_dim * e / 1e9
    return dict(workload=w.name, batch=w.batch, budget_pct=w.budget_pct, p=w.p, ms_total=round(ms, 2),
                tokens_per_s=round(w.batch * w.steps / ms * 1e3), final_cache_GB=round(cache_gb, 2),
                device_status=ctx.status())


def importance_time(w: synth.Workload, reps=5, device="cuda:0", n_seq=4):
    """Layer importance of one layer's hidden states (n_seq sequences of the workload's prompt
    length): the separate pass over (hidden_in, hidden_out); the producer's own residual addition
    (an elementwise kernel) followed by that pass; and the fused call that writes the sum and
    takes the statistic in one pass."""
    job = engine.Job(w.replace(steps=1, batch=n_seq), device)
    ctx = job.ctx
    ctx.begin_sequence_batch(n_seq, w.prompt)
    a, b = synth.hidden_pair(w, 0, device, batch=n_seq)
    attn = (b.float() - a.float()).to(w.dtype)
    out = torch.empty_like(a)
    nbytes = a.numel() * a.element_size()

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    ms_sep = timed(lambda: ctx.layer_importance(0, a, b))
    ms_two = timed(lambda: (torch.add(a, attn, out=out), ctx.layer_importance(0, a, out)))
    ms_fused = timed(lambda: ctx.layer_importance_fused(0, a, attn, out))
    return dict(workload=w.name, what="layer importance, one layer", tokens=n_seq * w.prompt, bytes_per_array=nbytes,
                separate_pass_ms=round(ms_sep, 4), separate_pass_GBs=round(2 * nbytes / ms_sep / 1e6, 1),
                add_then_pass_ms=round(ms_two, 4), add_then_pass_GBs=round(5 * nbytes / ms_two / 1e6, 1),
                fused_ms=round(ms_fused, 4), fused_GBs=round(3 * nbytes / ms_fused / 1e6, 1), device_status=ctx.status())


def compare_budgets():
    """Full cache vs a sequence-wise policy alone vs the layer-wise reallocation on the same
    kernels, on the shapes of the paper's throughput table (attention path only, no weights)."""
    rows = []
    shapes = [("mistral_7b", 512, 1024, synth.SLIDING_WINDOW, (1, 32, 64, 128, 224), 30.0, 20.0, 0.35),
              ("llama2_70b", 256, 512, synth.STREAMING_LLM, (1, 8, 16, 32, 64), 40.0, 30.0, 0.3)]
    for name, P, T, policy, batches, pct_alone, pct_squeeze, p in shapes:
        base = synth.WORKLOADS[name]().replace(prompt=P, steps=T, policy=policy)
        full_pct = 100.0 * (P + T) / P + 1.0
        for batch in batches:
            for label, pct, pp in (("full cache", full_pct, 1.0), ("sequence-wise alone", pct_alone, 1.0),
                                   ("layer-wise budgets", pct_squeeze, p)):
                w = base.replace(batch=batch, budget_pct=pct, p=pp, name=f"{name}_{label.replace(' ', '_')}")
                r = generation_throughput(w)
                r.update(shape=name, variant=label, prompt=P, gen=T)
                rows.append(r)
                print(json.dumps(r), flush=True)
                torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama2_7b")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--prompt", type=int, default=0)
    ap.add_argument("--budget-pct", type=float, default=0.0)
    ap.add_argument("--policy", default="")
    ap.add_argument("--steps", type=int, default=12)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--per-layer", action="store_true")
    ap.add_argument("--sample-clocks", action="store_true", help="decode step: SM clock, power and throttle reasons during the timed steps")
    ap.add_argument("--per-sequence", action="store_true", help="per-sequence budgets (a rotated budget vector per sequence)")
    ap.add_argument("--prefill", action="store_true", help="time sq_prefill_compress of one layer instead")
    ap.add_argument("--importance", action="store_true", help="time sq_layer_importance, separate and fused with the residual addition")
    ap.add_argument("--evict", action="store_true", help="time one explicit eviction of all layers to half the budgets")
    ap.add_argument("--all-kernels", action="store_true", help="launch every kernel of the library once or a few times")
    ap.add_argument("--layers", type=int, default=0, help="with --all-kernels: number of layers of the shape to keep")
    ap.add_argument("--compare-budgets", action="store_true",
                    help="generation throughput: full cache vs sequence-wise policy alone vs layer-wise budgets")
    ap.add_argument("--sweep-falcon", action="store_true",
                    help="decode-step time over the Falcon-7B-shaped grid: batch x prompt x budget x policy")
    args = ap.parse_args()
    if args.all_kernels:
        w = build_workload(args)
        kw = dict(steps=args.steps)
        if args.layers:
            kw["n_layer"] = args.layers
        print(json.dumps(touch_all_kernels(w.replace(**kw))), flush=True)
        return
    if args.compare_budgets:
        compare_budgets()
        return
    if args.sweep_falcon:
        for policy in ([args.policy] if args.policy else ["sliding_window", "streaming_llm", "h2o"]):
            for batch in (1, 8, 32, 128, 224):
                for prompt in (512, 2048, 8192, 16384):
                    for pct in (10.0, 20.0, 30.0, 50.0):
                        w = synth.falcon_7b(batch, prompt, pct, POLICIES[policy])
                        r = decode_step_time(w, args.steps, args.warmup, args.per_layer)
                        r.update(policy=policy, batch=batch, prompt=prompt, budget_pct=pct)
                        print(json.dumps(r), flush=True)
                        torch.cuda.empty_cache()
        return
    if args.importance:
        print(json.dumps(importance_time(build_workload(args), args.steps)), flush=True)
        return
    if args.prefill:
        print(json.dumps(prefill_compress_time(build_workload(args), args.steps)), flush=True)
        return
    if args.evict:
        print(json.dumps(evict_time(build_workload(args), min(args.steps, 5))), flush=True)
        return
    print(json.dumps(decode_step_time(build_workload(args), args.steps, args.warmup, args.per_layer,
                                      per_sequence=args.per_sequence, sample_clocks=args.sample_clocks)), flush=True)


if __name__ == "__main__":
    main()
