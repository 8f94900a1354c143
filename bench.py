#!/usr/bin/env python
"""Benchmark of the SqueezeAttention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one whole pass of the path over one synthetic batch: layer importance for every
layer, budget allocation, prefill compression of every layer, then all decode steps (one
fused launch per decode step over all layers).  The metric is generated tokens per second
(batch * decode steps / pass time).  With N > 1 every rank runs its own independent batch
(no data-path collective); the value is the sum over ranks / the slowest rank's time.

--impl reference times the CPU oracle (oracle/), as it stands, on the host cores on a bounded
sample of the same workload and extrapolates to the whole job.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2404_04793_b200 import dist_util, synth

METRIC = "decode tokens/sec at 1 B200 and fused attn+evict HBM GB/s as % of roofline"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram bytes (read+write) per decode launch of the default workload, from the ncu capture
# summarised in profiles/decode_attn_llama2_7b_sw_b2.md (batch-2 capture scaled by 4 to batch 8).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"llama2_7b_sw_bf16": 1.7373e9}


def workload_by_name(name):
    if name not in synth.WORKLOADS:
        raise SystemExit(f"unknown workload {name}; choose from {sorted(synth.WORKLOADS)}")
    return synth.WORKLOADS[name]()


# ------------------------------------------------------------------ clocks
class ClockSampler:
    Q = ("timestamp,uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.uuid = str(torch.cuda.get_device_properties(device_index).uuid)
        self.proc = None
        self.path = os.path.join("/tmp", f"sq_clocks_{os.getpid()}.csv")

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def _ts(text):
        import datetime
        try:
            return datetime.datetime.strptime(text.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the wall-clock times t_begin and t_end."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            p = [x.strip() for x in line.split(",")]
            if len(p) < 10 or (self.uuid not in p[1] and p[1] not in self.uuid):
                continue
            ts = self._ts(p[0])
            if ts is not None and t_begin is not None and not (t_begin - 0.1 <= ts <= t_end + 0.1):
                continue
            p = p[1:]
            try:
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            for n, v in zip(names, p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------ CPU oracle leg
def oracle_sample(w, n_units, n_imp_tokens, seed, device):
    """Times the oracle on a bounded sample of the workload and extrapolates linearly to the
    whole job (units of a layer cost the same; importance cost is per token).
    Returns (tokens_per_s, seconds_spent, description)."""
    from threadpoolctl import threadpool_limits
    with threadpool_limits(limits=1):
        return _oracle_sample(w, n_units, n_imp_tokens, seed, device)


def _oracle_sample(w, n_units, n_imp_tokens, seed, device):
    from oracle import sq_oracle as O
    rng = np.random.default_rng(seed)
    f64 = lambda t: t.detach().to("cpu").to(torch.float64).numpy()
    t_start = time.perf_counter()
    # importance: first n_imp_tokens tokens of every 8th layer (cost per token is the same)
    layers_imp = list(range(0, w.n_layer, max(1, w.n_layer // 4)))[:4]
    per_layer = max(1, n_imp_tokens // len(layers_imp))
    cos = np.array(synth.cos_targets(w.n_layer), dtype=np.float64)
    t_imp = 0.0
    n_imp = 0
    for l in layers_imp:
        nb = max(1, min(w.batch, per_layer // w.prompt))
        a, b = synth.hidden_pair(w, l, device, batch=nb, n_tok=min(per_layer, w.prompt))
        a, b = f64(a), f64(b)
        t0 = time.perf_counter()
        cos[l] = O.layer_importance(a, b)
        t_imp += time.perf_counter() - t0
        n_imp += a.shape[0] * a.shape[1] if a.ndim == 3 else a.shape[0]
    t0 = time.perf_counter()
    budgets, _ = O.allocate_budgets(cos.astype(np.float32), w.b_init, w.p)
    t_alloc = time.perf_counter() - t0
    # decode: sampled (layer, sequence, KV head) units, spread evenly over the layers
    layers = sorted(set(int(x) for x in np.linspace(0, w.n_layer - 1, min(n_units, w.n_layer)).round()))
    per = max(1, n_units // len(layers))
    g = w.group
    t_units = {}
    dec = [synth.decode_qkv(w, t, device) for t in range(w.steps)]
    for l in layers:
        q, k, v = synth.prompt_qkv(w, l, device, need_q=(w.policy == synth.H2O))
        spent = 0.0
        for _ in range(per):
            s, h = int(rng.integers(w.batch)), int(rng.integers(w.n_kv_head))
            kk, vv = f64(k[s, h]), f64(v[s, h])
            qq = None if q is None else f64(q[s, h * g:(h + 1) * g])
            steps = [(f64(dq[l, s, h * g:(h + 1) * g]), f64(dk[l, s, h]), f64(dv[l, s, h])) for dq, dk, dv in dec]
            t0 = time.perf_counter()
            u = O.UnitCache(w.policy, int(budgets[l]), w.n_sink, w.heavy_num, w.heavy_den)
            u.prefill(kk, vv, qq)
            for (a1, a2, a3) in steps:
                u.decode_step(a1, a2, a3)
            spent += time.perf_counter() - t0
        t_units[l] = spent / per
    # extrapolate: layers not sampled take the cost of the nearest sampled layer with the same budget class
    def unit_cost(l):
        same = [x for x in layers if budgets[x] == budgets[l]] or layers
        return t_units[min(same, key=lambda x: abs(x - l))]
    t_job = (t_imp / max(n_imp, 1)) * (w.n_layer * w.batch * w.prompt) + t_alloc \
        + sum(unit_cost(l) * w.batch * w.n_kv_head for l in range(w.n_layer))
    tok_s = w.batch * w.steps / t_job
    desc = (f"{len(layers) * per} (layer,seq,kv-head) units over {len(layers)} layers, all {w.steps} decode steps, "
            f"+ {n_imp} tokens of layer importance + the allocator; extrapolated linearly to "
            f"{w.n_layer * w.batch * w.n_kv_head} units and {w.n_layer * w.batch * w.prompt} tokens")
    return tok_s, time.perf_counter() - t_start, desc


def run_reference(args, w):
    rank, local_rank, world = dist_util.world()
    if rank != 0:
        return
    device = "cuda:0" if torch.cuda.is_available() else "cpu"
    vals, secs = [], []
    desc = ""
    for i in range(args.warmup + args.steps):
        v, s, desc = oracle_sample(w, n_units=8, n_imp_tokens=4096, seed=100 + i, device=device)
        if i >= args.warmup:
            vals.append(v); secs.append(s)
    value = len(vals) / sum(1.0 / v for v in vals)      # steps / total extrapolated time
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch * w.steps / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "prompt": w.prompt, "decode_steps": w.steps,
                   "policy": synth.POLICY_NAMES[w.policy], "b_init": w.b_init, "p": w.p},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "sample_seconds_per_step": statistics.mean(secs),
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ our arm
def run_ours(args, w):
    from paper_2404_04793_b200 import engine
    rank, local_rank, world = dist_util.init("nccl")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    # every rank owns an independent batch: a different seed family per rank
    wr = w.replace(wid=w.wid + 100 * rank) if world > 1 else w
    inp = engine.ResidentInputs(wr, dev)
    job = engine.Job(wr, dev, per_layer_decode=args.per_layer_decode)
    tokens = wr.batch * wr.steps

    ev = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(args.warmup):
        job.run(inp)
    torch.cuda.synchronize()
    budgets, is_g3 = job.ctx.get_budgets()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        job.run(inp)                      # keeps the GPU busy while the sampler starts up
    dist_util.barrier()
    torch.cuda.synchronize()
    t_begin = time.time()
    e0, e1 = ev(), ev()
    mids = []
    e0.record()
    for _ in range(args.steps):
        job.prefill(inp)
        a, b = ev(), ev()
        a.record()
        job.decode(inp)
        b.record()
        mids.append((a, b))
    e1.record()
    torch.cuda.synchronize()
    t_end = time.time()
    dist_util.barrier()
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    ms_step = e0.elapsed_time(e1) / args.steps
    ms_decode = sum(a.elapsed_time(b) for a, b in mids) / args.steps
    status = job.ctx.status()
    value, ms_max = dist_util.aggregate_throughput(tokens, ms_step, dev)

    # ---- per-layer launches (what a model that computes q layer by layer issues), replayed from
    # a CUDA graph so that the host's launch cost does not enter ----
    per_layer = None
    if not args.no_per_layer:
        job.prefill(inp)
        graph = job.capture_decode(inp, per_layer=True)
        for _ in range(2):
            job.prefill(inp)
            graph.replay()
        torch.cuda.synchronize()
        n_pl = max(1, min(args.steps, 5))
        tot = 0.0
        for _ in range(n_pl):
            job.prefill(inp)
            a, b = ev(), ev()
            a.record()
            graph.replay()
            b.record()
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        per_layer = {"ms_decode": tot / n_pl, "steps": n_pl}
        del graph

    # ---- end to end: the same pass fed from pinned host memory, outputs copied back ----
    e2e = None
    if not args.no_e2e:
        host = engine.ResidentInputs(wr, "cpu", gen_device=dev)
        out_host = torch.empty(job.out.shape, dtype=job.out.dtype).pin_memory()
        job.run_from_host(host, out_host)
        torch.cuda.synchronize()
        dist_util.barrier()
        s0, s1 = ev(), ev()
        n_e2e = max(1, min(args.steps, 3))
        s0.record()
        for _ in range(n_e2e):
            job.run_from_host(host, out_host)
        s1.record()
        torch.cuda.synchronize()
        dist_util.barrier()
        e2e_val, _ = dist_util.aggregate_throughput(tokens, s0.elapsed_time(s1) / n_e2e, dev)
        e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": host.bytes(),
               "d2h_bytes_per_step": out_host.numel() * out_host.element_size(), "steps": n_e2e}
        del host

    if rank != 0:
        dist_util.shutdown()
        return

    # ---- roofline of the dominant kernel: the fused decode launch ----
    e = 2 if wr.dtype == torch.bfloat16 else 4
    d, L, B = wr.head_dim, wr.n_layer, wr.batch
    kv_tokens = sum(min(wr.prompt + 1, b) for b in budgets)            # per unit, steady state
    alg_bytes = B * wr.n_kv_head * kv_tokens * 2 * d * e \
        + B * L * (wr.n_q_head * d * e * 2 + wr.n_kv_head * 2 * d * e) \
        + (B * wr.n_kv_head * kv_tokens * 8 if wr.policy == synth.H2O else 0)
    launches_per_step = wr.steps * (wr.n_layer if args.per_layer_decode else 1)
    sec_per_launch = ms_decode * 1e-3 / launches_per_step
    bytes_per_launch = alg_bytes / (wr.n_layer if args.per_layer_decode else 1)
    achieved = bytes_per_launch / sec_per_launch / 1e9
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak = float(json.load(open(peaks_path))["hbm_gbs"]); peak_kind = "measured"
    else:
        peak = FALLBACK_HBM_GBS; peak_kind = "fallback"
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None if args.per_layer_decode else NCU_TRAFFIC_BYTES_PER_LAUNCH.get(wr.name), "peak_kind": peak_kind, "kernel": "decode_attn_kernel",
                "algorithmic_bytes_per_launch": bytes_per_launch, "us_per_launch": sec_per_launch * 1e6,
                "frac_of_nominal_8000": achieved / 8000.0}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, secs, desc = oracle_sample(wr, n_units=256, n_imp_tokens=65536, seed=7, device=dev)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc, "seconds": secs}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wr.dtype == torch.bfloat16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "n_layer": L, "n_q_head": wr.n_q_head, "n_kv_head": wr.n_kv_head,
                   "head_dim": d, "batch_per_gpu": B, "prompt": wr.prompt, "decode_steps": wr.steps,
                   "policy": synth.POLICY_NAMES[wr.policy], "b_init": wr.b_init, "p": wr.p,
                   "budgets_min_max": [min(budgets), max(budgets)], "n_g3": int(sum(is_g3)),
                   "decode_launch": "per_layer" if args.per_layer_decode else "all_layers_fused",
                   "l2": "inputs larger than L2 (KV read per decode step %.2f GB)" % (alg_bytes / 1e9),
                   "parallelism": f"dp{world} (independent batches)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": job.kernel_launches_per_pass() * args.steps,
        "roofline": roofline, "cpu_baseline": cpu,
        "decode_only": {"tokens_per_s": tokens / (ms_decode * 1e-3), "ms_per_token_step": ms_decode / wr.steps,
                        "prefill_ms": ms_step - ms_decode},
        "device_status": status,
    }
    if per_layer is not None:
        pl_s = per_layer["ms_decode"] * 1e-3
        line["per_layer_launch"] = {"mode": "one launch per layer per step, CUDA-graph replay",
                                    "decode_tokens_per_s": tokens / pl_s, "us_per_launch": pl_s * 1e6 / (wr.steps * wr.n_layer),
                                    "hbm_gbs": alg_bytes * wr.steps / pl_s / 1e9, "hbm_frac": alg_bytes * wr.steps / pl_s / 1e9 / peak}
    print(json.dumps(line), flush=True)
    dist_util.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b")
    ap.add_argument("--per-layer-decode", action="store_true", help="one decode launch per layer instead of one per step")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-layer", action="store_true", help="skip the per-layer-launch (CUDA graph) measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = workload_by_name(args.workload)
    if args.batch:
        w = w.replace(batch=args.batch, name=w.name + f"_b{args.batch}")
    if args.decode_steps:
        w = w.replace(steps=args.decode_steps, name=w.name + f"_t{args.decode_steps}")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
