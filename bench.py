#!/usr/bin/env python
"""Benchmark of the SqueezeAttention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one whole pass of the path over one synthetic batch: layer importance for every
layer, budget allocation, prefill compression of every layer, then all decode steps, each
decode step issued as one launch per layer (what a model that computes a layer's query from the
previous layer's output has to issue), replayed from a CUDA graph.  The metric is generated
tokens per second (batch * decode steps / pass time).  The default workload is the largest cell
of the Falcon-7B-shaped sweep (batch 224, prompt 16384, budget 50 %, Sliding Window: 15 GB of
K/V read per decode step).  Beside the headline the line carries the same decode steps as one
fused launch over all layers (an upper bound no model can issue), decode-step records of the
other paper-shaped configurations, the whole pass of the Llama-2-7B-shaped configuration, the
pass fed from host memory, and the CPU oracle's timing.

With --gpus N > 1 and no RANK in the environment the script starts N ranks itself (one per
GPU); every rank runs its own independent batch (no data-path collective) and the value is the
sum of the ranks' tokens over the slowest rank's time.

--impl reference times the CPU oracle (oracle/), as it stands, on the host cores on a bounded
sample of the same workload per step and extrapolates to the whole job.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

# torch and the package are imported inside the functions that need them: the worker processes
# of the all-cores oracle timing import this file and need neither.

METRIC = "decode tokens/sec at 1 B200 and fused attn+evict HBM GB/s as % of roofline"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
DEFAULT_WORKLOAD = "falcon_7b_max"
# DRAM bytes (read + write) per byte of K/V a decode launch has to read, from ncu captures of each
# decode kernel on a small case (traffic grows in proportion to the units processed, each unit's
# K/V being read once); None once a kernel has changed since its counters were taken.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = {"decode_attn_kernel": 1.008, "decode_attn_tc_kernel": 1.018,
                                    "decode_attn_tc_stream_kernel": 1.033, "decode_attn_mma_kernel": None}


def workload_by_name(name):
    from paper_2404_04793_b200 import synth
    if name not in synth.WORKLOADS:
        raise SystemExit(f"unknown workload {name}; choose from {sorted(synth.WORKLOADS)}")
    return synth.WORKLOADS[name]()


def config_of(w, world, shard_batch=False):
    """The workload as the JSON line names it (both arms print the same keys)."""
    from paper_2404_04793_b200 import synth
    how = ("one batch sharded by sequence; one all-reduce of 2 x n_layer numbers per pass before the allocation"
           if shard_batch else "independent batches")
    return {"workload": w.name, "n_layer": w.n_layer, "n_q_head": w.n_q_head, "n_kv_head": w.n_kv_head,
            "head_dim": w.head_dim, "hidden": w.hidden, "batch_per_gpu": w.batch, "prompt": w.prompt,
            "decode_steps": w.steps, "policy": synth.POLICY_NAMES[w.policy], "b_init": w.b_init, "p": w.p,
            "parallelism": f"dp{world} ({how})"}


def maybe_spawn(argv, gpus):
    """`--gpus N` outside a launcher: start the N ranks and return their exit code; else None."""
    if gpus <= 1 or "RANK" in os.environ:
        return None
    from paper_2404_04793_b200 import dist_util
    return dist_util.spawn_ranks(gpus, [sys.executable, os.path.abspath(__file__), *argv])


# ------------------------------------------------------------------ clocks
class ClockSampler:
    Q = ("timestamp,uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        import torch
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
        sm, mx, watts, reasons = [], [], [], set()
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
            try:
                watts.append(float(p[3]))
            except ValueError:
                pass
            for n, v in zip(names, p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
            if watts:
                out["power_w"] = statistics.median(watts)
        return out


# ------------------------------------------------------------ CPU oracle leg
def _one_thread():
    from threadpoolctl import threadpool_limits
    return threadpool_limits(limits=1)


def oracle_unit_task(task):
    """One (layer, sequence, KV head) unit through the oracle: prompt, then its decode steps.
    Returns the seconds it took, the decode steps scaled to the trajectory's full length when only
    its first steps were sampled.  Runs in this process or in a worker of the all-cores pool."""
    from oracle import sq_oracle as O
    with _one_thread():
        t0 = time.perf_counter()
        u = O.UnitCache(task["policy"], task["budget"], task["n_sink"], task["heavy_num"], task["heavy_den"])
        u.prefill(task["k"], task["v"], task["q"])
        t1 = time.perf_counter()
        for (q, kn, vn) in task["steps"]:
            u.decode_step(q, kn, vn)
        t2 = time.perf_counter()
        return (t1 - t0) + (t2 - t1) * task.get("steps_scale", 1.0)


def oracle_importance_task(task):
    from oracle import sq_oracle as O
    with _one_thread():
        t0 = time.perf_counter()
        c = O.layer_importance(task["a"], task["b"])
        return time.perf_counter() - t0, c


def oracle_tasks(w, n_units, n_imp_tokens, seed, device, max_steps=None):
    """Draws a bounded sample of the workload for the oracle: importance chunks (a few layers,
    n_imp_tokens tokens in all) and n_units (layer, sequence, KV head) units with their decode
    steps: all of them, or the first max_steps when every sampled cache already holds its budget
    after the prompt (a decode step then costs the same all along, and the unit's decode time is
    scaled to the full trajectory).  Returns (importance tasks, unit tasks, budgets, steps sampled)."""
    import torch
    from oracle import sq_oracle as O
    from paper_2404_04793_b200 import synth
    rng = np.random.default_rng(seed)
    f64 = lambda t: t.detach().to("cpu").to(torch.float64).numpy()
    layers_imp = list(range(0, w.n_layer, max(1, w.n_layer // 4)))[:4]
    per_layer = max(1, n_imp_tokens // len(layers_imp))
    imp = []
    for l in layers_imp:
        a, b = synth.hidden_pair(w, l, device, batch=1, n_tok=min(per_layer, w.prompt))
        imp.append({"layer": l, "a": f64(a[0]), "b": f64(b[0])})
    # budgets from the generator's target similarities (the sampled layers are re-measured by the oracle)
    cos = np.array(synth.cos_targets(w.n_layer), dtype=np.float32)
    budgets, is_g3 = O.allocate_budgets(cos, w.b_init, w.p)
    # sampled layers: spread evenly within each budget class (the least important group / the rest)
    classes = [[l for l in range(w.n_layer) if bool(is_g3[l]) == c] for c in (False, True)]
    classes = [c for c in classes if c]
    per_class = -(-min(n_units, w.n_layer) // len(classes))
    layers = set()
    for members in classes:
        for i in np.linspace(0, len(members) - 1, min(per_class, len(members))).round():
            layers.add(members[int(i)])
    layers = sorted(layers)
    per = max(1, n_units // len(layers))
    g = w.group
    units = []
    for l in layers:
        q, k, v = synth.prompt_qkv(w, l, device, need_q=(w.policy == synth.H2O))
        for _ in range(per):
            s, h = int(rng.integers(w.batch)), int(rng.integers(w.n_kv_head))
            units.append({"layer": l, "seq": s, "head": h, "policy": w.policy, "budget": int(budgets[l]),
                          "n_sink": w.n_sink, "heavy_num": w.heavy_num, "heavy_den": w.heavy_den, "k": f64(k[s, h]),
                          "v": f64(v[s, h]), "q": None if q is None else f64(q[s, h * g:(h + 1) * g]), "steps": []})
        del q, k, v
    n_steps = w.steps
    if max_steps and max_steps < w.steps and all(u["budget"] <= w.prompt for u in units):
        n_steps = max_steps
    for t in range(n_steps):
        dq, dk, dv = synth.decode_qkv(w, t, device)
        for u in units:
            l, s, h = u["layer"], u["seq"], u["head"]
            u["steps"].append((f64(dq[l, s, h * g:(h + 1) * g]), f64(dk[l, s, h]), f64(dv[l, s, h])))
        del dq, dk, dv
    for u in units:
        u["steps_scale"] = w.steps / n_steps
    return imp, units, budgets, n_steps


def extrapolate(w, budgets, imp_s_per_token, alloc_s, unit_s_by_layer):
    """Whole-job seconds from the sampled costs: importance per token; a unit costs what the
    sampled layer with the nearest budget (then the nearest index) costs."""
    layers = sorted(unit_s_by_layer)

    def unit_cost(l):
        return unit_s_by_layer[min(layers, key=lambda x: (abs(int(budgets[x]) - int(budgets[l])), abs(x - l)))]

    return imp_s_per_token * (w.n_layer * w.batch * w.prompt) + alloc_s \
        + sum(unit_cost(l) * w.batch * w.n_kv_head for l in range(w.n_layer))


def oracle_sample(w, n_units, n_imp_tokens, seed, device, pool_cores=0, max_steps=None):
    """Times the oracle on a bounded sample of the workload and extrapolates linearly to the
    whole job.  One thread in this process; with pool_cores > 1 the same kind of sample, pool_cores
    times as large, is then also run as a plain parallel-for over that many worker processes.
    Returns a dict with tokens/s (one core), seconds spent, a description and, if asked for, the
    all-cores figures."""
    from oracle import sq_oracle as O
    t_start = time.perf_counter()
    n_total = n_units * max(1, pool_cores)
    imp, units, budgets, n_steps = oracle_tasks(w, n_total, n_imp_tokens * max(1, pool_cores), seed, device, max_steps)
    # ---- one core: the first n_units-worth of the sample (spread over the layers) ----
    stride = max(1, len(units) // max(1, n_units))
    mine = units[::stride][:n_units]
    imp_one = imp if pool_cores <= 1 else [{"layer": t["layer"], "a": t["a"][:max(1, len(t["a"]) // pool_cores)],
                                            "b": t["b"][:max(1, len(t["b"]) // pool_cores)]} for t in imp]
    t_imp, n_imp = 0.0, 0
    for t in imp_one:
        s, _ = oracle_importance_task(t)
        t_imp += s
        n_imp += t["a"].shape[0]
    with _one_thread():
        t0 = time.perf_counter()
        O.allocate_budgets(np.array([0.7] * (w.n_layer // 2) + [0.95] * (w.n_layer - w.n_layer // 2), dtype=np.float32),
                           w.b_init, w.p)
        t_alloc = time.perf_counter() - t0
    by_layer = {}
    for t in mine:
        by_layer.setdefault(t["layer"], []).append(oracle_unit_task(t))
    unit_s = {l: sum(v) / len(v) for l, v in by_layer.items()}
    t_job = extrapolate(w, budgets, t_imp / max(n_imp, 1), t_alloc, unit_s)
    total_units = w.n_layer * w.batch * w.n_kv_head
    out = {"value": w.batch * w.steps / t_job, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": (f"{len(mine)} (layer,seq,kv-head) units over {len(unit_s)} layers, "
                      + (f"all {w.steps} decode steps, " if n_steps == w.steps else
                         f"the first {n_steps} of {w.steps} decode steps (full caches: scaled to all steps), ")
                      +
                      f"+ {n_imp} tokens of layer importance + the allocator; extrapolated linearly to "
                      f"{total_units} units and {w.n_layer * w.batch * w.prompt} tokens"),
           "job_seconds_extrapolated": t_job}
    # ---- all cores: a plain parallel-for over independent units (and importance chunks) ----
    if pool_cores > 1:
        import multiprocessing as mp
        ctx = mp.get_context("spawn")          # CUDA may already be initialised in this process: never fork
        with ctx.Pool(pool_cores) as pool:
            pool.map(abs, range(pool_cores))   # workers up and imported before the clock starts
            t0 = time.perf_counter()
            r_imp = pool.map(oracle_importance_task, [{"layer": t["layer"], "a": c_a, "b": c_b} for t in imp
                                                      for c_a, c_b in zip(np.array_split(t["a"], pool_cores),
                                                                          np.array_split(t["b"], pool_cores)) if len(c_a)])
            wall_imp = time.perf_counter() - t0
            t0 = time.perf_counter()
            r_units = pool.map(oracle_unit_task, units, chunksize=1)
            wall_units = time.perf_counter() - t0
        n_imp_all = sum(t["a"].shape[0] for t in imp)
        # wall time per unit of work under the parallel-for, weighted like the one-core figure
        cpu_by_layer = {}
        for t, s in zip(units, r_units):
            cpu_by_layer.setdefault(t["layer"], []).append(s)
        speedup_units = sum(r_units) / wall_units
        unit_wall = {l: (sum(v) / len(v)) / speedup_units for l, v in cpu_by_layer.items()}
        t_job_all = extrapolate(w, budgets, wall_imp / max(n_imp_all, 1), t_alloc, unit_wall)
        out["all_cores"] = {"value": w.batch * w.steps / t_job_all, "unit": UNIT, "cores": pool_cores,
                            "sample": f"{len(units)} units and {n_imp_all} importance tokens as a parallel-for over "
                                      f"{pool_cores} worker processes (one thread each); extrapolated the same way",
                            "parallel_speedup_on_units": speedup_units}
    out["seconds"] = time.perf_counter() - t_start
    return out


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, w):
    import torch
    from paper_2404_04793_b200 import dist_util
    rank, local_rank, world = dist_util.world()
    if rank != 0:
        return
    device = "cuda:0" if torch.cuda.is_available() else "cpu"
    vals, secs = [], []
    desc = ""
    for i in range(args.warmup + args.steps):
        # a quarter of the trajectory per sample keeps the default --steps 5 --warmup 3 run near two minutes
        r = oracle_sample(w, n_units=2, n_imp_tokens=2048, seed=100 + i, device=device, max_steps=max(8, w.steps // 4))
        if i >= args.warmup:
            vals.append(r["value"]); secs.append(r["seconds"])
        desc = r["sample"]
    value = len(vals) / sum(1.0 / v for v in vals)      # steps / total extrapolated time
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.batch * w.steps / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc + " (per step)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "sample_seconds_per_step": statistics.mean(secs),
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ our arm
def hbm_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def decode_kernel_of(w, min_budget=None, per_layer=True):
    """The attention kernel that serves the decode launches of a workload (the library picks by
    shape; for wide groups also by launch size: long units that do not fill the CTA slots take
    the even-deal form, the rule of k_decode_tc_stream.cu restated here for the label)."""
    import torch
    g = w.group
    if w.dtype == torch.bfloat16 and w.head_dim == 64 and g > 32:
        units = w.batch * w.n_kv_head * (1 if per_layer else w.n_layer)
        slots = 2 * torch.cuda.get_device_properties(0).multi_processor_count
        tiles = -(-min(min_budget or w.b_init, w.prompt + 1) // 128)
        if slots <= 2 * units < 4 * slots and tiles >= 16:
            return "decode_attn_tc_stream_kernel"
        return "decode_attn_tc_kernel"
    if w.dtype == torch.bfloat16 and g > 1:
        return "decode_attn_mma_kernel"
    return "decode_attn_kernel"


def algorithmic_bytes_per_step(w, kv_bytes):
    """Bytes one decode step over all layers has to move: K and V of the kept tokens (kv_bytes,
    from the library's own count at the current fill level), q and out, the new token's k and v,
    and for H2O the fp32 score of every kept token read and written."""
    from paper_2404_04793_b200 import synth
    e = w.dtype.itemsize
    d, L, B = w.head_dim, w.n_layer, w.batch
    small = B * L * (w.n_q_head * d * e * 2 + w.n_kv_head * 2 * d * e)
    acc = (kv_bytes // (2 * d * e)) * 8 if w.policy == synth.H2O else 0
    return kv_bytes + small + acc


def hidden_seqs_for(w, budget_bytes=40e9):
    """Distinct sequences of hidden states kept per layer: the most that fit budget_bytes."""
    per_seq = 2 * w.prompt * w.hidden * w.dtype.itemsize * w.n_layer
    best = 1
    for s in range(1, w.batch + 1):
        if w.batch % s == 0 and s * per_seq <= budget_bytes:
            best = s
    return best


def time_replays(job, inp, graph, n, ev, refill=True):
    """Mean milliseconds of n graph replays, each (with refill) after a fresh prefill of the cache."""
    import torch
    tot = 0.0
    for _ in range(n):
        if refill:
            job.prefill(inp)
        a, b = ev(), ev()
        a.record()
        graph.replay()
        b.record()
        torch.cuda.synchronize()
        tot += a.elapsed_time(b)
    return tot / n


def decode_record(w, dev, peak, n_steps=8, reps=3, standin_scores=False, advance=0):
    """Decode-step timing of one configuration: the cache is filled through the library
    (importance, allocation, prefill compression; outside the timed region), then n_steps decode
    steps are replayed from CUDA graphs, as one launch per layer and as one fused launch.
    advance: decode steps run first (cycling through the n_steps inputs), for configurations whose
    caches only reach their budgets during generation; the replays then continue from that state."""
    import torch
    from paper_2404_04793_b200 import engine, synth
    wr = w.replace(steps=n_steps)
    inp = engine.ResidentInputs(wr, dev, hidden_seqs=1, standin_scores=standin_scores)
    # the context must admit every step issued here: the advance and the steps of both captures
    job = engine.Job(w.replace(steps=advance + 4 * n_steps), dev, keep_steps=n_steps)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    job.prefill(inp)
    for t in range(advance):
        job.ctx.decode_step(0, wr.n_layer, inp.q[t % n_steps], inp.k_new[t % n_steps], inp.v_new[t % n_steps],
                            job.out[t % n_steps])
    kv = job.ctx.kv_bytes_per_step(0, wr.n_layer)
    alg = algorithmic_bytes_per_step(wr, kv)
    budgets, is_g3 = job.ctx.get_budgets()
    rec = {"workload": w.name, "policy": synth.POLICY_NAMES[w.policy], "batch": w.batch, "prompt": w.prompt,
           "b_init": w.b_init, "budgets_min_max": [min(budgets), max(budgets)], "kernel": {"per_layer": decode_kernel_of(w, min(budgets), True), "fused": decode_kernel_of(w, min(budgets), False)},
           "algorithmic_bytes_per_step": alg, "steps_timed": n_steps * reps,
           "prompt_scores": "stand-in (scoring pass skipped while filling the cache)" if standin_scores else "computed"}
    if advance:
        rec["steps_before_timing"] = advance
    for form, per_layer in (("per_layer", True), ("fused", False)):
        if not advance:
            job.prefill(inp)
        graph = job.capture_decode(inp, per_layer=per_layer, steps=n_steps)
        time_replays(job, inp, graph, 1, ev, refill=not advance)
        ms = time_replays(job, inp, graph, reps, ev, refill=not advance) / n_steps
        gbs = alg / (ms * 1e-3) / 1e9
        rec[form] = {"ms_per_step": ms, "gbs": gbs, "frac": gbs / peak, "frac_of_nominal_8000": gbs / 8000.0,
                     "tokens_per_s": w.batch / (ms * 1e-3)}
        if gbs > peak:
            rec[form]["note"] = "above the measured peak, which is a copy (read + write): it understates what a read-mostly kernel can reach"
        del graph
    rec["device_status"] = job.ctx.status()
    job.ctx.close()
    del job, inp
    torch.cuda.empty_cache()
    return rec


def whole_pass_record(w, dev, peak, reps=3):
    """Whole pass (importance, allocation, prefill compression, all decode steps as per-layer
    launches from a CUDA graph) of a configuration small enough to keep every input resident."""
    import torch
    from paper_2404_04793_b200 import engine, synth
    inp = engine.ResidentInputs(w, dev)
    job = engine.Job(w, dev, per_layer_decode=True, keep_steps=min(w.steps, 16))
    ev = lambda: torch.cuda.Event(enable_timing=True)
    job.prefill(inp)
    graph = job.capture_decode(inp, per_layer=True)
    job.prefill(inp); graph.replay()
    torch.cuda.synchronize()
    a, b = ev(), ev()
    a.record()
    for _ in range(reps):
        job.prefill(inp)
        graph.replay()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    ms_dec = time_replays(job, inp, graph, reps, ev)
    kv = job.ctx.kv_bytes_per_step(0, w.n_layer)       # after the captured steps: the steady state
    alg = algorithmic_bytes_per_step(w, kv)
    gbs = alg * w.steps / (ms_dec * 1e-3) / 1e9
    rec = {"workload": w.name, "policy": synth.POLICY_NAMES[w.policy], "ms_per_pass": ms,
           "tokens_per_s": w.batch * w.steps / (ms * 1e-3), "decode_ms_per_step": ms_dec / w.steps,
           "decode_gbs": gbs, "decode_frac": gbs / peak, "decode_launch": "per_layer (CUDA-graph replay)",
           "device_status": job.ctx.status()}
    del graph
    job.ctx.close()
    del job, inp
    torch.cuda.empty_cache()
    return rec


def host_memory_available():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def run_ours(args, w):
    import torch
    from paper_2404_04793_b200 import dist_util, engine, synth
    rank, local_rank, world = dist_util.init("nccl")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    peak, peak_kind = hbm_peak()
    # every rank owns an independent batch (a different seed family per rank); with --shard-batch
    # the ranks hold the sequences of ONE batch, B / world each, and exchange the layer sums of the
    # importance pass before the allocation, so that all of them get the batch's budgets
    wr = w.replace(wid=w.wid + 100 * rank) if world > 1 else w
    exchange = None
    if args.shard_batch:
        if w.batch % world:
            raise SystemExit("--shard-batch needs a batch divisible by the number of ranks")
        wr = wr.replace(batch=w.batch // world)
        exchange = lambda ctx: dist_util.exchange_importance(ctx, dev)
    hs = hidden_seqs_for(wr)
    inp = engine.ResidentInputs(wr, dev, hidden_seqs=hs)
    job = engine.Job(wr, dev, per_layer_decode=True, keep_steps=min(wr.steps, 16), exchange=exchange)
    tokens = wr.batch * wr.steps
    ev = lambda: torch.cuda.Event(enable_timing=True)

    # ---- warm-up: whole passes with plain calls, then the decode steps captured once per form ----
    job.run(inp)
    job.prefill(inp)
    graph_pl = job.capture_decode(inp, per_layer=True)
    for _ in range(max(0, args.warmup - 1)):
        job.prefill(inp)
        graph_pl.replay()
    torch.cuda.synchronize()
    budgets, is_g3 = job.ctx.get_budgets()
    kv_bytes = job.ctx.kv_bytes_per_step(0, wr.n_layer)     # steady state: every layer at its budget
    alg_bytes = algorithmic_bytes_per_step(wr, kv_bytes)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        job.prefill(inp); graph_pl.replay()                  # keeps the GPU busy while the sampler starts up
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
        graph_pl.replay()
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
    del graph_pl

    # ---- the same decode steps as one fused launch over all layers (upper bound) ----
    fused = None
    if not args.no_fused:
        job.prefill(inp)
        graph_f = job.capture_decode(inp, per_layer=False)
        time_replays(job, inp, graph_f, 1, ev)
        ms_f = time_replays(job, inp, graph_f, max(1, min(args.steps, 3)), ev)
        fused = {"mode": "one launch per decode step over all layers (needs every layer's q at once: an upper "
                         "bound, not a form a model can issue)",
                 "decode_tokens_per_s": tokens / (ms_f * 1e-3), "ms_per_token_step": ms_f / wr.steps,
                 "hbm_gbs": alg_bytes * wr.steps / (ms_f * 1e-3) / 1e9,
                 "hbm_frac": alg_bytes * wr.steps / (ms_f * 1e-3) / 1e9 / peak}
        del graph_f

    # ---- end to end: the same pass fed from page-locked host memory, outputs copied back ----
    e2e = None
    if not args.no_e2e:
        # what the host holds is sized to its memory (at most 32 GB page-locked): fewer distinct
        # hidden-state sequences and prompt layers than the device-resident run keeps, if need be.
        # Layer l then sends the prompt tensors of layer l % n, so the bytes per pass stay the same.
        avail = host_memory_available() or 64e9
        host_budget = min(0.3 * avail / max(1, world), 32e9)
        hs_host = hidden_seqs_for(wr, 0.4 * host_budget)
        per_layer_prompt = (inp.bytes_per_pass() - 2 * sum(a.numel() * a.element_size() for a, _ in inp.hidden)
                            - inp.q.numel() * inp.q.element_size()) / wr.n_layer
        n_pl = wr.n_layer
        while n_pl > 1 and per_layer_prompt * n_pl > 0.4 * host_budget:
            n_pl //= 2
        host = engine.ResidentInputs(wr, "cpu", gen_device=dev, hidden_seqs=hs_host, prompt_layers=n_pl)
        out_host = torch.empty((2,) + tuple(job.out.shape[1:]), dtype=job.out.dtype, pin_memory=True)
        job.run_from_host(host, out_host)
        torch.cuda.synchronize()
        dist_util.barrier()
        s0, s1 = ev(), ev()
        n_e2e = max(1, min(args.steps, 2))
        s0.record()
        for _ in range(n_e2e):
            job.run_from_host(host, out_host)
        s1.record()
        torch.cuda.synchronize()
        dist_util.barrier()
        e2e_val, _ = dist_util.aggregate_throughput(tokens, s0.elapsed_time(s1) / n_e2e, dev)
        e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": host.bytes_per_pass(),
               "d2h_bytes_per_step": wr.steps * out_host[0].numel() * out_host.element_size(), "steps": n_e2e,
               "host_distinct_prompt_layers": n_pl, "host_hidden_sequences_per_layer": hs_host,
               "note": "per pass every distinct input tensor crosses PCIe once (a layer's hidden-state chunk is "
                       "then read hidden_repeat times on the device) and every step's output is copied back"}
        del host, out_host

    launches = job.kernel_launches_per_pass(inp, per_layer_decode=True) * args.steps
    hidden_repeat = inp.hidden_repeat
    job.ctx.close()
    del job, inp
    torch.cuda.empty_cache()
    if rank != 0:
        dist_util.shutdown()
        return

    # ---- roofline of the dominant kernel: the per-layer decode launch ----
    kernel = decode_kernel_of(wr, min(budgets))
    n_launch = wr.steps * wr.n_layer
    sec_per_launch = ms_decode * 1e-3 / n_launch
    bytes_per_launch = alg_bytes / wr.n_layer
    achieved = bytes_per_launch / sec_per_launch / 1e9
    ratio = NCU_TRAFFIC_PER_ALGORITHMIC_BYTE.get(kernel)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None if ratio is None else ratio * bytes_per_launch, "peak_kind": peak_kind,
                "kernel": kernel, "launch": "one per layer per decode step (average over the layers' budgets)",
                "algorithmic_bytes_per_launch": bytes_per_launch, "us_per_launch": sec_per_launch * 1e6,
                "frac_of_nominal_8000": achieved / 8000.0,
                "peak_note": "the measured peak is a copy (read + write); a read-mostly kernel can exceed it slightly (the wide-group kernel's tile loads alone, with no arithmetic, stream 7.3 TB/s on this pool)"}

    records, whole_pass = None, None
    if world == 1 and not args.no_records:
        records = []
        long_gen = synth.mistral_7b_long_generation(batch=224)
        for wl, standin, advance in ((synth.mistral_7b(), False, 0), (synth.llama2_70b(), False, 0),
                                     (synth.falcon_7b_max(synth.SLIDING_WINDOW), False, 0),
                                     (synth.falcon_7b_max(synth.H2O), True, 0),
                                     # budgets in absolute tokens above the prompt length: timed once the
                                     # caches have grown to their budgets
                                     (long_gen, False, 700)):
            if wl.name == wr.name and fused is not None:
                continue                                      # the headline itself: already in the line
            records.append(decode_record(wl, dev, peak, standin_scores=standin, advance=advance))
        if wr.name != synth.llama2_7b().name:
            whole_pass = whole_pass_record(synth.llama2_7b(), dev, peak)

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cores = min(host_cores(), 32)
        cpu = oracle_sample(wr, n_units=args.cpu_units, n_imp_tokens=16384, seed=7, device=dev,
                            pool_cores=cores if cores > 1 else 0)

    cfg = config_of(wr, world, args.shard_batch)
    cfg.update({"budgets_min_max": [min(budgets), max(budgets)], "n_g3": int(sum(is_g3)),
                "decode_launch": "per_layer (one launch per layer per step, CUDA-graph replay)",
                "hidden_states": f"{hs} distinct sequences per layer, fed {hidden_repeat}x (every token's bytes are read)",
                "l2": "inputs larger than L2 (K/V read per decode step %.2f GB, %.0f MB per launch)"
                      % (kv_bytes / 1e9, kv_bytes / wr.n_layer / 1e6)})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_max, "higher_is_better": True, "scaling": "strong" if args.shard_batch else "weak", "vs_baseline": None,
        "dtype": "bf16" if wr.dtype == torch.bfloat16 else "f32", "data": "synthetic", "config": cfg,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
        "decode_only": {"tokens_per_s": tokens / (ms_decode * 1e-3), "ms_per_token_step": ms_decode / wr.steps,
                        "prefill_ms": ms_step - ms_decode, "hbm_gbs": alg_bytes * wr.steps / (ms_decode * 1e-3) / 1e9,
                        "hbm_frac": alg_bytes * wr.steps / (ms_decode * 1e-3) / 1e9 / peak},
        "fused_launch_upper_bound": fused, "decode_records": records, "whole_pass_llama2_7b": whole_pass,
        "device_status": status,
    }
    print(json.dumps(line), flush=True)
    dist_util.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps")
    ap.add_argument("--cpu-units", type=int, default=4, help="units the one-core oracle timing samples")
    ap.add_argument("--shard-batch", action="store_true",
                    help="--gpus N: one batch of the workload's size sharded over the ranks (strong scaling) instead of one batch per rank")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-fused", action="store_true", help="skip the fused-launch upper bound")
    ap.add_argument("--no-records", action="store_true", help="skip the decode-step records of the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "ours" and args.gpus > 1 and "RANK" not in os.environ:
        import torch
        if torch.cuda.device_count() < args.gpus:
            print(f"bench.py: --gpus {args.gpus} needs {args.gpus} CUDA devices, found {torch.cuda.device_count()}",
                  file=sys.stderr)
            sys.exit(2)
    rc = maybe_spawn(sys.argv[1:], args.gpus)
    if rc is not None:
        sys.exit(rc)
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
