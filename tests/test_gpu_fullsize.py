"""Parity at the full sizes of the paper-shaped workloads, in the launch configuration bench.py times (one fused
decode launch per step over all layers): sampled (layer, sequence, KV head) units are
followed by the oracle through every step.  Units are independent, so a sample that always
holds the first and last unit and every layer of one sequence covers the layout arithmetic."""
import numpy as np
import pytest
import torch

from oracle import sq_oracle as O
from paper_2404_04793_b200 import engine, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _follow(w, n_units, steps, seed=0):
    w = w.replace(steps=steps)
    job = engine.Job(w, DEV)
    ctx = job.ctx
    ctx.begin_sequence_batch(w.batch, w.prompt)
    # hidden states are drawn and fed in pieces of at most 2^29 elements
    seq_per_piece = max(1, min(w.batch, (1 << 29) // (w.prompt * w.hidden)))
    for l in range(w.n_layer):
        for ci, s0 in enumerate(range(0, w.batch, seq_per_piece)):
            a, b = synth.hidden_pair(w, l, DEV, batch=min(seq_per_piece, w.batch - s0), chunk=ci)
            ctx.layer_importance(l, a, b)
            del a, b
    ctx.allocate_budgets(w.b_init, w.p)
    cos = ctx.get_cos_sim().numpy()
    targets = np.array(synth.cos_targets(w.n_layer))
    assert np.max(np.abs(cos - targets)) < 5e-3            # statistical limit of the generator
    budgets, is_g3 = ctx.get_budgets()
    wb, wg = O.allocate_budgets(cos, w.b_init, w.p)
    assert budgets == wb.tolist() and is_g3 == wg.tolist()
    assert sum(budgets) == w.n_layer * w.b_init
    units = H.sample_units(w, n_units, seed)
    by_layer = {}
    for u in units:
        by_layer.setdefault(u[0], []).append(u)
    g = w.group
    oracles = {}
    for l in range(w.n_layer):
        q, k, v = synth.prompt_qkv(w, l, DEV, need_q=(w.policy == synth.H2O))
        ctx.prefill_compress(l, k, v, q)
        for (_, s, h) in by_layer.get(l, []):
            u = O.UnitCache(w.policy, budgets[l], w.n_sink, w.heavy_num, w.heavy_den)
            u.prefill(H.f64(k[s, h]), H.f64(v[s, h]), None if q is None else H.f64(q[s, h * g:(h + 1) * g]))
            oracles[(l, s, h)] = u
        del q, k, v
    for key, u in oracles.items():
        pos, acc = ctx.get_kept(*key)
        assert pos == u.kept_positions(), key
    worst = 0.0
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        for (l, s, h), u in oracles.items():
            want = u.decode_step(H.f64(q[l, s, h * g:(h + 1) * g]), H.f64(kn[l, s, h]), H.f64(vn[l, s, h]))
            err = float(np.max(np.abs(H.f64(out[l, s, h * g:(h + 1) * g]) - want)))
            worst = max(worst, err)
            assert err <= H.TOL_OUT[w.dtype], (t, l, s, h, err)
    for key, u in oracles.items():
        pos, acc = ctx.get_kept(*key)
        assert pos == u.kept_positions(), key
        if w.policy == synth.H2O:
            assert np.allclose(acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), key
    assert ctx.status() == 0
    return worst


def test_llama2_7b_sliding_window_full_size():
    # the configuration the benchmark times: all 128 decode steps
    _follow(synth.llama2_7b(), n_units=48, steps=128)


def test_llama2_70b_streaming_full_size_first_steps():
    _follow(synth.llama2_70b(), n_units=90, steps=6)


def test_mistral_7b_h2o_full_size_first_steps():
    _follow(synth.mistral_7b(), n_units=40, steps=6)


def test_falcon_7b_mqa_cells():
    for policy, batch, prompt, pct in [(synth.SLIDING_WINDOW, 32, 2048, 20.0), (synth.STREAMING_LLM, 8, 8192, 10.0),
                                       (synth.H2O, 2, 2048, 30.0)]:
        _follow(synth.falcon_7b(batch, prompt, pct, policy), n_units=34, steps=4)


def test_falcon_7b_largest_cell_sampled():
    # the largest cell of the sweep: batch 224, prompt 16384, budget 50 % (15 GB of K/V per step)
    _follow(synth.falcon_7b(224, 16384, 50.0, synth.SLIDING_WINDOW), n_units=36, steps=2)


def test_llama2_7b_per_sequence_budgets_full_size():
    """The benchmark shape with one budget vector per sequence (the batch's vector rotated by one
    layer per sequence, so every sequence differs and every vector sums to n_layer * b_init)."""
    w = synth.llama2_7b().replace(steps=8)
    base, _ = O.allocate_budgets(np.array(synth.cos_targets(w.n_layer), dtype=np.float32), w.b_init, w.p)
    base = base.tolist()
    rows = [base[s:] + base[:s] for s in range(w.batch)]
    ctx = engine.context_for(w, DEV, per_sequence_budgets=1)
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets(rows)
    assert ctx.get_budgets()[0] == rows
    units = H.sample_units(w, 40, seed=3)
    by_layer = {}
    for u in units:
        by_layer.setdefault(u[0], []).append(u)
    oracles = {}
    for l in range(w.n_layer):
        _, k, v = synth.prompt_qkv(w, l, DEV, need_q=False)
        ctx.prefill_compress(l, k, v)
        for (_, s, h) in by_layer.get(l, []):
            u = O.UnitCache(w.policy, rows[s][l], w.n_sink, w.heavy_num, w.heavy_den)
            u.prefill(H.f64(k[s, h]), H.f64(v[s, h]), None)
            oracles[(l, s, h)] = u
        del k, v
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        for (l, s, h), u in oracles.items():
            want = u.decode_step(H.f64(q[l, s, h:h + 1]), H.f64(kn[l, s, h]), H.f64(vn[l, s, h]))
            assert np.max(np.abs(H.f64(out[l, s, h:h + 1]) - want)) <= H.TOL_OUT[w.dtype], (t, l, s, h)
    for key, u in oracles.items():
        assert ctx.get_kept(*key)[0] == u.kept_positions(), key
    assert ctx.status() == 0
