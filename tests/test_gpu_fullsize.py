"""Parity at the full sizes of the paper-shaped workloads (one fused decode launch per step over
all layers): sampled (layer, sequence, KV head) units are followed by the oracle through every
step -- free-running where the kept sets are integer logic, in lockstep on the library's own
score bits for H2O.  Units are independent, so a sample that always
holds the first and last unit and every layer of one sequence covers the layout arithmetic."""
import numpy as np
import pytest
import torch

from oracle import sq_oracle as O
from paper_2404_04793_b200 import engine, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _prefill_full_size(w, n_units, seed, oracle_prefill, every_layer=True):
    """Importance, allocation and prefill compression of the whole workload through the C ABI
    (budgets checked against the oracle).  Returns the context, the budgets, the sampled units
    and, per sampled unit, its prompt rows (K, V as fp64 [P, d]) and, with oracle_prefill, an
    oracle cache that has taken the same prompt."""
    ctx = engine.context_for(w, DEV)
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
    units = H.sample_units(w, n_units, seed, every_layer)
    by_layer = {}
    for u in units:
        by_layer.setdefault(u[0], []).append(u)
    g = w.group
    rows, oracles = {}, {}
    for l in range(w.n_layer):
        q, k, v = synth.prompt_qkv(w, l, DEV, need_q=(w.policy == synth.H2O))
        ctx.prefill_compress(l, k, v, q)
        for (_, s, h) in by_layer.get(l, []):
            rows[(l, s, h)] = (H.f64(k[s, h]), H.f64(v[s, h]))
            if oracle_prefill:
                u = O.UnitCache(w.policy, budgets[l], w.n_sink, w.heavy_num, w.heavy_den)
                u.prefill(*rows[(l, s, h)], None if q is None else H.f64(q[s, h * g:(h + 1) * g]))
                oracles[(l, s, h)] = u
        del q, k, v
    return ctx, budgets, units, rows, oracles


def _follow(w, n_units, steps, seed=0, every_layer=True):
    """Free-running: the oracle takes the same inputs from the prompt on and never sees the
    library's state.  Kept sets must be identical (Sliding Window / StreamingLLM: integer logic,
    any number of steps; H2O: while no two scores tie to fp32 accuracy, hence first steps only)."""
    w = w.replace(steps=steps)
    ctx, budgets, units, rows, oracles = _prefill_full_size(w, n_units, seed, True, every_layer)
    g = w.group
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


def _lockstep(w, n_units, steps, seed=0, every_layer=True, check_rows_every=32):
    """H2O at scale, every step: before a step the library's state of each sampled unit (kept
    positions and the bits of their scores) is read back; the oracle's C_seq and attention run on
    exactly those bits for that one step; the library's kept set after the step must be
    identical, its outputs within the output tolerance and its new scores within the score
    tolerance.  No near tie can excuse a difference, because both sides rank the same bits.
    The cached K/V rows are compared bit for bit with the rows those positions came from."""
    w = w.replace(steps=steps)
    ctx, budgets, units, rows, _ = _prefill_full_size(w, n_units, seed, False, every_layer)
    g, P = w.group, w.prompt
    new_rows = {key: ([], []) for key in units}            # K, V rows appended by the decode steps

    def row_of(key, which, p):
        return rows[key][which][p] if p < P else new_rows[key][which][p - P]

    state = {key: ctx.get_kept(*key) for key in units}
    for key, (pos, acc) in state.items():
        assert len(pos) == min(P, budgets[key[0]]) and np.isfinite(acc).all(), key
    worst = 0.0
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        for key in units:
            l, s, h = key
            new_rows[key][0].append(H.f64(kn[l, s, h]))
            new_rows[key][1].append(H.f64(vn[l, s, h]))
            pos, acc = state[key]
            u = O.UnitCache(w.policy, budgets[l], w.n_sink, w.heavy_num, w.heavy_den)
            u.pos, u.acc = list(pos), [float(a) for a in acc]
            u.K = [row_of(key, 0, p) for p in pos]
            u.V = [row_of(key, 1, p) for p in pos]
            u.next_pos = P + t
            want = u.decode_step(H.f64(q[l, s, h * g:(h + 1) * g]), new_rows[key][0][-1], new_rows[key][1][-1])
            got_pos, got_acc = ctx.get_kept(*key)
            assert got_pos == u.kept_positions(), (t, key)
            err = float(np.max(np.abs(H.f64(out[l, s, h * g:(h + 1) * g]) - want)))
            worst = max(worst, err)
            assert err <= H.TOL_OUT[w.dtype], (t, key, err)
            assert np.allclose(got_acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), (t, key)
            if t % check_rows_every == 0 or t == w.steps - 1:
                kk, vv = ctx.get_kv(*key)
                assert np.array_equal(H.f64(kk), np.stack([row_of(key, 0, p) for p in got_pos])), (t, key)
                assert np.array_equal(H.f64(vv), np.stack([row_of(key, 1, p) for p in got_pos])), (t, key)
            state[key] = (got_pos, got_acc)
    assert ctx.status() == 0
    return worst


def test_llama2_7b_sliding_window_full_size():
    # all 128 decode steps
    _follow(synth.llama2_7b(), n_units=48, steps=128)


def test_llama2_70b_streaming_full_size_all_steps():
    _follow(synth.llama2_70b(), n_units=84, steps=128)


def test_mistral_7b_h2o_full_size_first_steps_free_running():
    _follow(synth.mistral_7b(), n_units=40, steps=6)


def test_mistral_7b_h2o_full_size_lockstep_all_steps():
    # every one of the 256 steps, well past the point where the recent window has turned over
    _lockstep(synth.mistral_7b(), n_units=36, steps=256)


def test_falcon_7b_h2o_cell_lockstep_all_steps():
    # batch 32, prompt 8192, budget 50 %: 1.07 GB of K/V per decode step, all 128 steps
    _lockstep(synth.falcon_7b(32, 8192, 50.0, synth.H2O), n_units=16, steps=128, every_layer=False)


def test_mistral_7b_absolute_budget_generation_longer_than_prompt():
    """Budgets in absolute tokens above the prompt length (600 per layer for a 512-token prompt)
    and 1024 generated tokens: the important layers' caches grow for hundreds of steps, reach
    their budgets and evict from then on; the oracle follows every one of the 1024 steps."""
    w = synth.mistral_7b_long_generation(batch=32)
    assert w.b_init == 600 > w.prompt and w.steps == 1024
    _follow(w, n_units=10, steps=w.steps, every_layer=False)


def test_falcon_7b_mqa_cells():
    for policy, batch, prompt, pct in [(synth.SLIDING_WINDOW, 32, 2048, 20.0), (synth.STREAMING_LLM, 8, 8192, 10.0),
                                       (synth.H2O, 2, 2048, 30.0)]:
        _follow(synth.falcon_7b(batch, prompt, pct, policy), n_units=34, steps=4)


def test_falcon_7b_largest_cell_all_steps():
    # the largest cell of the sweep: batch 224, prompt 16384, budget 50 % (15 GB of K/V per step)
    _follow(synth.falcon_7b(224, 16384, 50.0, synth.SLIDING_WINDOW), n_units=10, steps=128, every_layer=False)


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
