"""Per-sequence budgets (Section 4.1 allocates for "the given prompt"): every sequence of a
batch is clustered on its own layer averages and gets its own per-layer budgets.  The CUDA
library must then match the oracle run sequence by sequence: cosines within tolerance, budgets
and kept sets identical, outputs within max-abs 1e-5 (fp32) / 1e-2 (bf16)."""
import numpy as np
import pytest
import torch

from oracle import sq_oracle as O
from paper_2404_04793_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _workload(wid, **kw):
    base = dict(n_layer=6, n_q_head=4, n_kv_head=2, head_dim=64, hidden=256, batch=3, prompt=96, steps=5,
                dtype=torch.float32, policy=synth.SLIDING_WINDOW, budget_pct=25.0, p=0.3)
    base.update(kw)
    return synth.Workload("perseq", wid, **base)


def _hidden_per_sequence(w):
    """Hidden states whose layer profile differs per sequence: sequence s takes, for layer l,
    the generator's pair of layer (l + 2 s) mod L, so the clusters fall on different layers."""
    pairs = [synth.hidden_pair(w, l, DEV) for l in range(w.n_layer)]
    out = []
    for l in range(w.n_layer):
        a = torch.stack([pairs[(l + 2 * s) % w.n_layer][0][s] for s in range(w.batch)])
        b = torch.stack([pairs[(l + 2 * s) % w.n_layer][1][s] for s in range(w.batch)])
        out.append((a.contiguous(), b.contiguous()))
    return out


def _allocate(ctx, w, chunks):
    ctx.begin_sequence_batch(w.batch, w.prompt)
    hidden = _hidden_per_sequence(w)
    want_cos = np.zeros((w.batch, w.n_layer))
    for l, (a, b) in enumerate(hidden):
        a2, b2 = a.reshape(-1, w.hidden), b.reshape(-1, w.hidden)
        n = a2.shape[0]
        edges = [round(i * n / chunks) for i in range(chunks + 1)]   # cuts inside sequences on purpose
        for i in range(chunks):
            ctx.layer_importance(l, a2[edges[i]:edges[i + 1]].contiguous(), b2[edges[i]:edges[i + 1]].contiguous())
        for s in range(w.batch):
            want_cos[s, l] = O.layer_importance(H.f64(a[s]), H.f64(b[s]))
    ctx.allocate_budgets(w.b_init, w.p)
    got_cos = ctx.get_cos_sim().numpy().astype(np.float64)
    assert got_cos.shape == (w.batch, w.n_layer)
    assert np.max(np.abs(got_cos - want_cos)) <= H.TOL_OUT[w.dtype]
    budgets, is_g3 = ctx.get_budgets()
    for s in range(w.batch):
        wb, wg = O.allocate_budgets(got_cos[s].astype(np.float32), w.b_init, w.p)
        assert budgets[s] == wb.tolist() and is_g3[s] == wg.tolist(), s
        assert sum(budgets[s]) == w.n_layer * w.b_init
    return budgets


def _decode_and_compare(ctx, w, budgets, per_layer_calls):
    prompt_cpu = H.prefill_all(ctx, w, DEV)
    units = H.all_units(w)
    oracles = {(l, s, h): H.oracle_unit(w, budgets[s], prompt_cpu, l, s, h) for (l, s, h) in units}
    g = w.group
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        if per_layer_calls:
            for l in range(w.n_layer):
                ctx.decode_step(l, l + 1, q[l], kn[l], vn[l], out[l])
        else:
            ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        torch.cuda.synchronize()
        qc, kc, vc, oc = q.cpu(), kn.cpu(), vn.cpu(), out.cpu()
        for (l, s, h) in units:
            u = oracles[(l, s, h)]
            want = u.decode_step(H.f64(qc[l, s, h * g:(h + 1) * g]), H.f64(kc[l, s, h]), H.f64(vc[l, s, h]))
            got = H.f64(oc[l, s, h * g:(h + 1) * g])
            assert float(np.max(np.abs(got - want))) <= H.TOL_OUT[w.dtype], (t, l, s, h)
            pos, acc = ctx.get_kept(l, s, h)
            assert pos == u.kept_positions(), (t, l, s, h)
            if w.policy == synth.H2O:
                assert np.allclose(acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), (t, l, s, h)
    return oracles


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
@pytest.mark.parametrize("dtype,head_dim,hq,hkv", [(torch.float32, 64, 2, 2), (torch.bfloat16, 128, 8, 2),
                                                   (torch.bfloat16, 64, 71, 1)])
def test_budgets_differ_per_sequence_and_decode_matches(policy, dtype, head_dim, hq, hkv):
    w = _workload(41, policy=policy, dtype=dtype, head_dim=head_dim, n_q_head=hq, n_kv_head=hkv,
                  heavy_mode="uniform4", budget_pct=40.0)
    ctx = H.make_ctx(w, per_sequence_budgets=1)
    budgets = _allocate(ctx, w, chunks=4)
    assert any(budgets[s] != budgets[0] for s in range(1, w.batch)), "the sequences should not share a budget vector"
    _decode_and_compare(ctx, w, budgets, per_layer_calls=False)
    assert ctx.status() == 0


def test_per_layer_calls_set_budgets_and_evict():
    w = _workload(42, policy=synth.H2O, dtype=torch.bfloat16, head_dim=128, n_q_head=4, n_kv_head=2, n_layer=3,
                  heavy_mode="uniform4", steps=6)
    budgets = [[40, 12, 30], [9, 55, 18], [101, 24, 33]]       # over budget, tiny, still growing
    ctx = H.make_ctx(w, b_init=max(max(r) for r in budgets), per_sequence_budgets=1)
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets(budgets)
    assert ctx.get_budgets()[0] == budgets
    oracles = _decode_and_compare(ctx, w.replace(steps=3), budgets, per_layer_calls=True)
    new_budgets = [[17, 12, 20], [9, 30, 10], [50, 24, 33]]
    ctx.evict(0, w.n_layer, new_budgets)
    for (l, s, h), u in oracles.items():
        u.b = new_budgets[s][l]
        u._compress()
        pos, _ = ctx.get_kept(l, s, h)
        assert pos == u.kept_positions(), (l, s, h)
        k, _ = ctx.get_kv(l, s, h)
        assert np.array_equal(H.f64(k), np.stack(u.K))
    assert ctx.get_budgets()[0] == new_budgets
    g = w.group
    for t in range(3, w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        qc, kc, vc, oc = q.cpu(), kn.cpu(), vn.cpu(), out.cpu()
        for (l, s, h), u in oracles.items():
            want = u.decode_step(H.f64(qc[l, s, h * g:(h + 1) * g]), H.f64(kc[l, s, h]), H.f64(vc[l, s, h]))
            assert np.max(np.abs(H.f64(oc[l, s, h * g:(h + 1) * g]) - want)) <= H.TOL_OUT[w.dtype]
            assert ctx.get_kept(l, s, h)[0] == u.kept_positions(), (t, l, s, h)
    assert ctx.status() == 0


def test_one_sequence_equals_the_batch_mode():
    """With a single sequence both modes see the same averages: same budgets, same bits out."""
    w = _workload(43, batch=1, dtype=torch.bfloat16, head_dim=128, n_q_head=8, n_kv_head=2, policy=synth.STREAMING_LLM)
    outs = []
    for mode in (0, 1):
        ctx = H.make_ctx(w, per_sequence_budgets=mode)
        H.run_importance_and_allocate(ctx, w, DEV)
        b = ctx.get_budgets()[0]
        outs.append([b[0] if mode else b])
        H.prefill_all(ctx, w, DEV, keep_inputs=False)
        for t in range(w.steps):
            q, kn, vn = synth.decode_qkv(w, t, DEV)
            out = torch.empty_like(q)
            ctx.decode_step(0, w.n_layer, q, kn, vn, out)
            outs[-1].append(out.cpu())
        assert ctx.status() == 0
    assert outs[0][0] == outs[1][0]
    for a, b in zip(outs[0][1:], outs[1][1:]):
        assert torch.equal(a, b)


def test_argument_and_order_errors():
    from paper_2404_04793_b200 import binding as B
    w = _workload(44, n_layer=3)
    ctx = H.make_ctx(w, per_sequence_budgets=1)
    ctx.begin_sequence_batch(w.batch, w.prompt)
    a, b = synth.hidden_pair(w, 0, DEV)
    half = a.reshape(-1, w.hidden)[: w.batch * w.prompt // 2].contiguous()
    for l in range(w.n_layer):
        ctx.layer_importance(l, half, half)
    with pytest.raises(B.SqError) as e:          # half of the prompt tokens are still missing
        ctx.allocate_budgets(w.b_init, w.p)
    assert e.value.code == B.SQ_ERR_STATE
    for l in range(w.n_layer):
        ctx.layer_importance(l, half, half)
    with pytest.raises(B.SqError) as e:          # more rows than batch * prompt_len
        ctx.layer_importance(0, half, half)
    assert e.value.code == B.SQ_ERR_INVALID_ARG
    ctx.allocate_budgets(w.b_init, w.p)
    budgets, _ = ctx.get_budgets()
    assert len(budgets) == w.batch and all(sum(r) == w.n_layer * w.b_init for r in budgets)
    with pytest.raises(ValueError):              # one list per sequence is expected
        ctx.set_budgets([10, 10, 10])
    with pytest.raises(B.SqError) as e:          # a sequence whose budgets do not fit the pool
        ctx.set_budgets([[10 * w.b_init] * w.n_layer] * w.batch)
    assert e.value.code == B.SQ_ERR_CAPACITY
    cfg = B.make_config(n_layer=2, n_q_head=2, n_kv_head=2, head_dim=64, hidden=64, max_batch=1, max_prompt=8,
                        max_new_tokens=1, dtype=torch.float32, policy=synth.SLIDING_WINDOW, per_sequence_budgets=2)
    with pytest.raises(B.SqError) as e:
        B.sq_query_sizes(cfg, 4)
    assert e.value.code == B.SQ_ERR_INVALID_ARG


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.H2O])
@pytest.mark.parametrize("hq,hkv,head_dim", [(8, 2, 128), (71, 1, 64), (2, 2, 128)])
def test_long_contexts_split_across_ctas(policy, hq, hkv, head_dim):
    """Few units with long, unequal budgets: the launch splits each unit's tokens over several
    CTAs, a different number of pieces per sequence."""
    w = _workload(45, policy=policy, dtype=torch.bfloat16, head_dim=head_dim, n_q_head=hq, n_kv_head=hkv, batch=2,
                  n_layer=2, prompt=3000, steps=3, hidden=64, heavy_mode="zipf")
    budgets = [[2500, 300], [700, 2900]]
    ctx = H.make_ctx(w, b_init=2900, per_sequence_budgets=1)
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets(budgets)
    prompt_cpu = H.prefill_all(ctx, w, DEV)
    units = H.all_units(w)
    oracles = {(l, s, h): H.oracle_unit(w, budgets[s], prompt_cpu, l, s, h) for (l, s, h) in units}
    g = w.group
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        if t == 1:   # one step layer by layer
            for l in range(w.n_layer):
                ctx.decode_step(l, l + 1, q[l], kn[l], vn[l], out[l])
        else:
            ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        qc, kc, vc, oc = q.cpu(), kn.cpu(), vn.cpu(), out.cpu()
        for (l, s, h) in units:
            u = oracles[(l, s, h)]
            want = u.decode_step(H.f64(qc[l, s, h * g:(h + 1) * g]), H.f64(kc[l, s, h]), H.f64(vc[l, s, h]))
            assert np.max(np.abs(H.f64(oc[l, s, h * g:(h + 1) * g]) - want)) <= H.TOL_OUT[w.dtype], (t, l, s, h)
    for (l, s, h) in units:
        if policy != synth.H2O:
            assert ctx.get_kept(l, s, h)[0] == oracles[(l, s, h)].kept_positions(), (l, s, h)
    assert ctx.status() == 0
