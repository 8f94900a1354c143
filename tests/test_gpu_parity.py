"""Parity of the CUDA library (through the C ABI) against the CPU oracle on the same seeded
inputs.  Budgets and kept-token sets must be identical; attention outputs and cosine
similarities within max-abs 1e-5 (fp32 inputs) / 1e-2 (bf16 inputs)."""
import math

import numpy as np
import pytest
import torch

from oracle import sq_oracle as O
from paper_2404_04793_b200 import binding as B
from paper_2404_04793_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def small(name, wid, **kw):
    base = dict(n_layer=3, n_q_head=4, n_kv_head=2, head_dim=64, hidden=256, batch=2, prompt=96, steps=6,
                dtype=torch.float32, policy=synth.SLIDING_WINDOW, budget_pct=25.0, p=0.3)
    base.update(kw)
    return synth.Workload(name, wid, **base)


# ------------------------------------------------------------------ importance
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("hidden,batch,prompt,chunks", [(128, 1, 256, 1), (4096, 2, 301, 3), (4544, 3, 67, 2)])
def test_layer_importance_matches_oracle(dtype, hidden, batch, prompt, chunks):
    w = small("imp", 11, n_layer=4, hidden=hidden, batch=batch, prompt=prompt, dtype=dtype)
    ctx = H.make_ctx(w)
    want = H.run_importance_and_allocate(ctx, w, DEV, chunks)
    got = ctx.get_cos_sim().numpy().astype(np.float64)
    assert np.max(np.abs(got - want)) <= H.TOL_OUT[dtype]
    assert ctx.status() == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("hidden,batch,prompt,chunks,in_place", [(128, 1, 256, 1, False), (4096, 2, 301, 3, False),
                                                                 (4544, 3, 67, 2, True)])
def test_fused_importance_matches_oracle_and_the_two_call_form(dtype, hidden, batch, prompt, chunks, in_place):
    """The statistic taken in the pass that forms the hidden state after self-attention: the
    stored sum is the dtype-rounded residual + attention output, the cosines are those of the
    oracle on (residual, stored sum), and the budgets are bit for bit those of the separate call."""
    w = small("impf", 12, hidden=hidden, batch=batch, prompt=prompt, dtype=dtype, n_layer=4)
    fused, plain = H.make_ctx(w), H.make_ctx(w)
    fused.begin_sequence_batch(w.batch, w.prompt)
    plain.begin_sequence_batch(w.batch, w.prompt)
    want = []
    for l in range(w.n_layer):
        resid, after = synth.hidden_pair(w, l, DEV)
        resid, after = resid.reshape(-1, hidden), after.reshape(-1, hidden)
        attn = (after.float() - resid.float()).to(dtype)                 # what the attention block adds
        stored = (resid.float() + attn.float()).to(dtype)                # one fp32 addition, rounded
        n = resid.shape[0]
        edges = [round(i * n / chunks) for i in range(chunks + 1)]
        out = torch.full_like(resid, float("nan"))
        for i in range(chunks):
            a, b = resid[edges[i]:edges[i + 1]].contiguous(), attn[edges[i]:edges[i + 1]].contiguous()
            if in_place:
                fused.layer_importance_fused(l, a, b, b)                 # the sum overwrites the attention output
                out[edges[i]:edges[i + 1]] = b
            else:
                o = out[edges[i]:edges[i + 1]]
                fused.layer_importance_fused(l, a, b, o)
            assert torch.equal(a, resid[edges[i]:edges[i + 1]])          # inputs other than the target are untouched
            plain.layer_importance(l, a, stored[edges[i]:edges[i + 1]].contiguous())   # same chunks: same summation order
        torch.cuda.synchronize()
        assert torch.equal(out, stored)
        want.append(O.layer_importance(H.f64(resid), H.f64(stored)))
    fused.allocate_budgets(w.b_init, w.p)
    plain.allocate_budgets(w.b_init, w.p)
    got = fused.get_cos_sim().numpy()
    assert np.max(np.abs(got - np.array(want))) <= H.TOL_OUT[dtype]
    assert np.array_equal(got, plain.get_cos_sim().numpy())
    assert fused.get_budgets() == plain.get_budgets()
    wb, wg = O.allocate_budgets(got, w.b_init, w.p)
    assert fused.get_budgets() == (wb.tolist(), wg.tolist())
    assert fused.status() == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_importance_state_exchange_gives_the_batch_budgets(dtype):
    """A batch sharded over two ranks (emulated by two contexts, each fed half the sequences):
    after the per-layer cosine sums and token counts are summed and put back, both allocate the
    budgets the oracle derives from the whole batch's layer averages, and so does a context that
    saw the whole batch."""
    w = small("shard", 13, n_layer=6, hidden=512, batch=4, prompt=96, dtype=dtype)
    whole = H.make_ctx(w)
    whole.begin_sequence_batch(w.batch, w.prompt)
    half = [H.make_ctx(w.replace(batch=2)) for _ in range(2)]
    for h in half:
        h.begin_sequence_batch(2, w.prompt)
    cos_rows = []
    for l in range(w.n_layer):
        a, b = synth.hidden_pair(w, l, DEV)                      # [batch, prompt, hidden]
        whole.layer_importance(l, a, b)
        for r, h in enumerate(half):
            h.layer_importance(l, a[2 * r:2 * r + 2].contiguous(), b[2 * r:2 * r + 2].contiguous())
        cos_rows.append(O.layer_importance(H.f64(a).reshape(-1, w.hidden), H.f64(b).reshape(-1, w.hidden)))
    states = [h.get_importance_state() for h in half]
    sums = [x + y for x, y in zip(states[0][0], states[1][0])]
    counts = [x + y for x, y in zip(states[0][1], states[1][1])]
    assert counts == [w.batch * w.prompt] * w.n_layer
    for h in half:
        h.set_importance_state(sums, counts)
        h.allocate_budgets(w.b_init, w.p)
    whole.allocate_budgets(w.b_init, w.p)
    cos = half[0].get_cos_sim().numpy().astype(np.float64)
    assert np.max(np.abs(cos - np.array(cos_rows))) <= H.TOL_OUT[dtype]
    assert np.max(np.abs(cos - whole.get_cos_sim().numpy().astype(np.float64))) <= 1e-6
    want_b, want_g = O.allocate_budgets(half[0].get_cos_sim().numpy(), w.b_init, w.p)
    for c in (half[0], half[1], whole):
        assert c.get_budgets() == (want_b.tolist(), want_g.tolist())
        assert c.status() == 0
    # argument and mode errors: a count below 1; per-sequence budgets have nothing to exchange
    with pytest.raises(B.SqError) as e:
        half[0].set_importance_state(sums, [0] * w.n_layer)
    assert e.value.code == B.SQ_ERR_INVALID_ARG
    per_seq = H.make_ctx(w, per_sequence_budgets=1)
    per_seq.begin_sequence_batch(w.batch, w.prompt)
    with pytest.raises(B.SqError) as e:
        per_seq.get_importance_state()
    assert e.value.code == B.SQ_ERR_UNSUPPORTED


def test_layer_importance_special_vectors():
    w = small("imp2", 12, n_layer=4, hidden=64, batch=1, prompt=8)
    ctx = H.make_ctx(w)
    ctx.begin_sequence_batch(1, 8)
    g = torch.Generator().manual_seed(5)
    x = torch.randn(8, 64, generator=g).to(DEV)
    zero_row = x.clone(); zero_row[3] = 0
    ortho_a = torch.zeros(8, 64, device=DEV); ortho_a[:, 0] = 2
    ortho_b = torch.zeros(8, 64, device=DEV); ortho_b[:, 5] = -3
    ctx.layer_importance(0, x, x.clone())
    ctx.layer_importance(1, x, (-2 * x).contiguous())
    ctx.layer_importance(2, ortho_a, ortho_b)
    ctx.layer_importance(3, zero_row, x)          # one zero-norm token contributes 0
    ctx.allocate_budgets(w.b_init, w.p)
    got = ctx.get_cos_sim().numpy()
    assert got[0] == pytest.approx(1.0, abs=1e-6)
    assert got[1] == pytest.approx(-1.0, abs=1e-6)
    assert got[2] == 0.0
    assert got[3] == pytest.approx(7.0 / 8.0, abs=1e-6)


# --------------------------------------------------------------------- budgets
@pytest.mark.parametrize("n_layer,n_cluster", [(4, 3), (32, 3), (32, 2), (80, 3), (7, 2), (256, 3)])
@pytest.mark.parametrize("b_init,p", [(102, 0.3), (409, 0.3), (819, 0.35), (1000, 0.3), (5, 0.1), (1228, 1.0)])
def test_budgets_bit_exact(n_layer, n_cluster, b_init, p):
    w = small("alloc", 13, n_layer=n_layer, hidden=64, batch=1, prompt=16)
    ctx = H.make_ctx(w, b_init=b_init, n_cluster=n_cluster)
    H.run_importance_and_allocate(ctx, w, DEV, b_init=b_init, p=p)
    cos = ctx.get_cos_sim().numpy()
    budgets, is_g3 = ctx.get_budgets()
    want_b, want_g = O.allocate_budgets(cos, b_init, p, n_cluster)
    assert budgets == want_b.tolist()
    assert is_g3 == want_g.tolist()
    assert sum(budgets) == n_layer * b_init


def test_budgets_with_tied_and_constant_similarities():
    """Layers fed identical hidden states get bit-identical similarities: exercises ties,
    fewer distinct values than clusters, and the single-value case."""
    g = torch.Generator().manual_seed(3)
    a = torch.randn(16, 64, generator=g)
    noise = torch.randn(16, 64, generator=g)
    variants = [a + 0.2 * noise, a + 0.8 * noise, a + 2.0 * noise]
    for pattern, n_cluster in [([0, 0, 1, 1], 2), ([0, 0, 1, 1], 3), ([2, 2, 2, 2], 3), ([0, 1, 2, 0, 1, 2], 3),
                               ([1, 0, 1, 0, 2], 2)]:
        w = small("tie", 14, n_layer=len(pattern), hidden=64, batch=1, prompt=16)
        ctx = H.make_ctx(w, b_init=100, n_cluster=n_cluster)
        ctx.begin_sequence_batch(1, 16)
        for l, v in enumerate(pattern):
            ctx.layer_importance(l, a.to(DEV), variants[v].to(DEV))
        ctx.allocate_budgets(100, 0.3)
        cos = ctx.get_cos_sim().numpy()
        budgets, is_g3 = ctx.get_budgets()
        want_b, want_g = O.allocate_budgets(cos, 100, 0.3, n_cluster)
        assert budgets == want_b.tolist() and is_g3 == want_g.tolist()
        assert len(set(cos.tolist())) == len(set(pattern))


# ------------------------------------------------------------ prefill / C_seq
def _check_kept(ctx, w, budgets, prompt_cpu, units, check_kv=True):
    for (l, s, h) in units:
        u = H.oracle_unit(w, budgets, prompt_cpu, l, s, h)
        pos, acc = ctx.get_kept(l, s, h)
        assert pos == u.kept_positions(), (l, s, h)
        if w.policy == synth.H2O:
            assert np.allclose(acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6)
        if check_kv:
            k, v = ctx.get_kv(l, s, h)
            assert np.array_equal(H.f64(k), np.stack(u.K)) and np.array_equal(H.f64(v), np.stack(u.V))


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
@pytest.mark.parametrize("dtype,head_dim", [(torch.float32, 64), (torch.bfloat16, 128)])
@pytest.mark.parametrize("budgets", [[24, 7, 40], [96, 200, 5], [95, 97, 96]])
def test_prefill_compress_keeps_what_cseq_keeps(policy, dtype, head_dim, budgets):
    w = small("pre", 15, policy=policy, dtype=dtype, head_dim=head_dim, heavy_mode="uniform4")
    ctx = H.make_ctx(w, b_init=max(budgets))
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets(budgets)
    prompt_cpu = H.prefill_all(ctx, w, DEV)
    _check_kept(ctx, w, budgets, prompt_cpu, H.all_units(w))
    assert ctx.status() == 0


def test_h2o_prompt_scores_match_oracle():
    for dtype, d, g, P in [(torch.float32, 64, 1, 150), (torch.bfloat16, 128, 4, 150), (torch.bfloat16, 64, 3, 150),
                           (torch.bfloat16, 128, 2, 700), (torch.bfloat16, 64, 5, 513), (torch.bfloat16, 128, 1, 128),
                           (torch.float32, 128, 2, 200),
                           # prompts that leave the second 64-column half of a score tile empty, one column
                           # wide, or ragged on the last tile (each half is drained by its own warps)
                           (torch.bfloat16, 128, 2, 40), (torch.bfloat16, 64, 2, 65), (torch.bfloat16, 128, 1, 193)]:
        w = small("score", 16, policy=synth.H2O, dtype=dtype, head_dim=d, n_q_head=2 * g, n_kv_head=2,
                  prompt=P, n_layer=1, heavy_mode="uniform4")
        ctx = H.make_ctx(w, b_init=w.prompt)
        ctx.begin_sequence_batch(w.batch, w.prompt)
        ctx.set_budgets([w.prompt])                   # keep everything: scores are read back per token
        q, k, v = synth.prompt_qkv(w, 0, DEV)
        ctx.prefill_compress(0, k, v, q)
        for s in range(w.batch):
            for h in range(2):
                pos, acc = ctx.get_kept(0, s, h)
                want = O.prefill_scores(H.f64(q[s, h * g:(h + 1) * g]), H.f64(k[s, h]))
                assert pos == list(range(w.prompt))
                assert np.allclose(acc, want, rtol=H.RTOL_ACC[dtype], atol=1e-6)
                assert abs(sum(acc) - g * w.prompt) < 1e-3 * g * w.prompt


def test_h2o_selection_on_identical_score_bits():
    """Selection alone: the same fp32 score bits go to both sides, including heavy ties,
    signed zeros, subnormals and equal scores everywhere."""
    P, U = 300, 6
    rng = np.random.default_rng(17)
    rows = [
        rng.random(P).astype(np.float32),
        np.round(rng.random(P) * 4).astype(np.float32) / 4,                 # many ties
        np.ones(P, dtype=np.float32),                                          # all equal
        np.where(rng.random(P) < 0.5, 0.0, -0.0).astype(np.float32),           # +0 / -0
        (rng.integers(0, 3, P) * np.float32(1e-42)).astype(np.float32),        # subnormals with ties
        np.concatenate([np.zeros(P - 5), rng.random(5)]).astype(np.float32),
    ]
    acc = np.stack(rows)
    for b, (hn, hd) in [(50, (1, 2)), (51, (1, 2)), (2, (1, 2)), (1, (1, 2)), (299, (2, 3)), (120, (9, 10)), (64, (0, 1))]:
        w = small("sel", 18, policy=synth.H2O, n_layer=1, n_q_head=2, n_kv_head=2, batch=3, prompt=P,
                  heavy_num=hn, heavy_den=hd)
        assert w.batch * w.n_kv_head == U
        ctx = H.make_ctx(w, b_init=b)
        ctx.begin_sequence_batch(w.batch, P)
        ctx.set_budgets([b])
        _, k, v = synth.prompt_qkv(w, 0, DEV, need_q=False)
        ctx.prefill_compress(0, k, v, None, torch.from_numpy(acc).to(DEV))
        for u in range(U):
            pos, got_acc = ctx.get_kept(0, u // 2, u % 2)
            keep = O.c_seq(O.H2O, list(range(P)), acc[u], b, heavy_num=hn, heavy_den=hd)
            assert pos == keep, (b, hn, hd, u)
            assert np.array_equal(np.array(got_acc, dtype=np.float32), acc[u][keep])
        assert ctx.status() == 0


# --------------------------------------------------------------------- decoding
def _run_decode_and_compare(w, budgets=None, units=None, per_layer_calls=False, check_every_step=True, **over):
    ctx = H.make_ctx(w, b_init=None if budgets is None else max(budgets), **over)
    if budgets is None:
        want_cos = H.run_importance_and_allocate(ctx, w, DEV)
        got_cos = ctx.get_cos_sim().numpy()
        assert np.max(np.abs(got_cos - want_cos)) <= H.TOL_OUT[w.dtype]
        budgets, is_g3 = ctx.get_budgets()
        want_b, want_g = O.allocate_budgets(got_cos, w.b_init, w.p)
        assert budgets == want_b.tolist() and is_g3 == want_g.tolist()
    else:
        ctx.begin_sequence_batch(w.batch, w.prompt)
        ctx.set_budgets(budgets)
    prompt_cpu = H.prefill_all(ctx, w, DEV)
    units = units or H.all_units(w)
    oracles = {u: H.oracle_unit(w, budgets, prompt_cpu, *u) for u in units}
    g = w.group
    worst = 0.0
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
            err = float(np.max(np.abs(got - want)))
            worst = max(worst, err)
            assert err <= H.TOL_OUT[w.dtype], (t, l, s, h, err)
            if check_every_step or t == w.steps - 1:
                pos, acc = ctx.get_kept(l, s, h)
                assert pos == u.kept_positions(), (t, l, s, h)
                if w.policy == synth.H2O:
                    assert np.allclose(acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), (t, l, s, h)
    assert ctx.status() == 0
    return worst


def test_tiny_config_full_trajectory():
    """The small reference configuration: 4 layers, 2 MHA heads of 64, fp32, prompt 256,
    16 steps, H2O (half heavy, half recent), total budget 40% of the prompt, p = 0.3."""
    w = synth.tiny()
    _run_decode_and_compare(w)


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
@pytest.mark.parametrize("dtype,head_dim,hq,hkv", [
    (torch.float32, 64, 2, 2), (torch.float32, 128, 8, 2), (torch.bfloat16, 128, 4, 4),
    (torch.bfloat16, 128, 8, 2), (torch.bfloat16, 128, 16, 2), (torch.bfloat16, 64, 71, 1),
    (torch.bfloat16, 64, 6, 2), (torch.bfloat16, 128, 20, 1), (torch.bfloat16, 64, 48, 2),
    (torch.bfloat16, 128, 40, 1), (torch.bfloat16, 64, 40, 1), (torch.bfloat16, 64, 128, 1)])
def test_decode_small_shapes(policy, dtype, head_dim, hq, hkv):
    w = small("dec", 19, policy=policy, dtype=dtype, head_dim=head_dim, n_q_head=hq, n_kv_head=hkv,
              heavy_mode="uniform4", steps=7)
    _run_decode_and_compare(w, budgets=[24, 9, 101])     # over budget, tiny budget, still growing


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
def test_decode_per_layer_calls_and_growth_through_budget(policy):
    # the cache fills up during decoding (prompt 20 < budget 23 < prompt + steps)
    w = small("grow", 20, policy=policy, prompt=20, steps=9, batch=1, heavy_mode="none")
    _run_decode_and_compare(w, budgets=[23, 6, 64], per_layer_calls=True)


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
@pytest.mark.parametrize("dtype,head_dim", [(torch.bfloat16, 128), (torch.bfloat16, 64), (torch.float32, 128),
                                            (torch.float32, 64)])
def test_decode_one_head_per_kv_head_few_unsplit_units(policy, dtype, head_dim):
    """One query head per KV head, few units, budgets short enough to stay unsplit: the launches
    that give every unit 16 warps.  The budgets take a warp through one to five loads with a ragged
    last one (a pass of the 16 warps covers 64 to 256 rows, by row size), called layer by layer
    and for all layers at once."""
    w = small("mha_few", 41, policy=policy, dtype=dtype, head_dim=head_dim, n_q_head=3, n_kv_head=3, batch=2,
              n_layer=3, prompt=330, steps=4, heavy_mode="zipf")
    _run_decode_and_compare(w, budgets=[277, 131, 65], per_layer_calls=True)
    _run_decode_and_compare(w.replace(wid=42), budgets=[200, 290, 129])


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.H2O])
def test_decode_split_k_long_context(policy):
    # few units, long budgets: the launch splits each unit's tokens over several CTAs
    w = small("split", 21, policy=policy, dtype=torch.bfloat16, head_dim=128, n_q_head=8, n_kv_head=2, batch=1,
              n_layer=2, prompt=3000, steps=3, heavy_mode="zipf")
    _run_decode_and_compare(w, budgets=[2500, 1100], check_every_step=False)


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
def test_decode_wide_mqa_long_context(policy):
    # Falcon-shaped group (71 query heads on one KV head): several 128-token tiles, ragged tail,
    # with and without split-K
    w = small("mqa", 28, policy=policy, dtype=torch.bfloat16, head_dim=64, n_q_head=71, n_kv_head=1, batch=2,
              n_layer=2, prompt=1500, steps=3, hidden=64, heavy_mode="zipf")
    _run_decode_and_compare(w, budgets=[1300, 700], check_every_step=False)
    w1 = w.replace(batch=1, prompt=2100, wid=29)
    _run_decode_and_compare(w1, budgets=[2050, 300], check_every_step=False)


@pytest.mark.parametrize("hq", [36, 68, 100])
@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.H2O])
def test_decode_wide_mqa_sparsely_filled_quarter(policy, hq):
    """Group sizes that leave 4 head rows in the second, third or fourth quarter of the 128-row
    tile (worked four threads to a row), over several tiles with a ragged tail, with and without
    split-K."""
    w = small("mqa_quad", 32 + hq, policy=policy, dtype=torch.bfloat16, head_dim=64, n_q_head=hq, n_kv_head=1, batch=2,
              n_layer=2, prompt=1500, steps=3, hidden=64, heavy_mode="zipf")
    _run_decode_and_compare(w, budgets=[1300, 900], check_every_step=False)
    w1 = w.replace(batch=1, prompt=2100, wid=w.wid + 1)
    _run_decode_and_compare(w1, budgets=[2050, 800], check_every_step=False)


@pytest.mark.parametrize("prompt", [400, 1000])
def test_decode_wide_mqa_growing_logits(prompt):
    """Keys late in the cache are far larger than the early ones, so the running reference of
    the softmax has to move after the first tile (4 tiles: every quarter a row per thread; 8 tiles:
    the third quarter in quads)."""
    w = small("mqa_grow", 30, policy=synth.SLIDING_WINDOW, dtype=torch.bfloat16, head_dim=64, n_q_head=71,
              n_kv_head=1, batch=1, n_layer=1, prompt=prompt, steps=2, hidden=64)
    b = prompt + 112
    ctx = H.make_ctx(w, b_init=b)
    ctx.begin_sequence_batch(1, w.prompt)
    ctx.set_budgets([b])
    _, k, v = synth.prompt_qkv(w, 0, DEV, need_q=False)
    k = k.clone()
    k[:, :, prompt // 3:2 * prompt // 3] *= 12.0
    k[:, :, 2 * prompt // 3:] *= 30.0
    ctx.prefill_compress(0, k, v)
    u = O.UnitCache(O.SLIDING_WINDOW, b)
    u.prefill(H.f64(k[0, 0]), H.f64(v[0, 0]))
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, 1, q, kn, vn, out)
        want = u.decode_step(H.f64(q[0, 0]), H.f64(kn[0, 0, 0]), H.f64(vn[0, 0, 0]))
        # so peaked that an output is close to one V row: where it exceeds 4 in magnitude the bf16
        # output format itself is coarser than 1e-2 (half an ulp is 0.0156 between 4 and 8)
        tol = np.maximum(H.TOL_OUT[w.dtype], 2.0 ** -7 * np.abs(want))
        assert np.all(np.abs(H.f64(out[0, 0]) - want) <= tol)
    assert ctx.status() == 0


@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.H2O])
def test_decode_wide_mqa_even_deal_launch(policy):
    """One layer of a batch whose units are long but fewer than the CTA slots goes to the kernel
    that deals the launch's tiles out evenly: segments end inside units, so pieces are merged by
    the last to arrive; a ragged last tile; and, for some sequences, keys that grow along the
    cache, so that the softmax reference has to move inside a segment."""
    w = small("mqa_deal", 31, policy=policy, dtype=torch.bfloat16, head_dim=64, n_q_head=71, n_kv_head=1,
              batch=160, n_layer=1, prompt=2100, steps=2, hidden=64, heavy_mode="none")
    b = 2200  # 18 tiles per unit, 160 units for 296 CTA slots; the cache is still growing
    ctx = H.make_ctx(w, b_init=b)
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets([b])
    q_p, k, v = synth.prompt_qkv(w, 0, DEV, need_q=(policy == synth.H2O))
    k = k.clone()
    grow = [0, 7, 159]
    for s_ in grow:
        k[s_, :, 700:1400] *= 10.0
        k[s_, :, 1400:] *= 25.0
    ctx.prefill_compress(0, k, v, q_p)
    seqs = [0, 1, 7, 80, 158, 159]
    units = {}
    for s_ in seqs:
        u = O.UnitCache(policy, b, w.n_sink, w.heavy_num, w.heavy_den)
        u.prefill(H.f64(k[s_, 0]), H.f64(v[s_, 0]), H.f64(q_p[s_]) if policy == synth.H2O else None)
        units[s_] = u
    for t in range(w.steps):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, 1, q[0], kn[0], vn[0], out[0])
        for s_, u in units.items():
            want = u.decode_step(H.f64(q[0, s_]), H.f64(kn[0, s_, 0]), H.f64(vn[0, s_, 0]))
            got = H.f64(out[0, s_])
            tol = np.maximum(H.TOL_OUT[w.dtype], 2.0 ** -7 * np.abs(want))
            assert np.all(np.abs(got - want) <= tol), (t, s_, np.max(np.abs(got - want)))
            if policy == synth.H2O:
                pos, acc = ctx.get_kept(0, s_, 0)
                assert pos == u.kept_positions()
                assert np.allclose(acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), (t, s_)
    assert ctx.status() == 0


def test_decode_budget_one_and_sinks_only_edge():
    w = small("edge", 22, policy=synth.SLIDING_WINDOW, steps=3)
    _run_decode_and_compare(w, budgets=[1, 2, 3])
    w = small("edge2", 23, policy=synth.STREAMING_LLM, steps=5)
    _run_decode_and_compare(w, budgets=[5, 6, 50])       # one, two recent slots beside the 4 sinks


def test_determinism_same_inputs_same_bits():
    w = small("det", 24, policy=synth.H2O, dtype=torch.bfloat16, head_dim=128, n_q_head=8, n_kv_head=2,
              heavy_mode="uniform4", steps=4)
    outs = []
    for _ in range(2):
        ctx = H.make_ctx(w, b_init=40)
        ctx.begin_sequence_batch(w.batch, w.prompt)
        ctx.set_budgets([40, 12, 30])
        H.prefill_all(ctx, w, DEV, keep_inputs=False)
        res = []
        for t in range(w.steps):
            q, kn, vn = synth.decode_qkv(w, t, DEV)
            out = torch.empty_like(q)
            ctx.decode_step(0, w.n_layer, q, kn, vn, out)
            res.append(out.cpu())
        res.append(ctx.get_kept(0, 1, 1))
        outs.append(res)
    for a, b in zip(outs[0][:-1], outs[1][:-1]):
        assert torch.equal(a, b)
    assert outs[0][-1] == outs[1][-1]


# ----------------------------------------------------------------------- evict
@pytest.mark.parametrize("policy", [synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
def test_evict_in_place_then_keep_decoding(policy):
    w = small("evict", 25, policy=policy, dtype=torch.bfloat16, head_dim=128, heavy_mode="uniform4", steps=8)
    budgets = [40, 30, 120]
    ctx = H.make_ctx(w, b_init=max(budgets))
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets(budgets)
    prompt_cpu = H.prefill_all(ctx, w, DEV)
    units = H.all_units(w)
    oracles = {u: H.oracle_unit(w, budgets, prompt_cpu, *u) for u in units}
    g = w.group
    new_budgets = [17, 30, 50]

    def step(t):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        qc, kc, vc, oc = q.cpu(), kn.cpu(), vn.cpu(), out.cpu()
        for (l, s, h) in units:
            u = oracles[(l, s, h)]
            want = u.decode_step(H.f64(qc[l, s, h * g:(h + 1) * g]), H.f64(kc[l, s, h]), H.f64(vc[l, s, h]))
            assert np.max(np.abs(H.f64(oc[l, s, h * g:(h + 1) * g]) - want)) <= H.TOL_OUT[w.dtype]
            pos, acc = ctx.get_kept(l, s, h)
            assert pos == u.kept_positions(), (t, l, s, h)

    for t in range(3):
        step(t)
    ctx.evict(0, w.n_layer, new_budgets)
    for (l, s, h) in units:
        u = oracles[(l, s, h)]
        u.b = new_budgets[l]
        u._compress()
    for (l, s, h) in units:
        pos, acc = ctx.get_kept(l, s, h)
        assert pos == oracles[(l, s, h)].kept_positions(), (l, s, h)
        k, v = ctx.get_kv(l, s, h)
        assert np.array_equal(H.f64(k), np.stack(oracles[(l, s, h)].K))
    for t in range(3, w.steps):
        step(t)
    assert ctx.get_budgets()[0] == new_budgets
    assert ctx.status() == 0


@pytest.mark.parametrize("dtype,head_dim,hq,hkv", [(torch.float32, 64, 4, 2), (torch.bfloat16, 128, 8, 2),
                                                  (torch.bfloat16, 64, 71, 1)])
def test_evict_of_a_growing_h2o_cache_to_exactly_its_length(dtype, head_dim, hq, hkv):
    """A cache still below its budget (prompt 20, budget 40, 10 steps -> 30 tokens) is lowered to
    a budget equal to its length: nothing is dropped, but the very next step is over budget, so
    the slot that step reuses has to be chosen by the eviction call itself."""
    w = small("evict_eq", 27, policy=synth.H2O, dtype=dtype, head_dim=head_dim, n_q_head=hq, n_kv_head=hkv,
              prompt=20, heavy_mode="uniform4", steps=13)
    budgets = [40, 40, 25]
    ctx = H.make_ctx(w, b_init=max(budgets))
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets(budgets)
    prompt_cpu = H.prefill_all(ctx, w, DEV)
    units = H.all_units(w)
    oracles = {u: H.oracle_unit(w, budgets, prompt_cpu, *u) for u in units}
    g = w.group

    def step(t):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        qc, kc, vc, oc = q.cpu(), kn.cpu(), vn.cpu(), out.cpu()
        for (l, s, h) in units:
            u = oracles[(l, s, h)]
            want = u.decode_step(H.f64(qc[l, s, h * g:(h + 1) * g]), H.f64(kc[l, s, h]), H.f64(vc[l, s, h]))
            assert np.max(np.abs(H.f64(oc[l, s, h * g:(h + 1) * g]) - want)) <= H.TOL_OUT[w.dtype], (t, l, s, h)
            pos, acc = ctx.get_kept(l, s, h)
            assert pos == u.kept_positions(), (t, l, s, h)
            assert np.allclose(acc, u.acc, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), (t, l, s, h)

    for t in range(10):
        step(t)
    new_budgets = [30, 35, 25]          # exactly the length / still above it / unchanged (already full)
    ctx.evict(0, w.n_layer, new_budgets)
    for (l, s, h) in units:
        oracles[(l, s, h)].b = new_budgets[l]
        oracles[(l, s, h)]._compress()
        assert ctx.get_kept(l, s, h)[0] == oracles[(l, s, h)].kept_positions()
    for t in range(10, w.steps):
        step(t)
    assert ctx.status() == 0


@pytest.mark.parametrize("policy,dtype,head_dim,hq,hkv", [
    (synth.SLIDING_WINDOW, torch.bfloat16, 128, 4, 4), (synth.STREAMING_LLM, torch.bfloat16, 128, 8, 2),
    (synth.H2O, torch.float32, 64, 4, 2), (synth.H2O, torch.bfloat16, 64, 71, 1)])
def test_checkpoint_and_resume_through_the_exported_layout(policy, dtype, head_dim, hq, hkv):
    """A batch stopped after some steps (one explicit eviction among them) and resumed in a fresh
    context from the exported layout table and a copy of the pool's bytes continues bit for bit
    like the batch that was never stopped."""
    w = small("ckpt", 28, policy=policy, dtype=dtype, head_dim=head_dim, n_q_head=hq, n_kv_head=hkv,
              heavy_mode="uniform4", steps=10)
    budgets = [40, 30, 120]

    def fresh():
        ctx = H.make_ctx(w, b_init=max(budgets))
        ctx.begin_sequence_batch(w.batch, w.prompt)
        return ctx

    def step(ctx, t):
        q, kn, vn = synth.decode_qkv(w, t, DEV)
        out = torch.empty_like(q)
        ctx.decode_step(0, w.n_layer, q, kn, vn, out)
        return out

    a = fresh()
    a.set_budgets(budgets)
    H.prefill_all(a, w, DEV, keep_inputs=False)
    for t in range(3):
        step(a, t)
    a.evict(0, w.n_layer, [25, 30, 64])
    step(a, 3)
    layout = a.export_layout()
    assert [e.budget for e in layout] == [25, 30, 64] and all(e.n_tok == w.prompt + 4 for e in layout)
    saved = a.pool_view.clone()
    b = fresh()
    b.import_layout(layout)
    b.pool_view.copy_(saved)
    assert b.get_budgets()[0] == [25, 30, 64]
    for t in range(4, w.steps):
        oa, ob = step(a, t), step(b, t)
        assert torch.equal(oa, ob), t
    for key in H.all_units(w):
        assert a.get_kept(*key) == b.get_kept(*key)
    assert a.status() == 0 and b.status() == 0
    # a table from another shape is refused
    other = H.make_ctx(w.replace(batch=w.batch + 1), b_init=max(budgets))
    other.begin_sequence_batch(w.batch + 1, w.prompt)
    with pytest.raises(B.SqError):
        other.import_layout(layout)


# ----------------------------------------------------------------- error paths
def test_call_order_and_argument_errors():
    w = small("err", 26)
    ctx = H.make_ctx(w, b_init=30)
    x = torch.zeros(16, w.hidden, device=DEV)
    with pytest.raises(B.SqError) as e:
        ctx.layer_importance(0, x, x)
    assert e.value.code == B.SQ_ERR_STATE
    ctx.begin_sequence_batch(w.batch, w.prompt)
    with pytest.raises(B.SqError) as e:
        ctx.allocate_budgets(30, 0.3)            # no importance yet
    assert e.value.code == B.SQ_ERR_STATE
    q, k, v = synth.prompt_qkv(w, 0, DEV, need_q=False)
    with pytest.raises(B.SqError) as e:
        ctx.prefill_compress(0, k, v)            # no budgets yet
    assert e.value.code == B.SQ_ERR_STATE
    with pytest.raises(B.SqError) as e:
        ctx.set_budgets([60, 60, 60])            # does not fit the pool sized for 3 * 30
    assert e.value.code == B.SQ_ERR_CAPACITY
    ctx.set_budgets([30, 30, 30])
    dq, dk, dv = synth.decode_qkv(w, 0, DEV)
    with pytest.raises(B.SqError) as e:
        ctx.decode_step(0, 3, dq, dk, dv, torch.empty_like(dq))   # not prefilled
    assert e.value.code == B.SQ_ERR_STATE
    for bad in [(0.0,), (1.5,), (-0.1,)]:
        with pytest.raises(B.SqError) as e:
            ctx.allocate_budgets(30, bad[0])
        assert e.value.code in (B.SQ_ERR_INVALID_ARG, B.SQ_ERR_STATE)
    with pytest.raises(B.SqError) as e:
        ctx.begin_sequence_batch(w.batch + 1, w.prompt)
    assert e.value.code == B.SQ_ERR_INVALID_ARG
    ws = small("err2", 27, policy=synth.STREAMING_LLM)
    c2 = H.make_ctx(ws, b_init=30)
    c2.begin_sequence_batch(ws.batch, ws.prompt)
    with pytest.raises(B.SqError) as e:
        c2.set_budgets([30, 4, 30])              # a budget that leaves no room beside the sinks
    assert e.value.code == B.SQ_ERR_INVALID_ARG


# ------------------------------------------------------- launch forms agree
def test_graph_replay_and_per_layer_calls_match_fused_launch():
    """The same decode steps issued as one launch per step, as one launch per layer, and as a
    CUDA-graph replay of the per-layer launches give identical bits."""
    from paper_2404_04793_b200 import engine
    w = small("forms", 31, policy=synth.STREAMING_LLM, dtype=torch.bfloat16, head_dim=128, n_q_head=8, n_kv_head=2,
              n_layer=4, steps=5)
    inp = engine.ResidentInputs(w, DEV)
    outs = []
    for mode in ("fused", "per_layer", "graph"):
        job = engine.Job(w, DEV, per_layer_decode=(mode == "per_layer"))
        job.prefill(inp)
        if mode == "graph":
            graph = job.capture_decode(inp, per_layer=True)
            job.prefill(inp)
            graph.replay()
        else:
            job.decode(inp)
        torch.cuda.synchronize()
        assert job.ctx.status() == 0
        outs.append(job.out.clone())
    assert torch.equal(outs[0], outs[1])
    assert torch.equal(outs[0], outs[2])
