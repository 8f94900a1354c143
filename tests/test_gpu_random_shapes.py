"""Seeded random sweep over shapes, policies, budgets and call forms: the CUDA library against
the oracle on sampled units, including an explicit eviction to random tighter budgets.
Kept sets, cached rows and budgets must be identical; outputs within the max-abs tolerance.
Where the exact output exceeds 1 in magnitude the bf16 formats themselves limit the agreement
(output rounding 2^-9..2^-8 relative, weights entering P.V rounded 2^-9 relative), so the bound
there is 2^-7 of the exact value; below that it is the plain 1e-2 (bf16) / 1e-5 (fp32)."""
import random

import numpy as np
import pytest
import torch

from paper_2404_04793_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"
SHAPES = [(torch.float32, 64, 2, 2), (torch.float32, 128, 4, 2), (torch.float32, 64, 8, 1), (torch.bfloat16, 128, 4, 4),
          (torch.bfloat16, 128, 8, 2), (torch.bfloat16, 128, 32, 1), (torch.bfloat16, 64, 71, 1), (torch.bfloat16, 64, 6, 2),
          (torch.bfloat16, 64, 48, 1), (torch.bfloat16, 64, 128, 1), (torch.bfloat16, 128, 20, 2), (torch.bfloat16, 64, 96, 1)]


def _check_out(got, want, dtype, where):
    tol = H.TOL_OUT[dtype]
    bound = np.maximum(tol, np.abs(want) * 2.0 ** -7) if dtype == torch.bfloat16 else tol
    assert np.all(np.abs(got - want) <= bound), where


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_configurations(seed):
    rng = random.Random(seed)
    for case in range(24):
        dtype, d, hq, hkv = rng.choice(SHAPES)
        policy = rng.choice([synth.SLIDING_WINDOW, synth.STREAMING_LLM, synth.H2O])
        L, B_ = rng.randint(1, 4), rng.randint(1, 4)
        prompt = rng.choice([rng.randint(8, 60), rng.randint(60, 400), rng.randint(400, 2600)])
        steps = rng.randint(2, 4)
        per_seq, per_layer = rng.random() < 0.4, rng.random() < 0.4
        hn, hd = rng.choice([(1, 2), (1, 3), (2, 3), (0, 1), (9, 10)])
        lo = 6 if policy == synth.STREAMING_LLM else 1

        def rb():
            return rng.choice([rng.randint(lo, 12), rng.randint(lo, prompt + steps + 3),
                               rng.randint(max(lo, prompt // 2), prompt + 2)])

        budgets = [[rb() for _ in range(L)] for _ in range(B_)] if per_seq else [rb() for _ in range(L)]
        bmax = max(max(r) for r in budgets) if per_seq else max(budgets)
        w = synth.Workload("rand", 7000 + 100 * seed + case, n_layer=L, n_q_head=hq, n_kv_head=hkv, head_dim=d,
                           hidden=64, batch=B_, prompt=prompt, steps=steps, dtype=dtype, policy=policy,
                           budget_pct=25.0, p=0.3, heavy_num=hn, heavy_den=hd,
                           heavy_mode=rng.choice(["none", "uniform4", "zipf"]))
        tag = (seed, case, str(dtype), d, hq, hkv, policy, L, B_, prompt, per_seq, per_layer, budgets)
        ctx = H.make_ctx(w, b_init=bmax, per_sequence_budgets=int(per_seq))
        ctx.begin_sequence_batch(w.batch, w.prompt)
        ctx.set_budgets(budgets)
        prompt_cpu = H.prefill_all(ctx, w, DEV)
        units = H.sample_units(w, 5, seed=case)
        oracles = {(l, s, h): H.oracle_unit(w, budgets[s] if per_seq else budgets, prompt_cpu, l, s, h)
                   for (l, s, h) in units}
        g = w.group
        diverged = False
        for t in range(steps):
            q, kn, vn = synth.decode_qkv(w, t, DEV)
            out = torch.empty_like(q)
            if per_layer:
                for l in range(L):
                    ctx.decode_step(l, l + 1, q[l], kn[l], vn[l], out[l])
            else:
                ctx.decode_step(0, L, q, kn, vn, out)
            qc, kc, vc, oc = q.cpu(), kn.cpu(), vn.cpu(), out.cpu()
            for (l, s, h) in units:
                u = oracles[(l, s, h)]
                want = u.decode_step(H.f64(qc[l, s, h * g:(h + 1) * g]), H.f64(kc[l, s, h]), H.f64(vc[l, s, h]))
                _check_out(H.f64(oc[l, s, h * g:(h + 1) * g]), want, dtype, (tag, t, l, s, h))
                if ctx.get_kept(l, s, h)[0] != u.kept_positions():
                    # only a free-running H2O trajectory may leave the oracle's (near-tied scores)
                    assert policy == synth.H2O, (tag, t, l, s, h)
                    diverged = True
            if diverged:
                break
        if not diverged:
            newb = [[rng.randint(lo, b) for b in r] for r in budgets] if per_seq else [rng.randint(lo, b) for b in budgets]
            ctx.evict(0, L, newb)
            for (l, s, h) in units:
                u = oracles[(l, s, h)]
                u.b = newb[s][l] if per_seq else newb[l]
                u._compress()
                assert ctx.get_kept(l, s, h)[0] == u.kept_positions(), (tag, "evict", l, s, h)
                if u.K:
                    k, v = ctx.get_kv(l, s, h)
                    assert np.array_equal(H.f64(k), np.stack(u.K)) and np.array_equal(H.f64(v), np.stack(u.V)), (tag, l, s, h)
        assert ctx.status() == 0, tag
        ctx.close()
