"""The allocation-free scoring entry point against the regular one.

sq_prompt_scores_static serves hosts that must not call cudaMalloc (pre-sized memory pools,
plugins whose runtime owns all allocations, services that forbid allocation after start-up):
its intermediate lives in a fixed array inside the library.  Here it is called twice in a row
through the C ABI -- the second call on a different, smaller problem, so stale contents of the
shared array would show -- and each result is compared with the scores sq_prefill_compress
computes for the same prompt and with the CPU oracle's, within the tolerance the other score
tests use.  A request that fills the array exactly is checked the same way, together with the
property the entry point exists for: a call changes neither the device's free memory nor the
allocator's count.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import sq_oracle as O
from paper_2404_04793_b200 import binding as B
from paper_2404_04793_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _scores_via_context(w, q, k, v):
    ctx = H.make_ctx(w, b_init=w.prompt)
    ctx.begin_sequence_batch(w.batch, w.prompt)
    ctx.set_budgets([w.prompt] * w.n_layer)        # keep every token so every score can be read back
    ctx.prefill_compress(0, k, v, q)
    out = np.zeros((w.batch, w.n_kv_head, w.prompt), dtype=np.float32)
    for s in range(w.batch):
        for h in range(w.n_kv_head):
            pos, acc = ctx.get_kept(0, s, h)
            assert pos == list(range(w.prompt))
            out[s, h] = acc
    return out


def _case(i, **kw):
    w = synth.Workload(f"noalloc{i}", 40 + i, n_layer=1, hidden=64, steps=1, policy=synth.H2O, budget_pct=100.0,
                       p=0.3, heavy_mode="uniform4", **kw)
    return (w,) + synth.prompt_qkv(w, 0, DEV)


def test_static_scores_match_regular_entry_point_and_oracle_twice_in_a_row():
    cases = [
        dict(dtype=torch.bfloat16, head_dim=128, n_q_head=8, n_kv_head=2, batch=2, prompt=333),
        dict(dtype=torch.float32, head_dim=64, n_q_head=3, n_kv_head=1, batch=1, prompt=97),
    ]
    for i, kw in enumerate(cases):
        w, q, k, v = _case(i, **kw)
        acc = torch.full((w.batch, w.n_kv_head, w.prompt), float("nan"), dtype=torch.float32, device=DEV)
        B.sq_prompt_scores_static(q, k, acc)
        torch.cuda.synchronize()
        got = acc.cpu().numpy()
        want = _scores_via_context(w, q, k, v)
        assert np.isfinite(got).all()
        assert np.allclose(got, want, rtol=H.RTOL_ACC[w.dtype], atol=1e-6)
        assert abs(got.sum() - w.batch * w.n_q_head * w.prompt) < 1e-3 * w.batch * w.n_q_head * w.prompt
        # and against the CPU oracle's definition of the prompt scores
        g = w.group
        for s in range(w.batch):
            for h in range(w.n_kv_head):
                exact = O.prefill_scores(H.f64(q[s, h * g:(h + 1) * g]), H.f64(k[s, h]))
                assert np.allclose(got[s, h], exact, rtol=H.RTOL_ACC[w.dtype], atol=1e-6), (i, s, h)


def test_static_scores_fill_the_array_exactly_and_allocate_nothing():
    """A request of exactly SQ_STATIC_SCORE_MAX_ROWS rows uses the array to its last entry (one
    more row is refused, see below); and across a call the device's free memory and torch's own
    allocation count stay where they were: the call draws on no allocator."""
    w, q, k, v = _case(2, dtype=torch.float32, head_dim=64, n_q_head=8, n_kv_head=2, batch=128, prompt=1024)
    assert w.batch * w.n_q_head * w.prompt == B.SQ_STATIC_SCORE_MAX_ROWS
    acc = torch.full((w.batch, w.n_kv_head, w.prompt), float("nan"), dtype=torch.float32, device=DEV)
    B.sq_prompt_scores_static(q, k, acc)                 # warm call (first use on the device resolves the array)
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    acc.fill_(float("nan"))
    B.sq_prompt_scores_static(q, k, acc)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    got = acc.cpu().numpy()
    assert np.isfinite(got).all()
    want = _scores_via_context(w, q, k, v)
    assert np.allclose(got, want, rtol=H.RTOL_ACC[w.dtype], atol=1e-6)
    # the last sequence and head sit at the end of the array: check them against the oracle too
    g = w.group
    exact = O.prefill_scores(H.f64(q[-1, -g:]), H.f64(k[-1, -1]))
    assert np.allclose(got[-1, -1], exact, rtol=H.RTOL_ACC[w.dtype], atol=1e-6)


def test_static_scores_reject_oversized_and_bad_requests():
    cap = B.SQ_STATIC_SCORE_MAX_ROWS
    q = torch.zeros(1, 2, 8, 64, device=DEV)
    k = torch.zeros(1, 1, 8, 64, device=DEV)
    acc = torch.zeros(1, 1, 8, device=DEV)
    P = B.c_void_p
    args = lambda batch, hq, p, d: (P(q.data_ptr()), P(k.data_ptr()), batch, hq, 1, p, d, B.SQ_F32, P(acc.data_ptr()), None)
    # one row too many: refused before anything is launched (the small tensors are never read)
    assert B.lib().sq_prompt_scores_static(*args(1, 2, cap // 2 + 1, 64)) == B.SQ_ERR_CAPACITY
    assert B.lib().sq_prompt_scores_static(*args(1, 2, 8, 96)) == B.SQ_ERR_UNSUPPORTED
    assert B.lib().sq_prompt_scores_static(*args(0, 2, 8, 64)) == B.SQ_ERR_INVALID_ARG
    assert B.lib().sq_prompt_scores_static(None, P(k.data_ptr()), 1, 2, 1, 8, 64, B.SQ_F32, P(acc.data_ptr()), None) \
        == B.SQ_ERR_INVALID_ARG
