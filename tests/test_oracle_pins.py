"""Pins for the CPU oracle: every function is checked against something other
than itself -- values the paper prints, closed forms, invariants, library
routines (scipy / scikit-learn / torch CPU) and brute force on tiny inputs."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import sq_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v) if "." in v else int(v)
    return out


# ----------------------------------------------------------------- importance
def test_cosine_closed_forms():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(64)
    y = rng.standard_normal(64)
    assert O.token_cosine(x, x) == pytest.approx(1.0, abs=1e-15)
    assert O.token_cosine(x, -x) == pytest.approx(-1.0, abs=1e-15)
    e0 = np.zeros(8); e0[0] = 2.0
    e1 = np.zeros(8); e1[3] = -5.0
    assert O.token_cosine(e0, e1) == 0.0
    assert O.token_cosine(3.0 * x, 0.25 * y) == pytest.approx(O.token_cosine(x, y), abs=1e-15)
    # 2-D: angle between (1,0) and (cos t, sin t) is t
    for t in (0.1, 1.0, 2.5):
        assert O.token_cosine([1.0, 0.0], [math.cos(t), math.sin(t)]) == pytest.approx(math.cos(t), abs=1e-15)
    assert O.token_cosine(np.zeros(4), np.ones(4)) == 0.0


def test_cosine_against_scipy_and_sklearn():
    from scipy.spatial.distance import cosine as scipy_cosine_distance
    from sklearn.metrics.pairwise import cosine_similarity
    rng = np.random.default_rng(1)
    a = rng.standard_normal((37, 96))
    b = a + 0.7 * rng.standard_normal((37, 96))
    per_tok = [1.0 - scipy_cosine_distance(a[j], b[j]) for j in range(37)]
    assert O.layer_importance(a, b) == pytest.approx(np.mean(per_tok), abs=1e-14)
    diag = np.diag(cosine_similarity(a, b))
    assert O.layer_importance(a, b) == pytest.approx(diag.mean(), abs=1e-14)
    # a transposed / mismatched pairing must not give the same number
    assert abs(O.layer_importance(a, b[::-1]) - diag.mean()) > 1e-3


def test_importance_is_mean_of_tokens_and_flattens_batch():
    # tokens with known cosines: cos = 1, 0, -1, 0.6  -> mean 0.15
    a = np.array([[1.0, 0.0], [1.0, 0.0], [1.0, 0.0], [5.0, 0.0]])
    b = np.array([[2.0, 0.0], [0.0, 3.0], [-4.0, 0.0], [3.0, 4.0]])
    assert O.layer_importance(a, b) == pytest.approx(0.15, abs=1e-15)
    assert O.layer_importance(a.reshape(2, 2, 2), b.reshape(2, 2, 2)) == pytest.approx(0.15, abs=1e-15)


def test_importance_noise_model_limit():
    # B = A + alpha*noise in high dimension: cos -> 1/sqrt(1+alpha^2)
    rng = np.random.default_rng(2)
    d, n, alpha = 4096, 64, 0.75
    a = rng.standard_normal((n, d))
    b = a + alpha * rng.standard_normal((n, d))
    assert O.layer_importance(a, b) == pytest.approx(1.0 / math.sqrt(1 + alpha * alpha), abs=3e-3)


# ----------------------------------------------------------------- clustering
def _partition_cost(x, labels):
    c = 0.0
    for g in set(labels):
        v = np.array([xi for xi, l in zip(x, labels) if l == g])
        c += float(((v - v.mean()) ** 2).sum())
    return c


def test_cluster_recovers_separated_groups_and_is_permutation_invariant():
    rng = np.random.default_rng(3)
    g1 = 0.62 + 0.01 * rng.standard_normal(3)
    g2 = 0.83 + 0.01 * rng.standard_normal(12)
    g3 = 0.97 + 0.005 * rng.standard_normal(17)
    x = np.concatenate([g1, g2, g3])
    truth = np.array([False] * 15 + [True] * 17)
    assert (O.cluster_layers(x, 3) == truth).all()
    perm = rng.permutation(len(x))
    assert (O.cluster_layers(x[perm], 3) == truth[perm]).all()
    # k = 2 on the same data merges the two lower groups or splits differently, but
    # the top group is still recovered because the largest gap is below it? check via cost
    is3 = O.cluster_layers(x, 2)
    labels = is3.astype(int)
    best = min(_partition_cost(np.sort(x), [0] * i + [1] * (len(x) - i)) for i in range(1, len(x)))
    assert _partition_cost(x, labels) == pytest.approx(best, rel=1e-12)


def test_cluster_small_cases():
    assert list(O.cluster_layers([0.0, 0.0, 1.0, 1.0], 2)) == [False, False, True, True]
    assert list(O.cluster_layers([1.0, 0.0, 1.0, 0.0], 2)) == [True, False, True, False]
    # fewer distinct values than clusters: k drops to the number of distinct values
    assert list(O.cluster_layers([0.5, 0.5, 0.9, 0.9], 3)) == [False, False, True, True]
    # one distinct value: no G3
    assert not O.cluster_layers([0.7, 0.7, 0.7], 3).any()
    # exact tie between {0 | 1,2} and {0,1 | 2}: the first cut in lexicographic order wins
    assert list(O.cluster_layers([0.0, 1.0, 2.0], 2)) == [False, True, True]
    # k = 3 on three values: top one alone
    assert list(O.cluster_layers([0.3, 0.1, 0.2], 3)) == [True, False, False]


def test_cluster_is_global_optimum_vs_sklearn_kmeans():
    from sklearn.cluster import KMeans
    rng = np.random.default_rng(4)
    for trial in range(6):
        n = int(rng.integers(6, 40))
        x = rng.uniform(0.5, 1.0, size=n)
        for k in (2, 3):
            is3 = O.cluster_layers(x, k)
            km = KMeans(n_clusters=k, n_init=50, random_state=trial).fit(x.reshape(-1, 1))
            # our top group together with the optimal split of the rest can be no
            # worse than Lloyd's best: compare through the top-group cut only
            top = np.sort(x)[::-1][: int(is3.sum())]
            rest = np.sort(x)[: n - int(is3.sum())]
            if k == 2:
                ours = float(((top - top.mean()) ** 2).sum() + ((rest - rest.mean()) ** 2).sum())
            else:
                ours = float(((top - top.mean()) ** 2).sum()) + min(
                    float(((rest[:i] - rest[:i].mean()) ** 2).sum() + ((rest[i:] - rest[i:].mean()) ** 2).sum())
                    for i in range(1, len(rest)))
            assert ours <= km.inertia_ * (1 + 1e-9)
            # and when Lloyd reaches the same inertia its top cluster is our G3
            if abs(ours - km.inertia_) <= 1e-9 * max(1.0, ours):
                top_label = int(np.argmax(km.cluster_centers_.ravel()))
                if not ((km.labels_ == top_label) == is3).all():
                    # equal-cost alternative partitions are allowed only on exact ties
                    assert _partition_cost(x, km.labels_) == pytest.approx(ours, rel=1e-9)


def test_cluster_brute_force_all_labelings_tiny():
    rng = np.random.default_rng(5)
    for _ in range(5):
        x = rng.uniform(0, 1, size=7)
        for k in (2, 3):
            best = None
            for labels in itertools.product(range(k), repeat=7):
                if len(set(labels)) != k:
                    continue
                c = _partition_cost(x, labels)
                if best is None or c < best[0] - 1e-15:
                    best = (c, labels)
            top_label = max(range(k), key=lambda g: np.mean([xi for xi, l in zip(x, best[1]) if l == g]))
            want = np.array([l == top_label for l in best[1]])
            assert (O.cluster_layers(x, k) == want).all()


# -------------------------------------------------------------------- budgets
def test_budget_worked_example_from_paper():
    g = _read_golden("budget_example_appendix_a2.txt")
    n, n_imp = g["n_layer"], g["n_important"]
    cos = np.array([0.7] * n_imp + [0.95] * g["n_unimportant"])
    budgets, is_g3 = O.allocate_budgets(cos, g["b_init"], g["p"], n_cluster=2)
    assert int(is_g3.sum()) == g["n_unimportant"]
    assert (budgets[is_g3] == g["b_unimportant"]).all()
    assert budgets[~is_g3].min() == g["b_important_printed"]
    assert budgets[~is_g3].max() - budgets[~is_g3].min() <= 1
    assert int(budgets.sum()) == g["total"]
    # three clusters (Algorithm 1) with a distinct special group: same two budget classes
    cos3 = np.array([0.6] * 3 + [0.8] * 15 + [0.97] * 14)
    b3, g3 = O.allocate_budgets(cos3, g["b_init"], g["p"], n_cluster=3)
    assert sorted(b3.tolist()) == sorted(budgets.tolist())
    assert g3.tolist() == [False] * 18 + [True] * 14


def test_budget_formula_and_invariants():
    rng = np.random.default_rng(6)
    for _ in range(50):
        n = int(rng.integers(3, 81))
        cos = rng.uniform(0.5, 1.0, size=n)
        b_init = int(rng.integers(1, 5000))
        p = float(rng.choice([0.1, 0.3, 0.35, 0.4, 0.9, 1.0]))
        budgets, is_g3 = O.allocate_budgets(cos, b_init, p)
        assert int(budgets.sum()) == n * b_init                   # total conserved
        assert (budgets >= 1).all()
        n3 = int(is_g3.sum())
        if n3:
            assert 0 < n3 < n
            b_low = max(1, math.floor(b_init * p))
            assert (budgets[is_g3] == b_low).all()
            # Algorithm 1 step 9 with the integer b_low, up to the remainder
            exact = (n * b_init - n3 * b_low) / (n - n3)
            assert np.all(np.abs(budgets[~is_g3] - exact) < 1.0)
            assert budgets[is_g3].max() <= b_init <= budgets[~is_g3].min()
            # G3 holds the largest similarities
            assert cos[is_g3].min() >= cos[~is_g3].max()
            # remainder goes to the lowest-indexed important layers
            imp = budgets[~is_g3]
            assert (np.diff(imp) <= 0).all()
    b, g3 = O.allocate_budgets([0.6, 0.8, 0.99], 100, 1.0)
    assert b.tolist() == [100, 100, 100]
    b, g3 = O.allocate_budgets([0.9, 0.9, 0.9], 100, 0.3)
    assert b.tolist() == [100, 100, 100] and not g3.any()


def test_kv_bytes_per_token_matches_paper():
    g = _read_golden("kv_bytes_section_2_1.txt")
    assert O.kv_bytes_per_token(g["n_layer"], g["d_model"], g["elem_bytes"]) == g["bytes_per_token"]


# ---------------------------------------------------------------------- C_seq
def test_cseq_sliding_window_and_streaming_definitions():
    pos = list(range(100, 140))
    rng = np.random.default_rng(7)
    perm = rng.permutation(40)
    shuffled = [pos[i] for i in perm]
    keep = O.c_seq(O.SLIDING_WINDOW, shuffled, None, 10)
    assert [shuffled[i] for i in keep] == list(range(130, 140))
    keep = O.c_seq(O.STREAMING_LLM, shuffled, None, 10, n_sink=4)
    assert [shuffled[i] for i in keep] == [100, 101, 102, 103] + list(range(134, 140))
    keep = O.c_seq(O.STREAMING_LLM, shuffled, None, 3, n_sink=4)
    assert [shuffled[i] for i in keep] == [100, 101, 102]
    # not over budget: unchanged
    for pol in (O.SLIDING_WINDOW, O.STREAMING_LLM, O.H2O):
        keep = O.c_seq(pol, shuffled, rng.random(40), 40)
        assert [shuffled[i] for i in keep] == pos
        keep = O.c_seq(pol, shuffled, rng.random(40), 64)
        assert [shuffled[i] for i in keep] == pos


def test_cseq_h2o_special_cases():
    rng = np.random.default_rng(8)
    n = 50
    pos = list(range(n))
    acc = rng.random(n)
    # heavy share 0 == sliding window
    keep = O.c_seq(O.H2O, pos, acc, 12, heavy_num=0, heavy_den=1)
    assert keep == list(range(n - 12, n))
    # all scores equal: lower positions win the heavy half
    keep = O.c_seq(O.H2O, pos, np.ones(n), 12, heavy_num=1, heavy_den=2)
    assert keep == list(range(6)) + list(range(n - 6, n))
    # a planted heavy hitter survives, a planted zero does not
    acc2 = acc.copy(); acc2[7] = 100.0; acc2[9] = -1.0
    keep = O.c_seq(O.H2O, pos, acc2, 12)
    assert 7 in keep and 9 not in keep and len(keep) == 12
    # odd budget: floor on the heavy half
    keep = O.c_seq(O.H2O, pos, acc, 13)
    assert len(keep) == 13 and keep[-7:] == list(range(n - 7, n))


def test_cseq_h2o_brute_force_subsets():
    """Among all b_h-subsets of the non-recent tokens, the kept one has the
    largest score sum; among equal sums the lexicographically smallest positions."""
    rng = np.random.default_rng(9)
    for trial in range(40):
        n = int(rng.integers(5, 13))
        b = int(rng.integers(2, n))
        pos = sorted(rng.choice(1000, size=n, replace=False).tolist())
        acc = rng.integers(0, 4, size=n).astype(np.float64) * 0.5      # many ties
        hn, hd = [(1, 2), (1, 3), (2, 3)][trial % 3]
        b_h = (b * hn) // hd
        b_r = b - b_h
        others = list(range(n - b_r))
        best = None
        for sub in itertools.combinations(others, b_h):
            key = (-sum(acc[i] for i in sub), tuple(pos[i] for i in sub))
            if best is None or key < best[0]:
                best = (key, sub)
        want = sorted(list(best[1]) + list(range(n - b_r, n)))
        assert O.c_seq(O.H2O, pos, acc, b, heavy_num=hn, heavy_den=hd) == want


def test_cseq_two_stage_equals_one_shot():
    """Compressing the prompt right after prefill and again after the first
    append keeps the same tokens as Algorithm 1's single compression at the
    first decode step (for H2O the appended token has score 0 and is recent)."""
    rng = np.random.default_rng(10)
    for pol in (O.SLIDING_WINDOW, O.STREAMING_LLM, O.H2O):
        for _ in range(20):
            P = int(rng.integers(8, 60))
            b = int(rng.integers(6, P))
            acc = rng.integers(0, 5, size=P).astype(np.float64)
            pos = list(range(P))
            one = O.c_seq(pol, pos + [P], list(acc) + [0.0], b)
            k1 = O.c_seq(pol, pos, acc, b)
            pos2 = [pos[i] for i in k1] + [P]
            acc2 = [acc[i] for i in k1] + [0.0]
            k2 = O.c_seq(pol, pos2, acc2, b)
            assert [pos2[i] for i in k2] == [(pos + [P])[i] for i in one]


# ------------------------------------------------------------ prefill scores
def test_prefill_scores_against_torch_sdpa_and_invariants():
    rng = np.random.default_rng(11)
    g, P, d = 3, 33, 16
    q = rng.standard_normal((g, P, d))
    k = rng.standard_normal((P, d))
    acc = O.prefill_scores(q, k)
    # library routine: causal SDPA with V = identity returns the attention matrix
    qt = torch.from_numpy(q)[None]
    kt = torch.from_numpy(k)[None, None].expand(1, g, P, d)
    eye = torch.eye(P, dtype=torch.float64)[None, None].expand(1, g, P, P)
    A = torch.nn.functional.scaled_dot_product_attention(qt, kt, eye, is_causal=True)[0]
    want = A.sum(dim=(0, 1)).numpy()
    assert np.allclose(acc, want, atol=1e-12)
    assert acc.sum() == pytest.approx(g * P, abs=1e-10)      # every row sums to one
    assert acc[-1] < 1.0 * g                                   # last column only sees the last row


def test_prefill_scores_uniform_keys_closed_form():
    # identical keys -> every causal row is uniform: acc[t] = g * sum_{r>=t} 1/(r+1)
    g, P, d = 2, 20, 8
    rng = np.random.default_rng(12)
    q = rng.standard_normal((g, P, d))
    k = np.tile(rng.standard_normal(d), (P, 1))
    acc = O.prefill_scores(q, k)
    want = [g * sum(1.0 / (r + 1) for r in range(t, P)) for t in range(P)]
    assert np.allclose(acc, want, atol=1e-12)


# ------------------------------------------------------------------- decoding
def _sdpa_full(q, K, V):
    qt = torch.from_numpy(np.asarray(q, dtype=np.float64))[None, :, None, :]        # [1,g,1,d]
    g = qt.shape[1]
    Kt = torch.from_numpy(np.asarray(K, dtype=np.float64))[None, None].expand(1, g, -1, -1)
    Vt = torch.from_numpy(np.asarray(V, dtype=np.float64))[None, None].expand(1, g, -1, -1)
    return torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt)[0, :, 0, :].numpy()


@pytest.mark.parametrize("policy", [O.SLIDING_WINDOW, O.STREAMING_LLM, O.H2O])
def test_decode_with_large_budget_equals_full_attention(policy):
    rng = np.random.default_rng(13 + policy)
    g, P, d, T = 2, 24, 16, 6
    Kp = rng.standard_normal((P, d)); Vp = rng.standard_normal((P, d))
    Qp = rng.standard_normal((g, P, d))
    u = O.UnitCache(policy, b=P + T)
    u.prefill(Kp, Vp, Qp)
    K, V = Kp.copy(), Vp.copy()
    acc_ref = O.prefill_scores(Qp, Kp) if policy == O.H2O else np.zeros(P)
    for t in range(T):
        q = rng.standard_normal((g, d)); kn = rng.standard_normal(d); vn = rng.standard_normal(d)
        out = u.decode_step(q, kn, vn)
        K = np.vstack([K, kn]); V = np.vstack([V, vn])
        assert np.allclose(out, _sdpa_full(q, K, V), atol=1e-12)
        if policy == O.H2O:
            before = np.append(acc_ref, 0.0)
            gain = np.array(u.acc) - before
            assert gain.sum() == pytest.approx(g, abs=1e-12)      # probabilities sum to one per head
            assert (gain > 0).all()
            acc_ref = np.array(u.acc)
    assert u.kept_positions() == list(range(P + T))


def test_decode_attends_exactly_over_the_kept_set():
    """After compression the output equals library attention restricted to the
    rows the policy definition keeps (sliding window: the last b; streaming:
    sinks + recent)."""
    rng = np.random.default_rng(20)
    g, P, d, T, b = 3, 40, 8, 10, 12
    Kp = rng.standard_normal((P, d)); Vp = rng.standard_normal((P, d))
    for policy in (O.SLIDING_WINDOW, O.STREAMING_LLM):
        u = O.UnitCache(policy, b=b, n_sink=4)
        u.prefill(Kp, Vp)
        K, V = Kp.copy(), Vp.copy()
        for t in range(T):
            q = rng.standard_normal((g, d)); kn = rng.standard_normal(d); vn = rng.standard_normal(d)
            out = u.decode_step(q, kn, vn)
            K = np.vstack([K, kn]); V = np.vstack([V, vn])
            n = K.shape[0]
            rows = list(range(n - b, n)) if policy == O.SLIDING_WINDOW else [0, 1, 2, 3] + list(range(n - (b - 4), n))
            assert u.kept_positions() == rows
            assert np.allclose(out, _sdpa_full(q, K[rows], V[rows]), atol=1e-12)


def test_decode_degenerate_cases():
    rng = np.random.default_rng(21)
    d = 8
    # budget 1: only the new token is left -> out = v_new for every head
    u = O.UnitCache(O.SLIDING_WINDOW, b=1)
    u.prefill(rng.standard_normal((5, d)), rng.standard_normal((5, d)))
    vn = rng.standard_normal(d)
    out = u.decode_step(rng.standard_normal((2, d)), rng.standard_normal(d), vn)
    assert np.allclose(out, np.tile(vn, (2, 1)), atol=0)
    # identical keys -> out = mean of V
    u = O.UnitCache(O.STREAMING_LLM, b=100)
    kk = rng.standard_normal(d)
    Vp = rng.standard_normal((7, d))
    u.prefill(np.tile(kk, (7, 1)), Vp)
    vn = rng.standard_normal(d)
    out = u.decode_step(rng.standard_normal((1, d)), kk, vn)
    assert np.allclose(out[0], np.vstack([Vp, vn]).mean(axis=0), atol=1e-13)
    # one query head per KV head (MHA) is the g = 1 case of the grouped form: two heads run as
    # two separate g = 1 units must give what plain multi-head attention gives, written here as
    # its own loop (full cache, so nothing is evicted) with scipy's softmax
    from scipy.special import softmax
    P, T, H_ = 9, 3, 2
    Kp = rng.standard_normal((H_, P, d)); Vp = rng.standard_normal((H_, P, d)); Qp = rng.standard_normal((H_, P, d))
    units = [O.UnitCache(O.H2O, b=P + T) for _ in range(H_)]
    for h in range(H_):
        units[h].prefill(Kp[h], Vp[h], Qp[h:h + 1])
    Kall = [list(Kp[h]) for h in range(H_)]
    Vall = [list(Vp[h]) for h in range(H_)]
    for t in range(T):
        q = rng.standard_normal((H_, d)); kn = rng.standard_normal((H_, d)); vn2 = rng.standard_normal((H_, d))
        for h in range(H_):
            got = units[h].decode_step(q[h:h + 1], kn[h], vn2[h])
            Kall[h].append(kn[h]); Vall[h].append(vn2[h])
            w_ = softmax(np.array([np.dot(q[h], kr) for kr in Kall[h]]) / np.sqrt(d))
            want = sum(w_[i] * Vall[h][i] for i in range(len(w_)))
            assert got.shape == (1, d) and np.allclose(got[0], want, atol=1e-13)


def test_h2o_trajectory_matches_step_by_step_definition():
    """Free-running H2O: at each step the kept set equals the brute-force
    definition applied to the previous set plus the new token, using scores
    recomputed independently from stored probabilities."""
    rng = np.random.default_rng(22)
    g, P, d, T, b = 2, 30, 8, 12, 10
    Kp = rng.standard_normal((P, d)); Vp = rng.standard_normal((P, d)); Qp = rng.standard_normal((g, P, d))
    u = O.UnitCache(O.H2O, b=b)
    u.prefill(Kp, Vp, Qp)
    scores = dict(zip(range(P), O.prefill_scores(Qp, Kp)))
    kept = set(u.kept_positions())
    assert len(kept) == b
    allK = {t: Kp[t] for t in range(P)}
    for t in range(T):
        q = rng.standard_normal((g, d)); kn = rng.standard_normal(d); vn = rng.standard_normal(d)
        newpos = P + t
        allK[newpos] = kn
        scores[newpos] = 0.0
        cand = sorted(kept | {newpos})
        recent = cand[-(b - b // 2):]
        others = [x for x in cand if x not in recent]
        heavy = sorted(others, key=lambda x: (-scores[x], x))[: b // 2]
        kept = set(heavy) | set(recent)
        u.decode_step(q, kn, vn)
        assert set(u.kept_positions()) == kept
        rows = sorted(kept)
        Km = np.stack([allK[x] for x in rows])
        for h in range(g):
            s = Km @ q[h] / math.sqrt(d)
            pr = torch.softmax(torch.from_numpy(s), dim=0).numpy()
            for x, pv in zip(rows, pr):
                scores[x] += pv
        assert np.allclose([scores[x] for x in rows], u.acc, atol=1e-12)
