"""Pins for the CPU oracle: each test ties one part of it to something other than itself
(the vanilla definition, a closed form printed in the paper, brute force, an invariant)."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import hack_oracle as ho

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_qkv(rng, b, H, sides, D):
    qs, ks, vs = [], [], []
    for s in sides:
        n = s * s
        qs.append(rng.standard_normal((b, H, n, D)))
        ks.append(rng.standard_normal((b, H, n, D)))
        vs.append(rng.standard_normal((b, H, n, D)))
    return qs, ks, vs


def _run(oracle, qs, ks, vs, layer=0):
    outs, recs = [], []
    for k in range(len(qs)):
        o, r = oracle.scale_step(layer, k, qs[k], ks[k], vs[k])
        outs.append(o)
        recs.append(r)
    return outs, recs


# ------------------------------------------------------------------ P1: full budget == vanilla
def test_full_budget_reproduces_vanilla_attention():
    """With B_C = B_S >= T_K nothing is ever evicted, so every scale's output must equal
    uncompressed next-scale attention over all scales <= k (Eq. 3-4)."""
    rng = np.random.default_rng(1)
    sides, b, H, D = (1, 2, 3, 4, 5), 2, 3, 8
    qs, ks, vs = _rand_qkv(rng, b, H, sides, D)
    T = sum(s * s for s in sides)
    mask = np.array([[1, 0, 1]])
    orc = ho.HackOracle(1, H, b, D, sides, mask, budget_c=T, budget_s=T)
    outs, recs = _run(orc, qs, ks, vs)
    for bb in range(b):
        for h in range(H):
            ref = ho.vanilla_var_attention([q[bb, h] for q in qs], [k[bb, h] for k in ks],
                                           [v[bb, h] for v in vs], 1.0 / math.sqrt(D))
            for k in range(len(sides)):
                np.testing.assert_allclose(outs[k][bb, h], ref[k], rtol=1e-12, atol=1e-13)
                assert not recs[k][(bb, h)].compressed
    assert orc.counters.score_pairs == 0


def test_trigger_is_strict():
    """Compression starts only when the candidate count EXCEEDS the budget (T' > B)."""
    rng = np.random.default_rng(2)
    sides, D = (1, 2, 3), 4                      # T = 1, 5, 14
    qs, ks, vs = _rand_qkv(rng, 1, 1, sides, D)
    orc = ho.HackOracle(1, 1, 1, D, sides, np.array([[1]]), budget_c=5, budget_s=5)
    _, recs = _run(orc, qs, ks, vs)
    assert [r[(0, 0)].compressed for r in recs] == [False, False, True]
    assert [len(r[(0, 0)].keep) for r in recs] == [1, 5, 5]


# ------------------------------------------------------------------ P2: softmax rows sum to one
def test_scores_sum_to_number_of_observation_rows():
    rng = np.random.default_rng(3)
    for n_obs, t in [(1, 7), (5, 33), (32, 500)]:
        q = rng.standard_normal((n_obs, 16)) * 3
        k = rng.standard_normal((t, 16)) * 3
        s = ho.subset_attention_scores(q, k, 0.25)
        assert s.shape == (t,)
        assert np.all(s >= 0)
        assert abs(s.sum() - n_obs) < 1e-10


def test_scores_match_elementwise_definition():
    """s_j = sum_i exp(z_ij) / sum_j' exp(z_ij') written out with scalar loops."""
    rng = np.random.default_rng(4)
    q = rng.standard_normal((3, 5))
    k = rng.standard_normal((6, 5))
    sm = 0.7
    s = ho.subset_attention_scores(q, k, sm)
    ref = np.zeros(6)
    for i in range(3):
        z = [sm * sum(q[i, d] * k[j, d] for d in range(5)) for j in range(6)]
        den = sum(math.exp(x) for x in z)
        for j in range(6):
            ref[j] += math.exp(z[j]) / den
    np.testing.assert_allclose(s, ref, rtol=1e-12)


def test_observation_rows_uniform_and_complete():
    assert list(ho.observation_rows(4, 32)) == [0, 1, 2, 3]          # all queries when N_k <= N_obs
    assert list(ho.observation_rows(64, 32)) == list(range(0, 64, 2))
    r = ho.observation_rows(100, 32)
    assert len(r) == 32 and r[0] == 0 and len(set(r)) == 32 and np.all(np.diff(r) >= 3)
    assert r[-1] < 100


def test_observation_rows_of_the_ablation_samplers():
    """Query-subset ablation: first n, last n, caller-drawn rows; every rule degenerates to all
    rows when the scale has no more than N_obs tokens."""
    assert list(ho.observation_rows(10, 4, ho.UNIFORM)) == [0, 2, 5, 7]
    assert list(ho.observation_rows(10, 4, ho.INIT)) == [0, 1, 2, 3]
    assert list(ho.observation_rows(10, 4, ho.RECENT)) == [6, 7, 8, 9]
    assert list(ho.observation_rows(10, 4, ho.CALLER, [9, 0, 4, 3])) == [9, 0, 4, 3]
    for sampler in (ho.UNIFORM, ho.INIT, ho.RECENT):
        assert list(ho.observation_rows(9, 32, sampler)) == list(range(9))
    for bad in ([0, 1, 2], [0, 1, 2, 2], [0, 1, 2, 10], [-1, 1, 2, 3]):
        with pytest.raises(ValueError):
            ho.observation_rows(10, 4, ho.CALLER, bad)
    assert list(ho.observation_rows(10, 4, ho.FULL)) == list(range(10))


def test_full_query_set_scores_are_the_column_sums_of_the_attention_matrix():
    """With every query observing, a contextual step keeps the keys with the largest column sums of
    the step's whole attention matrix (computed here with explicit loops)."""
    rng = np.random.default_rng(12)
    D, n_k = 6, 9
    q, k, v = rng.normal(size=(n_k, D)), rng.normal(size=(n_k, D)), rng.normal(size=(n_k, D))
    col = [0.0] * n_k
    for i in range(n_k):
        z = [sum(q[i, t] * k[j, t] for t in range(D)) / math.sqrt(D) for j in range(n_k)]
        den = sum(math.exp(x) for x in z)
        for j in range(n_k):
            col[j] += math.exp(z[j]) / den
    orc = ho.HackOracle(1, 1, 1, D, (3,), np.array([[1]]), budget_c=4, budget_s=4, n_obs=2, obs_sampler=ho.FULL)
    _, rec = orc.head_step(0, 0, 0, 0, q, k, v)
    np.testing.assert_allclose(rec.scores, col, rtol=1e-12)
    assert list(rec.keep) == sorted(sorted(range(n_k), key=lambda j: -col[j])[:4])


def test_sampler_decides_which_key_a_contextual_head_keeps():
    """Two planted keys: the first half of the queries looks at key 0, the second half at key 1.
    With one slot for old entries, the first-n rule keeps key 0, the last-n rule key 1, and caller
    rows taken from one half or the other reproduce the two; computed against a direct column sum."""
    D, n_k = 8, 16
    rng = np.random.default_rng(5)
    e0, e1 = np.eye(D)[0] * 6.0, np.eye(D)[1] * 6.0
    k_new = rng.normal(size=(n_k, D)) * 0.05
    k_new[0], k_new[1] = e0, e1
    q = rng.normal(size=(n_k, D)) * 0.05
    q[: n_k // 2] += e0
    q[n_k // 2:] += e1
    v = rng.normal(size=(n_k, D))
    for sampler, rows, expect in ((ho.INIT, None, 0), (ho.RECENT, None, 1),
                                  (ho.CALLER, [[3, 1, 6, 0]], 0), (ho.CALLER, [[15, 9, 12, 10]], 1)):
        orc = ho.HackOracle(1, 1, 1, D, (4,), np.array([[1]]), budget_c=1, budget_s=1, n_obs=4,
                            obs_sampler=sampler, obs_rows=rows)
        _, res = orc.head_step(0, 0, 0, 0, q, k_new, v)
        used = ho.observation_rows(n_k, 4, sampler, rows[0] if rows else None)
        z = (q[used] @ k_new.T) / math.sqrt(D)
        a = np.exp(z - z.max(axis=1, keepdims=True))
        a /= a.sum(axis=1, keepdims=True)
        assert int(np.argmax(a.sum(axis=0))) == expect
        assert list(res.keep) == [expect]


def test_caller_rows_order_does_not_change_scores():
    rng = np.random.default_rng(6)
    q, k = rng.normal(size=(40, 16)), rng.normal(size=(70, 16))
    rows = [31, 2, 17, 8, 25]
    s1 = ho.subset_attention_scores(q[ho.observation_rows(40, 5, ho.CALLER, rows)], k, 0.25)
    s2 = ho.subset_attention_scores(q[ho.observation_rows(40, 5, ho.CALLER, sorted(rows))], k, 0.25)
    np.testing.assert_allclose(s1, s2, rtol=1e-13)


# ------------------------------------------------------------------ P3: brute-force selection
def _best_subset_exhaustive(s, n):
    """argmax-n subset by exhaustive enumeration; among equal sums the lexicographically
    smallest index tuple wins (= ties go to lower indices)."""
    best, best_sum = None, -1.0
    for comb in itertools.combinations(range(len(s)), n):
        tot = sum(s[list(comb)])
        if tot > best_sum + 1e-15:
            best, best_sum = comb, tot
    return np.array(best, dtype=np.int64)


def test_contextual_selection_is_argmax_subset():
    rng = np.random.default_rng(5)
    for t, n in [(6, 2), (8, 3), (9, 8), (10, 1)]:
        s = rng.random(t)
        np.testing.assert_array_equal(ho.select_contextual(s, n), _best_subset_exhaustive(s, n))


def test_contextual_selection_matches_sort_definition():
    rng = np.random.default_rng(6)
    s = np.round(rng.random(200), 2)             # many ties
    for n in (1, 17, 100, 199, 200, 500):
        keep = ho.select_contextual(s, n)
        ranked = sorted(range(200), key=lambda j: (-s[j], j))[: min(n, 200)]
        np.testing.assert_array_equal(keep, np.array(sorted(ranked)))


def test_all_scores_tie_keeps_lowest_indices():
    """Constant queries make every logit equal, so all scores tie and the lowest indices win."""
    k = np.random.default_rng(7).standard_normal((40, 8))
    q = np.zeros((32, 8))
    s = ho.subset_attention_scores(q, k, 0.3)
    np.testing.assert_allclose(s, 32 / 40)
    np.testing.assert_array_equal(ho.select_contextual(s, 11), np.arange(11))


# ------------------------------------------------------------------ P4/P5/P10: structural rule
def test_structural_keeps_initial_and_latest_scales():
    rng = np.random.default_rng(8)
    sides, D = (1, 2, 3, 4, 5, 6), 8            # N = 1,4,9,16,25,36 ; T = 1,5,14,30,55,91
    qs, ks, vs = _rand_qkv(rng, 1, 2, sides, D)
    mask = np.array([[0, 1]])
    b_s, b_c = 50, 12
    orc = ho.HackOracle(1, 2, 1, D, sides, mask, budget_c=b_c, budget_s=b_s)
    starts = np.concatenate([[0], np.cumsum([s * s for s in sides])])
    seen_evicted = [set(), set()]
    prev_pos = [np.zeros(0, np.int64)] * 2
    for k in range(len(sides)):
        n_k = sides[k] ** 2
        _, recs = orc.scale_step(0, k, qs[k], ks[k], vs[k])
        for h in (0, 1):
            pos = recs[(0, h)].pos
            assert np.all(np.diff(pos) > 0)                          # ascending, unique
            cand = set(prev_pos[h].tolist()) | set(range(starts[k], starts[k + 1]))
            assert set(pos.tolist()) <= cand                         # only candidates survive
            assert not (set(pos.tolist()) & seen_evicted[h])         # evicted never returns
            seen_evicted[h] |= cand - set(pos.tolist())
            prev_pos[h] = pos
        pos_s = set(recs[(0, 0)].pos.tolist())
        assert set(range(0, min(5, starts[k + 1]))) <= pos_s         # scales 1-2 (5 tokens)
        assert set(range(starts[k], starts[k + 1])) <= pos_s         # latest scale
        t_cand = recs[(0, 0)].n_candidates
        n_prot = min(5, starts[k + 1]) + (n_k if k >= 2 else 0)
        assert len(pos_s) == min(t_cand, max(b_s, n_prot))
        assert len(recs[(0, 1)].pos) == min(recs[(0, 1)].n_candidates, b_c)
    assert orc.counters.overflows == 0


def test_structural_zero_free_budget_keeps_exactly_protected():
    """B_S = N_init + N_k  (M = 0)  =>  kept = first two scales + current scale, nothing else."""
    s = np.random.default_rng(9).random(5 + 9 + 16)
    sid = np.array([1] + [2] * 4 + [3] * 9 + [4] * 16)
    keep = ho.select_structural(s, sid, 4, 2, 5 + 16)
    np.testing.assert_array_equal(keep, np.concatenate([np.arange(5), np.arange(14, 30)]))


def test_structural_free_slots_filled_by_score():
    s = np.array([9, 9, 9, 9, 9, .1, .5, .3, .5, .2, 9, 9, 9], dtype=float)
    sid = np.array([1, 2, 2, 2, 2, 3, 3, 3, 3, 3, 4, 4, 4])
    keep = ho.select_structural(s, sid, 4, 2, 5 + 3 + 2)
    np.testing.assert_array_equal(keep, [0, 1, 2, 3, 4, 6, 8, 10, 11, 12])   # ties -> lower index
    keep = ho.select_structural(s, sid, 4, 2, 5 + 3 + 3)
    np.testing.assert_array_equal(keep, [0, 1, 2, 3, 4, 6, 7, 8, 10, 11, 12])


def test_structural_overflow_policies():
    """B_S smaller than the protected set: policy 0 keeps all protected entries (more than B_S),
    policy 1 lets the current scale compete and keeps exactly B_S."""
    rng = np.random.default_rng(10)
    s = rng.random(5 + 9 + 16)
    sid = np.array([1] + [2] * 4 + [3] * 9 + [4] * 16)
    keep0 = ho.select_structural(s, sid, 4, 2, 12, ho.KEEP_PROTECTED)
    np.testing.assert_array_equal(keep0, np.concatenate([np.arange(5), np.arange(14, 30)]))
    keep1 = ho.select_structural(s, sid, 4, 2, 12, ho.COMPETE)
    assert len(keep1) == 12 and set(range(5)) <= set(keep1.tolist())
    rest = np.array(sorted(set(keep1.tolist()) - set(range(5))))
    ranked = sorted(range(5, 30), key=lambda j: (-s[j], j))[:7]
    np.testing.assert_array_equal(rest, sorted(ranked))


# ------------------------------------------------------------------ P6: compaction copies rows
def test_stored_rows_are_bit_copies_of_inputs():
    rng = np.random.default_rng(11)
    sides, D = (1, 2, 3, 4, 5), 4
    qs, ks, vs = _rand_qkv(rng, 1, 2, sides, D)
    orc = ho.HackOracle(1, 2, 1, D, sides, np.array([[1, 0]]), budget_c=9, budget_s=30)
    _run(orc, qs, ks, vs)
    k_all = np.concatenate([k[0] for k in ks], axis=1)
    v_all = np.concatenate([v[0] for v in vs], axis=1)
    for h in range(2):
        st = orc.state[0][0][h]
        assert np.array_equal(st.k, k_all[h][st.pos])
        assert np.array_equal(st.v, v_all[h][st.pos])
        assert np.all(np.diff(st.pos) > 0)
    assert orc.state[0][0][0].k.shape[0] == 9


# ------------------------------------------------------------------ P7: attention properties
def test_attention_is_convex_combination_and_permutation_invariant():
    rng = np.random.default_rng(12)
    q = rng.standard_normal((7, 8)) * 2
    k = rng.standard_normal((19, 8))
    v = rng.standard_normal((19, 8))
    o = ho.attend(q, k, v, 0.35)
    assert np.all(o <= v.max(axis=0) + 1e-12) and np.all(o >= v.min(axis=0) - 1e-12)
    perm = rng.permutation(19)
    np.testing.assert_allclose(ho.attend(q, k[perm], v[perm], 0.35), o, rtol=1e-12, atol=1e-14)
    # one key only -> output is that key's value; identical keys -> mean of values
    np.testing.assert_allclose(ho.attend(q, k[:1], v[:1], 0.35), np.repeat(v[:1], 7, axis=0))
    np.testing.assert_allclose(ho.attend(q, np.repeat(k[:1], 19, axis=0), v, 0.35),
                               np.repeat(v.mean(axis=0, keepdims=True), 7, axis=0), rtol=1e-12)


def test_attention_scale_and_transpose_sensitivity():
    """A dominant logit pins the output to one value row: catches a dropped sm_scale, a
    transposed operand or a sign error."""
    D = 4
    k = np.eye(D)[:3] * 50.0                      # three orthogonal keys
    v = np.array([[1., 0, 0, 0], [0, 2., 0, 0], [0, 0, 3., 0]])
    q = np.array([[0, 1., 0, 0]])                 # matches key 1
    o = ho.attend(q, k, v, 1.0)
    np.testing.assert_allclose(o, v[1:2], atol=1e-12)
    o_small = ho.attend(q, k, v, 1e-9)            # scale -> 0 gives the plain mean
    np.testing.assert_allclose(o_small, v.mean(axis=0, keepdims=True), atol=1e-6)


# ------------------------------------------------------------------ P8: complexity closed forms
def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


@pytest.mark.parametrize("row", _golden_rows("complexity_closed_forms.txt"))
def test_counters_match_closed_forms(row):
    a, K, t_final, total_pairs = (int(x) for x in row)
    sides = tuple(a ** k for k in range(K))
    D = 2
    rng = np.random.default_rng(13)
    qs, ks, vs = _rand_qkv(rng, 1, 1, sides, D)
    # full cache: attention pairs = sum N_k T_k  (Eq. 15-17), T_K = Eq. 14
    T = sum(s * s for s in sides)
    assert T == t_final == (a ** (2 * K) - 1) // (a * a - 1)
    orc = ho.HackOracle(1, 1, 1, D, sides, np.array([[1]]), budget_c=T, budget_s=T)
    _run(orc, qs, ks, vs)
    assert orc.counters.attention_pairs == total_pairs
    num = 1 - a ** (2 * K) - a ** (2 * K + 2) + a ** (4 * K + 2)
    den = (a * a - 1) ** 2 * (a * a + 1)
    assert num % den == 0 and num // den == total_pairs
    # budgeted: pairs = sum N_k min(T_k, B) <= B sum N_k (Eq. 12 / 18-21); overhead bound Eq. 13 / 22
    for B in (3, 7, max(T // 3, 1)):
        orc = ho.HackOracle(1, 1, 1, D, sides, np.array([[1]]), budget_c=B, budget_s=B, n_obs=4)
        _run(orc, qs, ks, vs)
        n = [s * s for s in sides]
        t_k = np.cumsum(n)
        assert orc.counters.attention_pairs == sum(nk * min(tk, B) for nk, tk in zip(n, t_k))
        assert orc.counters.attention_pairs <= B * sum(n)
        k_s = next((i for i, tk in enumerate(t_k) if tk > B), None)
        if k_s is not None:
            assert orc.counters.score_pairs <= sum(4 * (B + nk) for nk in n[k_s:])
            assert orc.counters.score_pairs > 0


# ------------------------------------------------------------------ P9: f_C against a 10-line brute force
def test_contextual_step_equals_full_column_sum_topk():
    """All heads contextual and N_obs >= N_k: the kept set is the top-B of the column sums of the
    FULL attention matrix of the step, computed here from scratch."""
    rng = np.random.default_rng(14)
    sides, D, B = (1, 2, 3, 4), 6, 11
    qs, ks, vs = _rand_qkv(rng, 1, 1, sides, D)
    orc = ho.HackOracle(1, 1, 1, D, sides, np.array([[1]]), budget_c=B, budget_s=B, n_obs=64)
    kept_pos = np.zeros(0, dtype=np.int64)
    k_all = np.concatenate([k[0, 0] for k in ks])
    start = 0
    for k in range(len(sides)):
        n_k = sides[k] ** 2
        cand = np.concatenate([kept_pos, np.arange(start, start + n_k)])
        start += n_k
        if len(cand) > B:
            logits = (qs[k][0, 0] @ k_all[cand].T) / math.sqrt(D)
            A = np.exp(logits - logits.max(1, keepdims=True))
            A /= A.sum(1, keepdims=True)
            col = A.sum(0)
            kept_pos = np.sort(cand[sorted(range(len(cand)), key=lambda j: (-col[j], j))[:B]])
        else:
            kept_pos = cand
        _, recs = orc.scale_step(0, k, qs[k], ks[k], vs[k])
        np.testing.assert_array_equal(recs[(0, 0)].pos, kept_pos)


# ------------------------------------------------------------------ budgets (Eq. 7)
@pytest.mark.parametrize("row", _golden_rows("budgets.txt"))
def test_budget_split_matches_hand_derivation(row):
    t_k, frac, alpha, rule, param = int(row[0]), float(row[1]), float(row[2]), row[3], float(row[4])
    b, b_c, b_s = int(row[5]), int(row[6]), int(row[7])
    assert int(math.floor(frac * t_k + 1e-9)) == b
    assert ho.split_budget(b, alpha, rule, param, t_k) == (b_c, b_s)
    if b_s < t_k:
        assert alpha * b_c + (1 - alpha) * b_s <= b + 1e-9           # Eq. 7 as an upper bound


def test_mean_kept_length_within_budget():
    """No overflow => the stack-mean kept length never exceeds B (Eq. 7)."""
    rng = np.random.default_rng(15)
    sides, D, H = (1, 2, 3, 4, 5, 6, 7), 4, 4       # T_K = 140
    T = sum(s * s for s in sides)
    B = int(0.5 * T)
    alpha = 0.5
    b_c, b_s = ho.split_budget(B, alpha, "fraction", 0.1, T)
    qs, ks, vs = _rand_qkv(rng, 1, H, sides, D)
    orc = ho.HackOracle(1, H, 1, D, sides, np.array([[1, 0, 1, 0]]), budget_c=b_c, budget_s=b_s)
    for k in range(len(sides)):
        orc.scale_step(0, k, qs[k], ks[k], vs[k])
        assert orc.stored_lengths(0).mean() <= B
    assert orc.counters.overflows == 0
    assert orc.counters.peak_entries == orc.stored_lengths(0).sum()


# ------------------------------------------------------------------ Eq. 6: attention variance
def test_attention_variance_closed_forms():
    """Uniform attention has no column variance; attention that is (nearly) a permutation matrix has
    sigma = T * (1/N)(1 - 1/N) = 1 - 1/N for N = T; identical query rows give zero whatever the keys."""
    n, d = 12, 12
    k = np.eye(d) * 200.0                      # query i = key i: softmax row i is one-hot to 1e-80
    assert ho.attention_variance(np.eye(d), k, 1.0) == pytest.approx(1.0 - 1.0 / n, rel=1e-12)
    assert ho.attention_variance(np.zeros((n, d)), k, 1.0) == pytest.approx(0.0, abs=1e-30)
    rng = np.random.default_rng(3)
    q1 = np.repeat(rng.normal(size=(1, d)), n, axis=0)
    assert ho.attention_variance(q1, rng.normal(size=(30, d)), 0.3) == pytest.approx(0.0, abs=1e-30)


def test_attention_variance_matches_loops():
    rng = np.random.default_rng(4)
    q, k = rng.normal(size=(7, 5)), rng.normal(size=(9, 5))
    a = np.zeros((7, 9))
    for i in range(7):
        z = [0.4 * sum(q[i, t] * k[j, t] for t in range(5)) for j in range(9)]
        den = sum(math.exp(x) for x in z)
        for j in range(9):
            a[i, j] = math.exp(z[j]) / den
    sigma = 0.0
    for j in range(9):
        mean = sum(a[i, j] for i in range(7)) / 7
        sigma += sum((a[i, j] - mean) ** 2 for i in range(7)) / 7
    assert ho.attention_variance(q, k, 0.4) == pytest.approx(sigma, rel=1e-12)
    # transposing the roles of rows and columns is a different number (variance over queries, not keys)
    assert abs(float(np.var(a, axis=1).sum()) - sigma) > 1e-3


def test_classify_heads_ranks_globally():
    sigma = np.array([[0.9, 0.1, 0.5], [0.2, 0.8, 0.1]])
    assert ho.classify_heads(sigma, 0.5).tolist() == [[0, 1, 0], [1, 0, 1]]
    assert ho.classify_heads(sigma, 1 / 3).tolist() == [[0, 1, 0], [0, 0, 1]]     # per-layer ratio varies
    assert ho.classify_heads(np.zeros((2, 2)), 0.5).tolist() == [[1, 1], [0, 0]]   # ties: (layer, head) order


def test_variance_ranking_recovers_the_planted_head_types():
    """The synthetic workloads plant vertical patterns in contextual heads and position-following
    ones in structural heads; Eq. 6 on the last scale's full attention matrix must separate them."""
    from workloads import SyntheticQKV, get_config
    cfg = get_config(0, n_layers=2)
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy().astype(np.uint8)
    sigma = np.zeros((cfg.n_layers, cfg.n_heads))
    last = cfg.n_scales - 1
    for l in range(cfg.n_layers):
        ks = [gen.qkv(l, s)[1].double().numpy() for s in range(cfg.n_scales)]
        q = gen.qkv(l, last)[0].double().numpy()
        for h in range(cfg.n_heads):
            k_all = np.concatenate([x[0, h] for x in ks], axis=0)
            sigma[l, h] = ho.attention_variance(q[0, h], k_all, 1.0 / math.sqrt(cfg.head_dim))
    alpha = float(mask.mean())
    assert ho.classify_heads(sigma, alpha).tolist() == mask.tolist()
    assert sigma[mask == 1].max() < sigma[mask == 0].min()


# ------------------------------------------------------------------ final-scale merge (a reading; see the oracle's header)
def test_merge_special_cases():
    """What the reading fixes by itself: a discarded entry identical to a retained one is averaged in
    with weight 1; one orthogonal or opposed to every retained key changes nothing; retained entries
    without assignments keep their bits; equal similarities go to the lowest index."""
    k_kept = np.array([[1.0, 0.0, 0.0], [0.0, 2.0, 0.0], [0.0, 2.0, 0.0]])
    v_kept = np.array([[1.0, 1.0, 1.0], [2.0, 2.0, 2.0], [3.0, 3.0, 3.0]])
    k_ev = np.array([[3.0, 0.0, 0.0], [0.0, 0.0, 5.0], [-1.0, -1.0, 0.0], [0.0, 1.0, 0.0]])
    v_ev = np.array([[5.0, 5.0, 5.0], [9.0, 9.0, 9.0], [7.0, 7.0, 7.0], [4.0, 4.0, 4.0]])
    assign, weight = ho.merge_assign(k_ev, k_kept)
    assert assign.tolist()[0] == 0 and weight[0] == pytest.approx(1.0)
    assert weight[1] == 0.0 and weight[2] == 0.0
    assert assign.tolist()[3] == 1 and weight[3] == pytest.approx(1.0)       # tie between kept 1 and 2: lowest index
    k_m, v_m = ho.merge_apply(k_kept, v_kept, k_ev, v_ev, assign, weight)
    np.testing.assert_allclose(k_m[0], [2.0, 0.0, 0.0])                      # (k_c + 1 * k_e) / 2
    np.testing.assert_allclose(v_m[0], [3.0, 3.0, 3.0])
    np.testing.assert_allclose(k_m[1], [0.0, 1.5, 0.0])
    np.testing.assert_allclose(v_m[1], [3.0, 3.0, 3.0])
    assert np.array_equal(k_m[2], k_kept[2]) and np.array_equal(v_m[2], v_kept[2])


def test_merge_matches_loops_and_stays_in_the_hull():
    rng = np.random.default_rng(8)
    k_kept, v_kept = rng.normal(size=(6, 5)), rng.normal(size=(6, 5))
    k_ev, v_ev = rng.normal(size=(11, 5)), rng.normal(size=(11, 5))
    assign, weight = ho.merge_assign(k_ev, k_kept)
    k_m, v_m = ho.merge_apply(k_kept, v_kept, k_ev, v_ev, assign, weight)
    for c in range(6):
        num_k, num_v, den = list(k_kept[c]), list(v_kept[c]), 1.0
        for e in range(11):
            best, best_c = -2.0, -1
            for cc in range(6):
                dot = sum(k_ev[e, t] * k_kept[cc, t] for t in range(5))
                cos = dot / math.sqrt(sum(x * x for x in k_ev[e]) * sum(x * x for x in k_kept[cc]))
                if cos > best:
                    best, best_c = cos, cc
            if best_c == c and best > 0:
                for t in range(5):
                    num_k[t] += best * k_ev[e, t]
                    num_v[t] += best * v_ev[e, t]
                den += best
        np.testing.assert_allclose(k_m[c], np.array(num_k) / den, rtol=1e-12)
        np.testing.assert_allclose(v_m[c], np.array(num_v) / den, rtol=1e-12)
    both = np.concatenate([v_kept, v_ev])
    assert np.all(v_m >= both.min(axis=0) - 1e-12) and np.all(v_m <= both.max(axis=0) + 1e-12)


def test_merge_runs_only_at_the_last_scale_of_contextual_heads():
    rng = np.random.default_rng(9)
    sides, D = (1, 2, 3, 4), 8
    mask = np.array([[1, 0]])
    plain = ho.HackOracle(1, 2, 1, D, sides, mask, budget_c=6, budget_s=30)
    merged = ho.HackOracle(1, 2, 1, D, sides, mask, budget_c=6, budget_s=30, merge_last=True)
    for k, side in enumerate(sides):
        n = side * side
        q, kk, v = (rng.normal(size=(1, 2, n, D)) for _ in range(3))
        o_p, rec_p = plain.scale_step(0, k, q, kk, v)
        o_m, rec_m = merged.scale_step(0, k, q, kk, v)
        last = k == len(sides) - 1
        assert (rec_m[(0, 0)].merge_assign is not None) == last and rec_m[(0, 1)].merge_assign is None
        assert np.array_equal(rec_p[(0, 0)].keep, rec_m[(0, 0)].keep)           # the selection is the same
        if last:
            rec = rec_m[(0, 0)]
            assert len(rec.evicted) + len(rec.keep) == rec.n_candidates
            assert not np.allclose(o_p[0, 0], o_m[0, 0]) and np.array_equal(o_p[0, 1], o_m[0, 1])
        else:
            assert np.array_equal(o_p, o_m)
