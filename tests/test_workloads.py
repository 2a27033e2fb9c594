"""Generator sanity: determinism, shapes, mask ratios, and that the planted attention patterns
show up in the oracle's scores (sinks are selected, structural heads look at the same place)."""
import math

import numpy as np
import torch

from oracle import hack_oracle as ho
from workloads import SyntheticQKV, get_config, list_configs


def test_schedules_and_budget_literals():
    totals = {0: 680, 1: 680, 2: 2240, 3: 10521, 4: 10521}
    for (idx, frac, alpha) in list_configs():
        c = get_config(idx, frac, alpha)
        assert c.total_tokens == totals[idx]
        assert c.budget_total == int(math.floor(frac * c.total_tokens + 1e-9))
        rule, param = ("fraction", 0.05 if frac < 0.5 else 0.10) if c.budget_rule == "var" else ("ratio", 2.0)
        assert ho.split_budget(c.budget_total, alpha, rule, param, c.total_tokens) == (c.budget_c, c.budget_s)


def test_generator_is_deterministic_and_chunk_independent():
    c = get_config(1, n_layers=2)
    g1, g2 = SyntheticQKV(c), SyntheticQKV(c)
    for (layer, scale) in [(0, 0), (1, 4), (1, 9)]:
        a, b = g1.qkv(layer, scale), g2.qkv(layer, scale)
        for x, y in zip(a, b):
            assert x.dtype == torch.bfloat16 and torch.equal(x, y)
            assert x.shape == (c.batch, c.n_heads, c.tokens_per_scale[scale], c.head_dim)
    q0, _, _ = g1.qkv(0, 5)
    q1, _, _ = g1.qkv(1, 5)
    assert not torch.equal(q0, q1)


def test_values_are_standard_normal_where_unmodified():
    c = get_config(3, n_layers=1)
    g = SyntheticQKV(c)
    _, _, v = g.qkv(0, 9, as_float64=True)
    assert abs(v.mean().item()) < 0.01 and abs(v.std().item() - 1.0) < 0.01
    # fourth moment of a normal is 3: catches a broken Box-Muller
    assert abs((v ** 4).mean().item() - 3.0) < 0.1


def test_mask_ratios():
    for idx, alpha in [(1, 0.5), (2, 0.4), (4, 0.25), (4, 0.75)]:
        c = get_config(idx, alpha=alpha, budget_frac=None if idx != 4 else 0.3)
        m = SyntheticQKV(c).head_is_contextual
        assert m.shape == (c.n_layers, c.n_heads)
        assert int(m.sum()) == int(round(alpha * c.n_layers * c.n_heads))
    m = SyntheticQKV(get_config(3)).head_is_contextual
    assert torch.equal(m[:, :8], torch.ones(32, 8, dtype=torch.uint8)) and int(m[:, 8:].sum()) == 0
    # a layer-restricted workload keeps the masks of the layers it keeps
    full = SyntheticQKV(get_config(1)).head_is_contextual
    part = SyntheticQKV(get_config(1, n_layers=3)).head_is_contextual
    assert torch.equal(full[:3], part)


def test_planted_patterns_show_in_oracle_scores():
    """Config 0, all scales: contextual heads keep most of the planted sink keys (far above the
    chance level), every head ends at its budget, and the mean kept length is within B."""
    c = get_config(0)
    g = SyntheticQKV(c)
    mask = g.head_is_contextual.numpy()
    orc = ho.HackOracle(c.n_layers, c.n_heads, c.batch, c.head_dim, c.sides, mask,
                        c.budget_c, c.budget_s)
    sink_pos = {h: [] for h in range(c.n_heads)}
    start = 0
    for k in range(c.n_scales):
        q, kk, v = (t.numpy() for t in g.qkv(0, k, as_float64=True))
        sinks = g.sink_positions(0, k).numpy()
        for h in range(c.n_heads):
            sink_pos[h] += (start + np.nonzero(sinks[h])[0]).tolist()
        start += c.tokens_per_scale[k]
        _, recs = orc.scale_step(0, k, q, kk, v)
    recall = []
    for h in range(c.n_heads):
        rec = recs[(0, h)]
        assert rec.compressed
        if mask[0, h]:
            assert len(rec.pos) == c.budget_c
            recall.append(len(set(sink_pos[h]) & set(rec.pos.tolist())) / len(sink_pos[h]))
        else:
            assert len(rec.pos) == c.budget_s
    # chance level would be B_C / T' ~ 0.1; the planted sinks are found far more often
    assert np.mean(recall) > 0.75, recall
    lens = orc.stored_lengths(0)
    assert lens.mean() <= c.budget_total
