"""Host-only checks of the C-ABI library: it loads, exports every symbol include/hack.h declares,
its budget splitter agrees with the hand-derived literals, and argument errors are reported
before any device work (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hb():
    import __graft_entry__ as ge
    ge.build()
    import paper_2504_09261_b200 as pkg
    return pkg


def test_library_exports_every_declared_symbol(hb):
    hdr = open(os.path.join(ROOT, "include", "hack.h")).read()
    declared = set(re.findall(r"HACK_API\s+[\w\s\*]+?\b(hack_\w+)\s*\(", hdr))
    assert declared == set(hb.EXPORTS), declared ^ set(hb.EXPORTS)
    from paper_2504_09261_b200 import binding
    for name in declared:
        assert hasattr(binding.lib, name), name


def _golden_rows(name):
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


@pytest.mark.parametrize("row", _golden_rows("budgets.txt"))
def test_split_budget_matches_hand_derivation(hb, row):
    t_k, alpha, rule, param = int(row[0]), float(row[2]), row[3], float(row[4])
    b, b_c, b_s = int(row[5]), int(row[6]), int(row[7])
    rule_id = hb.RULE_FRACTION if rule == "fraction" else hb.RULE_RATIO
    assert hb.hack_split_budget(b, alpha, rule_id, param, t_k) == (b_c, b_s)


def test_split_budget_rejects_bad_arguments(hb):
    for args in [(100, 0.0, 0, 0.1, 680), (100, 1.0, 0, 0.1, 680), (100, 0.5, 7, 0.1, 680),
                 (0, 0.5, 0, 0.1, 680), (100, 0.5, 1, -2.0, 680)]:
        with pytest.raises(hb.HackError) as e:
            hb.hack_split_budget(*args)
        assert e.value.status == 1
        assert hb.hack_last_error()


def test_init_rejects_bad_configs_before_touching_the_device(hb):
    good = dict(n_layers=1, n_heads=2, head_dim=64, batch=1, sides=(1, 2, 3), dtype=hb.HACK_F32,
                head_is_contextual=[1, 0], budget_c=4, budget_s=8)
    bad = [
        (dict(head_dim=48), 2), (dict(dtype=5), 2), (dict(n_obs=64), 2), (dict(budget_c=0), 1),
        (dict(n_layers=0, head_is_contextual=[]), 1), (dict(sides=(1, 0, 3)), 1),
        (dict(head_is_contextual=[1, 2]), 1), (dict(n_init_scales=9), 1), (dict(overflow_policy=3), 1),
        (dict(sm_scale=-1.0), 1),
    ]
    for change, status in bad:
        kw = dict(good)
        kw.update(change)
        with pytest.raises(hb.HackError) as e:
            hb.HackCache(**kw)
        assert e.value.status == status, (change, e.value)


def test_null_cache_is_an_argument_error(hb):
    from paper_2504_09261_b200 import binding
    assert binding.lib.hack_reset(None) == 1
    assert binding.lib.hack_scale_step(None, 0, 0, None, None, None, None, None) == 1
    assert binding.lib.hack_free_cache(None) == 0
    assert binding.lib.hack_poll_status(None, None) == 1


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2504_09261_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f


def test_classify_heads_matches_the_oracle_rule(hb):
    import numpy as np
    from oracle import hack_oracle as ho
    assert hb.hack_classify_heads([[0.9, 0.1, 0.5], [0.2, 0.8, 0.1]], 2, 3, 0.5) == [[0, 1, 0], [1, 0, 1]]
    assert hb.hack_classify_heads([[0.0, 0.0], [0.0, 0.0]], 2, 2, 0.5) == [[1, 1], [0, 0]]      # ties: (layer, head) order
    rng = np.random.default_rng(11)
    for alpha in (0.0, 0.25, 0.4, 0.5, 0.75, 1.0):
        sigma = rng.lognormal(size=(5, 7))
        sigma[2, 3] = sigma[0, 1]                                                              # a tie across layers
        assert hb.hack_classify_heads(sigma.tolist(), 5, 7, alpha) == ho.classify_heads(sigma, alpha).tolist()
    for bad in (([[0.1, float("nan")]], 1, 2, 0.5), ([[0.1, 0.2]], 1, 2, 1.5), ([[0.1, 0.2]], 1, 2, -0.1)):
        with pytest.raises(hb.HackError) as e:
            hb.hack_classify_heads(*bad)
        assert e.value.status == 1
