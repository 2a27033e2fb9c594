"""GPU parity over the whole stack of the large workloads.

The per-layer head masks of configs 2 and 4 come from one global permutation (the contextual share
differs from layer to layer), so a layer's launch shapes depend on where it sits in the stack.  These
tests build every cache with the workload's real layer count and compare, at every scale, a
deterministic sample of (layer, batch, head) triples spread over the stack plus every head of one
full layer with the CPU oracle (teacher-forced protocol of tests/parity_util.py).  The inputs come
from the seeded generator running on the device; the oracle reads a host copy of the same bytes.
"""
import numpy as np
import pytest
import torch

from workloads import SyntheticQKV, get_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


def _ok(rep):
    assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.problems)
    assert rep.heads_checked > 0
    print(rep.summary())


def _sample(cfg, layers, per_layer, full_layer=None):
    from tests.parity_util import sample_heads
    pairs_of = {l: sample_heads(cfg, l, per_layer) for l in layers}
    if full_layer is not None:
        pairs_of[full_layer] = sample_heads(cfg, full_layer, None)
    return pairs_of


@pytest.mark.parametrize("frac", [0.3, 0.5, 0.7])
def test_config2_triples_over_the_stack(frac):
    """30 layers x 30 heads x batch 8: sampled triples from layers across the stack at every budget of
    the sweep, and all 240 (batch, head) pairs of layer 14 at the smallest budget."""
    from tests.parity_util import run_parity
    cfg = get_config(2, budget_frac=frac)
    pairs_of = _sample(cfg, [3, 11, 19, 27] if frac == 0.3 else [5, 17, 29], 6, 14 if frac == 0.3 else None)
    rep = run_parity(cfg, layers=sorted(pairs_of), fused=True, pairs_of=pairs_of, gen_on_gpu=True,
                     free_running=True)
    _ok(rep)
    assert rep.compressed_heads > 0


def test_config3_triples_over_the_stack_and_one_full_layer():
    """32 layers x 16 heads x batch 2, head_dim 128, 10 521 tokens: triples from four layers and all
    32 (batch, head) pairs of layer 9, every scale."""
    from tests.parity_util import run_parity
    cfg = get_config(3)
    pairs_of = _sample(cfg, [5, 13, 22, 31], 3, 9)
    rep = run_parity(cfg, layers=sorted(pairs_of), fused=True, pairs_of=pairs_of, gen_on_gpu=True,
                     free_running=True)
    _ok(rep)
    assert rep.compressed_heads > 0


@pytest.mark.parametrize("alpha,frac,layer", [
    (0.25, 0.10, 2), (0.25, 0.30, 6), (0.25, 0.50, 11), (0.50, 0.10, 15), (0.50, 0.30, 19),
    (0.50, 0.50, 24), (0.75, 0.10, 28), (0.75, 0.30, 33), (0.75, 0.50, 39)])
def test_config4_every_point_of_the_sweep(alpha, frac, layer):
    """40 layers x 32 heads x batch 2: each of the nine (contextual share, budget) points on a layer of
    its own, so that the nine runs also walk the stack."""
    from tests.parity_util import run_parity
    cfg = get_config(4, budget_frac=frac, alpha=alpha)
    pairs_of = _sample(cfg, [layer], 3)
    rep = run_parity(cfg, layers=[layer], fused=True, pairs_of=pairs_of, gen_on_gpu=True, free_running=True)
    _ok(rep)
    assert rep.compressed_heads > 0


def test_uncompressed_bf16_run_at_full_length_against_the_definition():
    """Budgets = T_K on the 10 521-token schedule (nothing is scored or evicted): the outputs of a
    mid scale and of the last scale against next-scale attention written as its definition (Eq. 3-4:
    one full softmax per query row over every key of the scales so far), a few sampled heads."""
    import paper_2504_09261_b200 as hb
    from oracle import hack_oracle as ho
    from tests.parity_util import OUT_TOL
    cfg = get_config(3, n_layers=1)
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg, device=dev)
    mask = gen.head_is_contextual.numpy()
    t_k = cfg.total_tokens
    cache = hb.HackCache(1, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_BF16, mask, t_k, t_k)
    heads = [(0, 2), (0, 11), (1, 7)]                    # contextual, structural, second batch element
    keys = {bh: [] for bh in heads}
    vals = {bh: [] for bh in heads}
    check_scales = (8, cfg.n_scales - 1)
    sm_scale = 1.0 / np.sqrt(cfg.head_dim)
    worst = 0.0
    for k in range(cfg.n_scales):
        q, kk, v = gen.qkv(0, k)
        out = torch.full_like(q, float("nan"))
        info = cache.hack_step_info(0, k)
        assert not info.triggered_c and not info.triggered_s
        cache.hack_scale_step(0, k, q, kk, v, out)
        torch.cuda.synchronize()
        for (b, h) in heads:
            keys[(b, h)].append(kk[b, h].to(torch.float64).cpu().numpy())
            vals[(b, h)].append(v[b, h].to(torch.float64).cpu().numpy())
        if k in check_scales:
            for (b, h) in heads:
                # a single "scale" whose keys are all keys so far is the definition of this step
                ref = ho.vanilla_var_attention([q[b, h].to(torch.float64).cpu().numpy()],
                                               [np.concatenate(keys[(b, h)], axis=0)],
                                               [np.concatenate(vals[(b, h)], axis=0)], sm_scale)[0]
                d = float(np.max(np.abs(out[b, h].to(torch.float64).cpu().numpy() - ref)))
                worst = max(worst, d)
                assert d <= OUT_TOL["bf16"], f"scale {k} b {b} h {h}: off by {d:.3e}"
    cache.hack_poll_status()
    assert cache.hack_get_lengths(0) == [t_k] * (cfg.batch * cfg.n_heads)
    cache.close()
    print(f"uncompressed bf16, T_K = {t_k}: max |d| = {worst:.3e}")
