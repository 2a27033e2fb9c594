"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

from workloads import get_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


def _assert_ok(rep):
    assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.problems)
    assert rep.heads_checked > 0


def test_config0_fp32_all_scales_all_heads():
    """Single layer, fp32, every scale compared (heads start compressing at scale 5)."""
    from tests.parity_util import run_parity
    rep = run_parity(get_config(0), layers=[0], fused=True)
    _assert_ok(rep)
    assert rep.compressed_heads > 0
    assert rep.max_out_abs <= 1e-5 and rep.max_score_err <= 1.0


def test_config1_bf16_two_layers():
    from tests.parity_util import run_parity
    rep = run_parity(get_config(1, n_layers=2), layers=[0, 1], fused=True, heads_per_layer=64)
    _assert_ok(rep)
    assert rep.compressed_heads > 0


@pytest.mark.parametrize("frac", [0.3, 0.5, 0.7])
def test_config2_bf16_budget_sweep_sampled_heads(frac):
    from tests.parity_util import run_parity
    rep = run_parity(get_config(2, budget_frac=frac, n_layers=1), layers=[0], fused=True,
                     heads_per_layer=12)
    _assert_ok(rep)


def test_config3_bf16_head_dim_128_sampled_heads():
    """Full 13-scale 1024^2 schedule at full size, one layer, sampled (batch, head) pairs."""
    from tests.parity_util import run_parity
    rep = run_parity(get_config(3, n_layers=1), layers=[0], fused=True, heads_per_layer=6)
    _assert_ok(rep)
    assert rep.compressed_heads > 0


def test_config4_overflow_policies():
    """Smallest budget of the wide sweep: B_S < N_init + N_k at the last scales (both rules)."""
    from tests.parity_util import run_parity
    cfg = get_config(4, budget_frac=0.10, alpha=0.25, n_layers=1)
    for policy in (0, 1):
        rep = run_parity(cfg, layers=[0], fused=True, heads_per_layer=4, policy=policy)
        _assert_ok(rep)


def test_full_budget_equals_uncompressed_attention():
    """B_C = B_S = T_K: nothing is scored or evicted; output is vanilla next-scale attention."""
    from tests.parity_util import run_parity
    cfg = get_config(0)
    rep = run_parity(cfg, layers=[0], fused=True, budget_c=cfg.total_tokens, budget_s=cfg.total_tokens)
    _assert_ok(rep)
    assert rep.compressed_heads == 0


def test_tiny_budgets_and_ties():
    """Budget 1 for contextual heads, budget below the protected set for structural heads."""
    from tests.parity_util import run_parity
    rep = run_parity(get_config(0), layers=[0], fused=True, budget_c=1, budget_s=3)
    _assert_ok(rep)
    rep = run_parity(get_config(0), layers=[0], fused=True, budget_c=1, budget_s=3, policy=1)
    _assert_ok(rep)


def test_state_machine_and_argument_errors():
    import paper_2504_09261_b200 as hb
    from tests.parity_util import make_cache
    from workloads import SyntheticQKV
    cfg = get_config(0)
    gen = SyntheticQKV(cfg)
    cache = make_cache(cfg, gen.head_is_contextual.numpy())
    q, k, v = (t.cuda() for t in gen.qkv(0, 0))
    out = torch.empty_like(q)
    with pytest.raises(hb.HackError) as e:
        cache.hack_scale_step(0, 1, q, k, v, out)          # scale 0 has not run yet
    assert e.value.status == 5
    with pytest.raises(hb.HackError) as e:
        cache.hack_attend(0, 0, q, out)                    # compaction must come first
    assert e.value.status == 5
    with pytest.raises(hb.HackError) as e:
        cache.hack_scale_step(0, 0, q, None, v, out)
    assert e.value.status == 1
    with pytest.raises(hb.HackError) as e:
        cache.hack_scale_step(3, 0, q, k, v, out)
    assert e.value.status == 1
    with pytest.raises(hb.HackError) as e:
        cache.hack_scale_step(0, 0, q.data_ptr() + 4, k, v, out)   # misaligned
    assert e.value.status == 1
    cache.hack_scale_step(0, 0, q, k, v, out)
    torch.cuda.synchronize()
    assert cache.hack_get_lengths(0) == [1] * cfg.n_heads
    live, peak, reserved = cache.hack_kv_bytes()
    assert live == cfg.n_heads * 1 * cfg.head_dim * 4 * 2 and peak == live and reserved > live
    assert cache.hack_launch_count() >= 1
    cache.hack_reset()
    assert cache.hack_get_lengths(0) == [0] * cfg.n_heads
    cache.hack_scale_step(0, 0, q, k, v, out)
    cache.hack_poll_status()
    cache.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    from tests.parity_util import make_cache
    from workloads import SyntheticQKV
    cfg = get_config(1, n_layers=1)
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    a, b = make_cache(cfg, mask), make_cache(cfg, mask)
    for k in range(cfg.n_scales):
        q, kk, v = gen.qkv(0, k)
        qp, kp, vp = q.pin_memory(), kk.pin_memory(), v.pin_memory()
        out_host = torch.empty_like(q).pin_memory()
        a.hack_scale_step_host(0, k, qp, kp, vp, out_host)
        qd, kd, vd = q.cuda(), kk.cuda(), v.cuda()
        out_dev = torch.empty_like(qd)
        b.hack_scale_step(0, k, qd, kd, vd, out_dev)
        torch.cuda.synchronize()
        assert torch.equal(out_host, out_dev.cpu())
    a.close()
    b.close()


def test_deterministic_across_runs():
    from tests.parity_util import make_cache
    from workloads import SyntheticQKV
    cfg = get_config(1, n_layers=1)
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    outs = []
    for _ in range(2):
        c = make_cache(cfg, mask)
        res = []
        for k in range(cfg.n_scales):
            q, kk, v = (t.cuda() for t in gen.qkv(0, k))
            out = torch.empty_like(q)
            c.hack_scale_step(0, k, q, kk, v, out)
            res.append(out)
        torch.cuda.synchronize()
        pos = [c.hack_read_head(0, 0, h, 2) for h in range(cfg.n_heads)]
        outs.append((res, pos))
        c.close()
    for x, y in zip(outs[0][0], outs[1][0]):
        assert torch.equal(x, y)
    assert outs[0][1] == outs[1][1]
