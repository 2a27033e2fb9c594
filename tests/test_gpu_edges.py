"""GPU parity on shapes outside the five benchmark workloads: the code paths that only unusual
sizes reach (long candidate lists, odd head counts, head_dim 128 in fp32, one observation row,
a single scale) still have to agree with the CPU oracle under the same teacher-forced protocol."""
from dataclasses import replace

import pytest

from workloads import get_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


def _ok(rep):
    assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.problems)
    assert rep.heads_checked > 0


def _custom(base_index, **kw):
    cfg = get_config(base_index, n_layers=1)
    return replace(cfg, name=cfg.name + "-custom", **kw)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_long_candidate_list_takes_the_general_selection_path(dtype):
    """17 429 candidates per head: more than the register-resident selection holds (16 384), many
    scoring chunks per head, a ragged last chunk.  The new scale competes (policy 1) so that the
    kept length stays small and the oracle's attention stays cheap."""
    from tests.parity_util import run_parity
    cfg = _custom(0, sides=(1, 2, 132), n_heads=2, batch=1, dtype=dtype)
    rep = run_parity(cfg, layers=[0], fused=True, budget_c=300, budget_s=500, policy=1)
    _ok(rep)
    assert rep.compressed_heads > 0


def test_fp32_head_dim_128_and_odd_head_count():
    """fp32 runs on the SIMT kernels only; head_dim 128 and 3 heads x batch 1 are not in config 0."""
    from tests.parity_util import run_parity
    cfg = _custom(0, head_dim=128, n_heads=3, batch=1, sides=(1, 2, 3, 5, 9, 14))
    rep = run_parity(cfg, layers=[0], fused=True, budget_c=40, budget_s=120)
    _ok(rep)
    assert rep.compressed_heads > 0


def test_bf16_small_grid_single_query_tile_per_cta():
    """Few heads and a mid-sized scale: the tensor-core attention runs with one query tile per CTA
    and ragged last tiles in both the query and the key direction."""
    from tests.parity_util import run_parity
    cfg = _custom(3, n_heads=3, batch=1, sides=(1, 2, 4, 7, 11, 19))
    rep = run_parity(cfg, layers=[0], fused=True, budget_c=90, budget_s=400)
    _ok(rep)
    assert rep.compressed_heads > 0


def test_single_observation_row_and_single_scale():
    """n_obs = 1 (one query row scores every key) and a schedule of one scale."""
    from tests.parity_util import run_parity
    cfg = _custom(1, n_obs=1, n_heads=4, batch=1, sides=(1, 2, 4, 8, 12))
    rep = run_parity(cfg, layers=[0], fused=True, budget_c=20, budget_s=100)
    _ok(rep)
    one = _custom(1, n_heads=2, batch=1, sides=(9,), n_init_scales=1)
    rep = run_parity(one, layers=[0], fused=True, budget_c=30, budget_s=50, policy=1)
    _ok(rep)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("sampler", ["init", "recent", "caller", "full"])
def test_query_subset_rules_of_the_ablation(sampler, dtype):
    """The alternatives the paper's query-subset ablation compares with uniform spacing (first n,
    last n, random rows drawn by the caller, and every query: the ablation's reference) against the oracle under the same rule, with N_obs = 8
    and 32 so that both subset sizes of the size ablation's range and a ragged last scale occur."""
    import paper_2504_09261_b200 as hb
    from workloads import random_observation_rows
    from tests.parity_util import run_parity
    code = {"init": hb.HACK_OBS_INIT, "recent": hb.HACK_OBS_RECENT, "caller": hb.HACK_OBS_CALLER,
            "full": hb.HACK_OBS_FULL}[sampler]
    for n_obs in (8, 32):
        cfg = _custom(1 if dtype == "bf16" else 0, n_obs=n_obs, n_heads=4, batch=1, dtype=dtype,
                      sides=(1, 2, 3, 5, 8, 13, 19))
        rows = random_observation_rows(cfg, seed=n_obs) if sampler == "caller" else None
        rep = run_parity(cfg, layers=[0], fused=True, budget_c=60, budget_s=260, obs_sampler=code, obs_rows=rows)
        _ok(rep)
        assert rep.compressed_heads > 0


def test_caller_rows_are_checked_and_required():
    import paper_2504_09261_b200 as hb
    import torch
    from workloads import SyntheticQKV
    cfg = _custom(0, n_heads=2, batch=1, sides=(1, 2, 6), n_obs=4)
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    uniform = hb.HackCache(1, 2, cfg.head_dim, 1, cfg.sides, hb.HACK_F32, mask, 4, 8, n_obs=4)
    with pytest.raises(hb.HackError) as e:
        uniform.hack_set_obs_rows(2, [0, 1, 2, 3])
    assert e.value.status == 5
    uniform.close()
    cache = hb.HackCache(1, 2, cfg.head_dim, 1, cfg.sides, hb.HACK_F32, mask, 4, 8, n_obs=4,
                         obs_sampler=hb.HACK_OBS_CALLER)
    for bad in ([0, 1, 2], [0, 1, 2, 2], [0, 1, 2, 36], [-1, 1, 2, 3]):
        with pytest.raises(hb.HackError) as e:
            cache.hack_set_obs_rows(2, bad)
        assert e.value.status == 1
    dev = torch.device("cuda:0")
    for k in range(3):
        q, kk, v = (t.to(dev) for t in gen.qkv(0, k))
        out = torch.empty_like(q)
        if cache.hack_step_info(0, k).triggered_c:
            with pytest.raises(hb.HackError) as e:           # scoring without rows for this scale
                cache.hack_scale_step(0, k, q, kk, v, out)
            assert e.value.status == 5
            cache.hack_set_obs_rows(k, [35, 0, 7, 20] if k == 2 else list(range(min(4, cfg.sides[k] ** 2))))
        cache.hack_scale_step(0, k, q, kk, v, out)
    torch.cuda.synchronize()
    assert cache.hack_get_lengths(0) == [4, 41]      # structural head: 5 initial + 36 new tokens are protected
    cache.close()


def test_graph_replay_reproduces_direct_calls():
    """bench.py times CUDA-graph replays of the hack_scale_step calls; a replay has to write the
    same bytes as the direct calls did (the length plan is fixed, so a captured loop is complete)."""
    import torch
    from workloads import SyntheticQKV
    import paper_2504_09261_b200 as hb
    cfg = get_config(1, n_layers=2)
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg, device=dev)
    mask = gen.head_is_contextual
    L, K = cfg.n_layers, cfg.n_scales
    qkv = [[gen.qkv(l, k) for k in range(K)] for l in range(L)]

    def fresh():
        return hb.HackCache(L, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_BF16, mask.numpy(),
                            cfg.budget_c, cfg.budget_s, device=0)

    def loop(cache, outs, stream_handle):
        cache.hack_reset()
        for k in range(K):
            for l in range(L):
                q, kk, v = qkv[l][k]
                cache.hack_scale_step(l, k, q, kk, v, outs[l][k], stream_handle)

    direct = fresh()
    out_a = [[torch.zeros_like(qkv[l][k][0]) for k in range(K)] for l in range(L)]
    loop(direct, out_a, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()

    replayed = fresh()
    out_b = [[torch.zeros_like(qkv[l][k][0]) for k in range(K)] for l in range(L)]
    loop(replayed, out_b, torch.cuda.current_stream().cuda_stream)     # one-time kernel attributes
    torch.cuda.synchronize()
    for row in out_b:
        for t in row:
            t.zero_()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(g, stream=side):
        loop(replayed, out_b, torch.cuda.current_stream().cuda_stream)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    for l in range(L):
        for k in range(K):
            assert torch.equal(out_a[l][k].view(torch.int16), out_b[l][k].view(torch.int16)), (l, k)
    for l in range(L):
        assert direct.hack_get_lengths(l) == replayed.hack_get_lengths(l)
    direct.close()
    replayed.close()


def test_kept_list_beyond_65536_entries():
    """A budget above 65 536 entries: the compaction has to find the boundary between stored
    survivors and new rows in a kept list longer than its probe round covers at once.  Schedule
    (1, 2, 258, 30): the third scale brings 66 564 tokens and is only appended; the fourth exceeds
    the budget of 66 600, so 66 600 of 67 469 candidates survive.  Scores, index list, stored rows
    and positions are compared at that step, and its attention output (900 queries) as well; the
    oracle skips the output of the huge third scale (a 66 564 x 66 569 matrix in fp64)."""
    import numpy as np
    import torch
    import paper_2504_09261_b200 as hb
    from oracle import hack_oracle as ho
    from workloads import SyntheticQKV
    from tests.parity_util import OUT_TOL, SCORE_ATOL, SCORE_RTOL, _rows_bytes
    cfg = _custom(1, n_heads=2, batch=1, sides=(1, 2, 258, 30))
    budget = 66600
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg, device=dev)
    mask = gen.head_is_contextual.numpy()
    cache = hb.HackCache(1, cfg.n_heads, cfg.head_dim, 1, cfg.sides, hb.HACK_BF16, mask, budget, budget,
                         overflow_policy=hb.HACK_OVERFLOW_COMPETE)
    orc = ho.HackOracle(1, cfg.n_heads, 1, cfg.head_dim, cfg.sides, mask, budget, budget,
                        overflow_policy=ho.COMPETE)
    bh = cfg.n_heads
    scores = torch.zeros((bh, cache.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.full((bh, cache.kept_stride), -1, dtype=torch.int32, device=dev)
    for k in range(cfg.n_scales):
        q, kk, v = gen.qkv(0, k)
        out = torch.full_like(q, float("nan"))
        info = cache.hack_step_info(0, k)
        last = k == cfg.n_scales - 1
        assert bool(info.triggered_c and info.triggered_s) == last
        cache.hack_score(0, k, q, kk, scores)
        cache.hack_select(0, k, scores, idx)
        cache.hack_compact(0, k, idx, kk, v)
        cache.hack_attend(0, k, q, out)
        torch.cuda.synchronize()
        cache.hack_poll_status()
        q64, k64, v64 = (t.to(torch.float64).cpu().numpy() for t in (q, kk, v))
        override = {(0, h): scores[h, :info.cand_c].cpu().numpy().astype(np.float64) for h in range(bh)} if last else None
        o_ref, recs = orc.scale_step(0, k, q64, k64, v64, scores_override=override, need_output=last)
        if not last:
            continue
        assert info.kept_c == budget and info.kept_s == budget and info.cand_c == 67469
        for h in range(bh):
            rec = recs[(0, h)]
            sg = scores[h, :info.cand_c].cpu().numpy().astype(np.float64)
            den = SCORE_RTOL * np.maximum(np.abs(sg), np.abs(rec.scores)) + SCORE_ATOL
            assert np.all(np.abs(sg - rec.scores) <= den)
            assert np.array_equal(idx[h, :budget].cpu().numpy().astype(np.int64), rec.keep)
            st = orc.state[0][0][h]
            assert np.array_equal(np.frombuffer(cache.hack_read_head(0, 0, h, 2), dtype=np.int32).astype(np.int64), st.pos)
            assert cache.hack_read_head(0, 0, h, 0) == _rows_bytes(st.k, torch.bfloat16)
            assert cache.hack_read_head(0, 0, h, 1) == _rows_bytes(st.v, torch.bfloat16)
            d = float(np.max(np.abs(out[0, h].to(torch.float64).cpu().numpy() - o_ref[0, h])))
            assert d <= OUT_TOL["bf16"], f"head {h}: attention output off by {d:.3e}"
    cache.close()


@pytest.mark.parametrize("head_dim", [64, 128])
def test_output_store_stops_at_the_last_query_row(head_dim):
    """The tensor-core attention writes a 128-row output tile with one tiled store per 64 columns;
    the scales here have 36, 144 and 400 queries, so the last tile of every head reaches past the
    head's rows.  The output tensor of every step is a view into a larger buffer that carries a
    pattern behind it: the pattern has to survive, every head's rows have to be written (no row
    keeps the fill value), and a second run into a fresh buffer has to give the same bytes (a tile
    that reached into the next head's rows would race with that head's own store)."""
    import torch
    from workloads import SyntheticQKV
    import paper_2504_09261_b200 as hb
    cfg = _custom(3, n_heads=3, batch=2, head_dim=head_dim, sides=(1, 2, 6, 12, 20))
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg, device=dev)
    mask = gen.head_is_contextual
    K = cfg.n_scales
    qkv = [gen.qkv(0, k) for k in range(K)]
    guard = 4096                                   # elements behind the output
    fill = -12345.0                                # rounds to -12352 in bf16; the checks compare raw bits

    def run():
        cache = hb.HackCache(1, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_BF16, mask.numpy(), 150, 450,
                             device=0)
        bufs, outs = [], []
        for k in range(K):
            n = qkv[k][0].numel()
            buf = torch.full((n + guard,), fill, dtype=torch.bfloat16, device=dev)
            bufs.append(buf)
            outs.append(buf[:n].view(qkv[k][0].shape))
        for k in range(K):
            q, kk, v = qkv[k]
            cache.hack_scale_step(0, k, q, kk, v, outs[k])
        torch.cuda.synchronize()
        cache.hack_poll_status()                   # raises on a device-side error
        cache.close()
        return bufs, outs

    bufs_a, outs_a = run()
    bufs_b, outs_b = run()
    fill_bits = torch.tensor([fill], dtype=torch.bfloat16).view(torch.int16).item()
    for k in range(K):
        n = qkv[k][0].numel()
        tail = bufs_a[k][n:].view(torch.int16)
        assert bool((tail == fill_bits).all()), f"scale {k}: the store wrote behind the output"
        rows = outs_a[k].reshape(-1, cfg.head_dim).view(torch.int16)
        untouched = (rows == fill_bits).all(dim=1)
        assert not bool(untouched.any()), f"scale {k}: {int(untouched.sum())} output rows were never written"
        assert torch.equal(outs_a[k].view(torch.int16), outs_b[k].view(torch.int16)), f"scale {k}: two runs differ"
