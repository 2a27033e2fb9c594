"""GPU parity of the final-scale merge of contextual heads (the sentence after Eq. 10) against the
CPU oracle under the same reading (cosine-nearest retained key, similarity-weighted average).

Protocol: every step is teacher-forced with the GPU's fp32 scores, so both sides keep the same
entries.  The counterpart of a discarded entry is an arg-max over fp32 (GPU) or fp64 (oracle)
similarities: where the two best similarities of an entry are closer than 1e-5 (ten times the fp32 error of a cosine here) either counterpart is
valid, so the retained rows such an entry could be folded into are only checked to lie in the hull of
the rows involved; all other rows are compared value by value.
Bar, written here: |x_gpu - x_oracle| <= 6e-3 |x_oracle| + 2e-3 for merged rows (the result is rounded
to bf16: half an ulp is 2^-9 relative; weights come from fp32 similarities); rows without assignments
keep their bits; the attention output of the step within the bf16 bar of the other parity tests."""
import math
from dataclasses import replace

import numpy as np
import pytest

from workloads import SyntheticQKV, get_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


def _rows(cache, layer, b, h, which, head_dim):
    import torch
    raw = cache.hack_read_head(layer, b, h, which)
    return torch.frombuffer(bytearray(raw), dtype=torch.bfloat16).view(-1, head_dim).double().numpy()


@pytest.mark.parametrize("base,sides,budget_c,budget_s", [
    (1, (1, 2, 4, 7, 11, 19), 150, 420),      # head_dim 64; 361 discarded entries per contextual head
    (3, (1, 2, 4, 7, 12, 20), 300, 700),      # head_dim 128; ragged tiles on both sides
])
def test_merge_matches_the_oracle(base, sides, budget_c, budget_s):
    import torch
    import paper_2504_09261_b200 as hb
    from oracle import hack_oracle as ho
    cfg = replace(get_config(base, n_layers=1), name="merge", n_heads=4, batch=2, sides=sides)
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    D, H, B = cfg.head_dim, cfg.n_heads, cfg.batch

    def make(merge):
        return hb.HackCache(1, H, D, B, cfg.sides, hb.HACK_BF16, mask, budget_c, budget_s, n_obs=cfg.n_obs,
                            merge_last=merge)

    gpu, plain = make(True), make(False)
    orc = ho.HackOracle(1, H, B, D, cfg.sides, mask, budget_c, budget_s, n_obs=cfg.n_obs, merge_last=True)
    bh = B * H
    scores = torch.empty((bh, gpu.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, gpu.kept_stride), dtype=torch.int32, device=dev)
    scores2, idx2 = torch.empty_like(scores), torch.empty_like(idx)
    last = cfg.n_scales - 1
    for k in range(cfg.n_scales):
        q, kk, v = gen.qkv(0, k)
        qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
        out, out_plain = torch.empty_like(qd), torch.empty_like(qd)
        info = gpu.hack_step_info(0, k)
        gpu.hack_score(0, k, qd, kd, scores)
        gpu.hack_select(0, k, scores, idx)
        gpu.hack_compact(0, k, idx, kd, vd)
        gpu.hack_attend(0, k, qd, out)
        plain.hack_score(0, k, qd, kd, scores2)
        plain.hack_select(0, k, scores2, idx2)
        plain.hack_compact(0, k, idx2, kd, vd)
        plain.hack_attend(0, k, qd, out_plain)
        torch.cuda.synchronize()
        sc = scores.double().cpu().numpy()
        override = {}
        for b in range(B):
            for h in range(H):
                ctx = bool(mask[0, h])
                if (info.triggered_c if ctx else info.triggered_s):
                    override[(b, h)] = sc[b * H + h, : (info.cand_c if ctx else info.cand_s)]
        o_ref, recs = orc.scale_step(0, k, q.double().numpy(), kk.double().numpy(), v.double().numpy(),
                                     scores_override=override)
        if k < last:
            assert torch.equal(out.view(torch.int16), out_plain.view(torch.int16))   # no merge before the last scale
    assert gpu.hack_get_lengths(0) == plain.hack_get_lengths(0)
    assert info.triggered_c, "the test must evict in contextual heads at the last scale"

    checked = loose = merged_rows = 0
    for b in range(B):
        for h in range(H):
            st = orc.state[0][b][h]
            k_gpu, v_gpu = _rows(gpu, 0, b, h, 0, D), _rows(gpu, 0, b, h, 1, D)
            k_pl, v_pl = _rows(plain, 0, b, h, 0, D), _rows(plain, 0, b, h, 1, D)
            if not mask[0, h]:
                assert np.array_equal(k_gpu, k_pl) and np.array_equal(v_gpu, v_pl)     # structural heads never merge
                continue
            rec = recs[(b, h)]
            assign, weight = rec.merge_assign, rec.merge_weight
            ev_k, ev_v = rec.evicted_k, rec.evicted_v
            assert np.array_equal(k_pl, rec.kept_k_before) and np.array_equal(v_pl, rec.kept_v_before)
            n_kept = k_pl.shape[0]
            touched = np.zeros(n_kept, dtype=bool)
            touched[assign[weight > 0]] = True
            # retained rows that an entry with two nearly equal best similarities could go to
            cos = (ev_k @ k_pl.T) / (np.linalg.norm(ev_k, axis=1, keepdims=True) * np.linalg.norm(k_pl, axis=1)[None, :])
            part = np.partition(cos, -2, axis=1)
            ambiguous = np.zeros(n_kept, dtype=bool)
            for e in np.nonzero((part[:, -1] - part[:, -2]) < 1e-5)[0]:
                ambiguous[np.argsort(cos[e])[-2:]] = True
            strict = ~ambiguous
            for got, ref, before in ((k_gpu, st.k, k_pl), (v_gpu, st.v, v_pl)):
                err = np.abs(got - ref)
                ok = err <= 6e-3 * np.abs(ref) + 2e-3
                assert ok[strict].all(), (b, h, float(err[strict].max()))
                untouched = strict & ~touched
                assert np.array_equal(got[untouched], before[untouched])                # bits kept
            lo = np.minimum(v_pl.min(axis=0), ev_v.min(axis=0)) - 1e-2
            hi = np.maximum(v_pl.max(axis=0), ev_v.max(axis=0)) + 1e-2
            assert np.all(v_gpu >= lo) and np.all(v_gpu <= hi)
            checked += int(strict.sum())
            loose += int(ambiguous.sum())
            merged_rows += int(touched.sum())
            assert not np.array_equal(k_gpu, k_pl)                                       # the merge did something
    assert merged_rows > 0 and loose <= 0.1 * (checked + loose), (checked, loose, merged_rows)
    # the step's attention ran on the merged cache
    err = np.abs(out.double().cpu().numpy() - o_ref)
    assert err.max() <= 2e-2, float(err.max())
    gpu.close()
    plain.close()


def test_fused_step_merges_like_the_staged_calls():
    import torch
    import paper_2504_09261_b200 as hb
    cfg = replace(get_config(3, n_layers=1), name="merge-fused", n_heads=4, batch=1, sides=(1, 2, 4, 7, 12, 20))
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    caches = [hb.HackCache(1, cfg.n_heads, cfg.head_dim, 1, cfg.sides, hb.HACK_BF16, mask, 300, 700, merge_last=True)
              for _ in range(2)]
    bh = cfg.n_heads
    scores = torch.empty((bh, caches[0].cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, caches[0].kept_stride), dtype=torch.int32, device=dev)
    outs = []
    for k in range(cfg.n_scales):
        q, kk, v = (t.to(dev) for t in gen.qkv(0, k))
        outs = [torch.empty_like(q), torch.empty_like(q)]
        caches[0].hack_score(0, k, q, kk, scores)
        caches[0].hack_select(0, k, scores, idx)
        caches[0].hack_compact(0, k, idx, kk, v)
        caches[0].hack_attend(0, k, q, outs[0])
        caches[1].hack_scale_step(0, k, q, kk, v, outs[1])
    torch.cuda.synchronize()
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
    for h in range(cfg.n_heads):
        for which in (0, 1):
            assert caches[0].hack_read_head(0, 0, h, which) == caches[1].hack_read_head(0, 0, h, which)
    for c in caches:
        c.close()


def test_merge_needs_bf16():
    import paper_2504_09261_b200 as hb
    cfg = get_config(0, n_layers=1)
    gen = SyntheticQKV(cfg)
    with pytest.raises(hb.HackError) as e:
        hb.HackCache(1, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_F32, gen.head_is_contextual.numpy(),
                     30, 300, merge_last=True)
    assert e.value.status == 2
