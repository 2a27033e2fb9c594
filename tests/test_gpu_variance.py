"""GPU parity of the attention variance per head (Eq. 6, offline head classification) against the
CPU oracle: on the uncompressed cache at the last scale (the setting of Eq. 6) and on a compressed,
ragged cache; plus the classification of the synthetic workload's planted head types.

Bar, written here: |sigma_gpu - sigma_oracle| <= 1e-3 * sigma_oracle + 1e-6.  The oracle works in
fp64 on the same bf16 inputs widened exactly; the GPU forms the logits with fp32 accumulation
(relative error of a probability about 1e-4 at these logit magnitudes), uses the hardware exp2
(2^-22) and a per-column mean-of-squares minus squared-mean in fp32."""
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


def _custom(base_index, **kw):
    cfg = get_config(base_index, n_layers=kw.pop("n_layers", 1))
    return replace(cfg, name=cfg.name + "-variance", **kw)


def _run_to_last(cfg, budget_c, budget_s, layer=0):
    """Decodes one layer up to (not including) the attention of the last scale; returns the cache,
    the last scale's Q on the device and everything the oracle needs."""
    import torch
    import paper_2504_09261_b200 as hb
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    cache = hb.HackCache(cfg.n_layers, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_BF16, mask,
                         budget_c, budget_s, n_obs=cfg.n_obs, device=0)
    bh = cfg.batch * cfg.n_heads
    scores = torch.empty((bh, cache.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, cache.kept_stride), dtype=torch.int32, device=dev)
    last = cfg.n_scales - 1
    for k in range(cfg.n_scales):
        q, kk, v = (t.to(dev) for t in gen.qkv(layer, k))
        if k < last:
            out = torch.empty_like(q)
            cache.hack_scale_step(layer, k, q, kk, v, out)
        else:
            cache.hack_score(layer, k, q, kk, scores)
            cache.hack_select(layer, k, scores, idx)
            cache.hack_compact(layer, k, idx, kk, v)
    torch.cuda.synchronize()
    return cache, gen, q, mask


def _oracle_sigma(cache, cfg, q_dev, layer=0):
    """Oracle on the rows the cache holds (read back byte for byte) and the bf16 queries."""
    import torch
    from oracle import hack_oracle as ho
    qd = q_dev.double().cpu().numpy()
    sig = np.zeros((cfg.batch, cfg.n_heads))
    for b in range(cfg.batch):
        for h in range(cfg.n_heads):
            raw = cache.hack_read_head(layer, b, h, 0)
            k_rows = torch.frombuffer(bytearray(raw), dtype=torch.bfloat16).view(-1, cfg.head_dim).double().numpy()
            sig[b, h] = ho.attention_variance(qd[b, h], k_rows, 1.0 / math.sqrt(cfg.head_dim))
    return sig


@pytest.mark.parametrize("base,sides", [(1, (1, 2, 4, 7, 11, 19)), (3, (1, 2, 4, 7, 12, 20))])
def test_variance_on_the_uncompressed_cache_of_the_last_scale(base, sides):
    import torch
    cfg = _custom(base, n_heads=4, batch=2, sides=sides)
    t_k = sum(s * s for s in sides)
    cache, gen, q, mask = _run_to_last(cfg, t_k, t_k)
    twin, _, q2, _ = _run_to_last(cfg, t_k, t_k)
    out = torch.empty_like(q)
    out_plain = torch.empty_like(q)
    sigma = torch.full((cfg.batch * cfg.n_heads,), float("nan"), device=q.device)
    cache.hack_attend_variance(0, cfg.n_scales - 1, q, out, sigma)
    twin.hack_attend(0, cfg.n_scales - 1, q2, out_plain)
    torch.cuda.synchronize()
    assert cache.hack_get_lengths(0) == [t_k] * (cfg.batch * cfg.n_heads)
    assert torch.equal(out.view(torch.int16), out_plain.view(torch.int16))       # the attention output is untouched
    ref = _oracle_sigma(cache, cfg, q).reshape(-1)
    got = sigma.double().cpu().numpy()
    assert np.all(np.abs(got - ref) <= 1e-3 * ref + 1e-6), (got, ref)
    # structural heads follow the query's position, contextual heads do not (planted in the inputs)
    ctx = np.tile(mask[0].astype(bool), cfg.batch)
    assert got[ctx].max() < got[~ctx].min()
    cache.close()
    twin.close()


def test_variance_on_a_compressed_ragged_cache():
    import torch
    cfg = _custom(3, n_heads=6, batch=1, sides=(1, 2, 4, 7, 11, 19))
    cache, gen, q, mask = _run_to_last(cfg, 70, 420)
    lengths = cache.hack_get_lengths(0)
    assert len(set(lengths)) == 2 and max(lengths) % 128 != 0          # two head types, ragged last key block
    out = torch.empty_like(q)
    sigma = torch.full((cfg.n_heads,), float("nan"), device=q.device)
    cache.hack_attend_variance(0, cfg.n_scales - 1, q, out, sigma)
    torch.cuda.synchronize()
    ref = _oracle_sigma(cache, cfg, q).reshape(-1)
    got = sigma.double().cpu().numpy()
    assert np.all(np.abs(got - ref) <= 1e-3 * ref + 1e-6), (got, ref)
    cache.close()


def test_variance_needs_the_tensor_core_path():
    import torch
    import paper_2504_09261_b200 as hb
    cfg = get_config(0, n_layers=1)                 # fp32 cache
    gen = SyntheticQKV(cfg)
    cache = hb.HackCache(1, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_F32,
                         gen.head_is_contextual.numpy(), 1000, 1000)
    dev = torch.device("cuda:0")
    q, kk, v = (t.to(dev) for t in gen.qkv(0, 0))
    bh = cfg.batch * cfg.n_heads
    scores = torch.empty((bh, cache.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, cache.kept_stride), dtype=torch.int32, device=dev)
    cache.hack_score(0, 0, q, kk, scores)
    cache.hack_select(0, 0, scores, idx)
    cache.hack_compact(0, 0, idx, kk, v)
    sigma = torch.zeros(cfg.batch * cfg.n_heads, device=dev)
    with pytest.raises(hb.HackError) as e:
        cache.hack_attend_variance(0, 0, q, torch.empty_like(q), sigma)
    assert e.value.status == 2
    cache.hack_attend(0, 0, q, torch.empty_like(q))     # the step is still pending and can be finished
    torch.cuda.synchronize()
    cache.close()


def test_classification_recovers_the_planted_head_types():
    """Eq. 6 end to end on a synthetic stack: sigma of every (layer, head) on the GPU, averaged over
    the batch (the 'samples'), ranked globally, alpha = the planted ratio."""
    import torch
    import paper_2504_09261_b200 as hb
    from oracle import hack_oracle as ho
    cfg = _custom(1, n_layers=3, batch=2)
    t_k = sum(s * s for s in cfg.sides)
    dev = torch.device("cuda:0")
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy().astype(np.uint8)
    cache = hb.HackCache(cfg.n_layers, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_BF16, mask,
                         t_k, t_k, device=0)
    sigma = torch.zeros((cfg.n_layers, cfg.batch * cfg.n_heads), device=dev)
    bh = cfg.batch * cfg.n_heads
    scores = torch.empty((bh, cache.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, cache.kept_stride), dtype=torch.int32, device=dev)
    last = cfg.n_scales - 1
    for l in range(cfg.n_layers):
        for k in range(cfg.n_scales):
            q, kk, v = (t.to(dev) for t in gen.qkv(l, k))
            out = torch.empty_like(q)
            if k < last:
                cache.hack_scale_step(l, k, q, kk, v, out)
            else:
                cache.hack_score(l, k, q, kk, scores)
                cache.hack_select(l, k, scores, idx)
                cache.hack_compact(l, k, idx, kk, v)
                cache.hack_attend_variance(l, k, q, out, sigma[l])
    torch.cuda.synchronize()
    mean_sigma = sigma.view(cfg.n_layers, cfg.batch, cfg.n_heads).double().mean(dim=1).cpu().numpy()
    alpha = float(mask.mean())
    got = hb.hack_classify_heads(mean_sigma.tolist(), cfg.n_layers, cfg.n_heads, alpha)
    assert got == ho.classify_heads(mean_sigma, alpha).tolist()
    assert got == mask.tolist()
    cache.close()
