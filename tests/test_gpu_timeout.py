"""A bounded device-side wait that runs out.

Every mbarrier wait in the tensor-core kernels has a limit; when it expires the CTA raises the status
word, drains the copies and MMAs it has in flight, frees its tensor memory and returns.  The limit
is normally about a second, so nothing ever reaches it.  Here hack_set_wait_limit makes it one cycle
for one scoring launch: the consumers' first wait for an accumulator (which needs a key tile from
HBM and an MMA, a microsecond at least) gives up, hack_poll_status reports the time-out, and the
same cache, reset and back on the default limit, then passes the ordinary parity run.  Nothing
spins and nothing faults: the wait itself returns.
"""
from dataclasses import replace

import pytest
import torch

from workloads import SyntheticQKV, get_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


@pytest.mark.parametrize("head_dim", [64, 128])
def test_scoring_wait_runs_out_and_the_cache_stays_usable(head_dim):
    import paper_2504_09261_b200 as hb
    from tests.parity_util import make_cache, run_parity
    base = get_config(1 if head_dim == 64 else 3, n_layers=1)
    cfg = replace(base, name=base.name + "-tiny", n_heads=4, batch=1, sides=(1, 2, 4, 8, 12),
                  budget_c=40, budget_s=120)
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    cache = make_cache(cfg, mask)
    dev = torch.device("cuda:0")
    bh = cfg.batch * cfg.n_heads
    scores = torch.zeros((bh, cache.cand_stride), dtype=torch.float32, device=dev)
    # walk to the first step that scores
    k = 0
    while True:
        info = cache.hack_step_info(0, k)
        q, kk, v = (t.to(dev) for t in gen.qkv(0, k))
        if info.triggered_c or info.triggered_s:
            break
        cache.hack_scale_step(0, k, q, kk, v, torch.empty_like(q))
        k += 1
    cache.hack_poll_status()                       # nothing has gone wrong so far
    with pytest.raises(hb.HackError) as e:
        cache.hack_set_wait_limit(-1)
    assert e.value.status == 1
    cache.hack_set_wait_limit(1)
    cache.hack_score(0, k, q, kk, scores)
    with pytest.raises(hb.HackError) as e:
        cache.hack_poll_status()
    assert e.value.status == 6, str(e.value)          # HACK_ERR_TIMEOUT
    cache.hack_poll_status()                       # the word was cleared by the call that reported it
    cache.hack_set_wait_limit(0)
    # the context, the library and this very cache are as usable as before
    rep = run_parity(cfg, layers=[0], fused=True, staged_cache=cache)
    assert rep.ok(), rep.summary() + "\n" + "\n".join(rep.problems)
    assert rep.compressed_heads > 0
    cache.close()
