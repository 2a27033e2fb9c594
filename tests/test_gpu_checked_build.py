"""The checked build: the stand-in for a memory checker on this path.

libhack_b200_checked.so is the same source compiled with -DHACK_DEBUG_CHECKS: every ragged index a
kernel forms (list entries, rows of a head, candidates, slots of the index list) is compared with its
bound before use, a violation skips the access and leaves a code in the status word, and every
(layer, batch, head) has a guard row behind its rows in the K, V and position planes.  The binding
selects that library when HACK_B200_CHECKED=1 and then verifies status word and guard rows whenever
a cache is closed, so running the ordinary GPU tests in such a process checks every kernel launch
they make.  test_gpu_suite_passes_in_the_checked_build does exactly that in a child process; the
tests below it only run inside that child.
"""
import os
import subprocess
import sys

import pytest
import torch

from workloads import SyntheticQKV, get_config

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHECKED = os.environ.get("HACK_B200_CHECKED", "0") == "1"


@pytest.fixture(scope="module", autouse=True)
def _built():
    import __graft_entry__ as ge
    ge.build()


@pytest.mark.skipif(CHECKED, reason="this is the child process")
def test_gpu_suite_passes_in_the_checked_build():
    env = dict(os.environ, HACK_B200_CHECKED="1")
    files = ["tests/test_gpu_checked_build.py", "tests/test_gpu_parity.py", "tests/test_gpu_edges.py",
             "tests/test_gpu_merge.py", "tests/test_gpu_variance.py", "tests/test_gpu_timeout.py",
             "tests/test_gpu_parity_stack.py", "tests/test_zz_no_alloc.py"]
    res = subprocess.run([sys.executable, "-m", "pytest", "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider",
                          "-k", "not config4_every_point and not config2_triples"] + files,
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = "\n".join((res.stdout + res.stderr).splitlines()[-25:])
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "no tests ran" not in res.stdout, tail


@pytest.mark.skipif(not CHECKED, reason="needs the checked build (run by the test above)")
def test_this_process_runs_the_checked_library():
    import paper_2504_09261_b200 as hb
    assert hb.binding.lib.hack_debug_build() == 1
    assert hb.binding._LIB_PATH.endswith("libhack_b200_checked.so")


@pytest.mark.skipif(not CHECKED, reason="needs the checked build (run by the test above)")
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_an_index_list_out_of_range_is_caught_not_followed(dtype):
    """hack_compact is handed an index list whose entries lie far outside the candidate list.  The
    kernels' checks skip every access formed from it, the status word names the site, the guard rows
    stay intact, and the cache works again after a reset."""
    import paper_2504_09261_b200 as hb
    from tests.parity_util import make_cache
    cfg = get_config(0 if dtype == "f32" else 1, n_layers=1)
    gen = SyntheticQKV(cfg)
    mask = gen.head_is_contextual.numpy()
    cache = make_cache(cfg, mask)
    dev = torch.device("cuda:0")
    bh = cfg.batch * cfg.n_heads
    k = 0
    while True:
        info = cache.hack_step_info(0, k)
        q, kk, v = (t.to(dev) for t in gen.qkv(0, k))
        if info.triggered_c or info.triggered_s:
            break
        cache.hack_scale_step(0, k, q, kk, v, torch.empty_like(q))
        k += 1
    cache.hack_poll_status()
    idx = torch.full((bh, cache.kept_stride), 1_000_000, dtype=torch.int32, device=dev)
    cache.hack_compact(0, k, idx, kk, v)
    with pytest.raises(hb.HackError) as e:
        cache.hack_poll_status()
    assert e.value.status == 5 and "bounds check" in str(e.value)
    assert cache.hack_debug_check() == 0
    cache.hack_reset()
    for kk_ in range(cfg.n_scales):
        q, kk, v = (t.to(dev) for t in gen.qkv(0, kk_))
        cache.hack_scale_step(0, kk_, q, kk, v, torch.empty_like(q))
    cache.hack_poll_status()
    cache.close()                                   # verifies the guard rows once more
