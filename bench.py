#!/usr/bin/env python
"""Benchmark of the per-scale decoding hot path (score -> select -> compact -> attend).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

A "step" is one pass of the whole hot path over one batch of synthetic input: the full decoding
loop of one image batch, every layer at every scale, each (layer, scale) served by one
hack_scale_step call.  The default workload is config 3 (Infinity-2B-shaped stack, 1024x1024,
13 scales, batch 2, bf16, budget 30 %), the configuration the roofline target is quoted on.
Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from workloads import SyntheticQKV, get_config  # noqa: E402
from workloads import sharding  # noqa: E402

METRIC = "scale-step tokens/s (score+select+compact+attend)"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}      # the figures the target names
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")


def measured_traffic(config_index: int):
    """DRAM bytes of one last-scale attention launch as ncu counted them, or None when there is no
    record for this workload or the kernel source has changed since the counters were taken."""
    import hashlib
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(f"attend_tc_config{config_index}_last_scale")
        if not rec:
            return None
        src = os.path.join(ROOT, rec["source"])
        with open(src, "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != rec["source_sha256"]:
                return None
        return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])
    except Exception:
        return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- work model
def step_work(info, cfg, n_ctx_heads, persist=True):
    """Algorithmic FLOPs and bytes of one (layer, scale) step from its length plan."""
    D, e, b, H = cfg.head_dim, (4 if cfg.dtype == "f32" else 2), cfg.batch, cfg.n_heads
    n_c, n_s = b * n_ctx_heads, b * (H - n_ctx_heads)
    kept = n_c * info.kept_c + n_s * info.kept_s
    cand = n_c * info.cand_c * info.triggered_c + n_s * info.cand_s * info.triggered_s
    attend_flops = 4.0 * info.n_new * D * kept
    score_flops = 2.0 * info.n_obs_rows * D * cand
    nbytes = cand * (D * e + 8) + 2 * kept * 2 * D * e + 2 * info.n_new * H * b * D * e
    return attend_flops, score_flops, float(nbytes)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.index)],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 7:
                        continue
                    try:
                        sm.append(float(parts[0]))
                        smax.append(float(parts[1]))
                    except ValueError:
                        continue
                    for n, v in zip(names, parts[3:7]):
                        if v.lower().startswith("active"):
                            reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- oracle arm
_ORACLE_INPUTS = {}


def oracle_sample_run(cfg, n_pairs: int):
    """Time the CPU oracle, as it stands, on layer 0 of the workload: all scales, n_pairs of the
    (batch, head) pairs.  Returns (seconds, fraction of one full step covered, threads)."""
    import numpy as np
    from oracle import hack_oracle as ho
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    one = cfg.with_layers(1)
    gen = SyntheticQKV(one)
    mask = gen.head_is_contextual.numpy()
    pairs_all = [(b, h) for b in range(cfg.batch) for h in range(cfg.n_heads)]
    # alternate contextual / structural heads so the sample has the workload's mix
    ctx = [p for p in pairs_all if mask[0, p[1]]]
    stc = [p for p in pairs_all if not mask[0, p[1]]]
    n_c = max(1, round(n_pairs * len(ctx) / len(pairs_all))) if ctx else 0
    pairs = ctx[:n_c] + stc[: n_pairs - n_c]
    if cfg.index not in _ORACLE_INPUTS:          # generated once, outside the timed part
        _ORACLE_INPUTS[cfg.index] = [tuple(t.to(torch.float64).numpy() for t in gen.qkv(0, k))
                                     for k in range(cfg.n_scales)]
    inputs = _ORACLE_INPUTS[cfg.index]
    orc = ho.HackOracle(1, cfg.n_heads, cfg.batch, cfg.head_dim, cfg.sides, mask, cfg.budget_c,
                        cfg.budget_s, n_obs=cfg.n_obs, n_init_scales=cfg.n_init_scales)
    t0 = time.perf_counter()
    for k in range(cfg.n_scales):
        q, kk, v = inputs[k]
        orc.scale_step(0, k, q, kk, v, heads=pairs)
    dt = time.perf_counter() - t0
    frac = (len(pairs) / len(pairs_all)) / cfg.n_layers
    return dt, frac, threads, len(pairs)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_config(args.config)
    tokens = cfg.batch * cfg.total_tokens
    n_pairs = args.oracle_pairs
    for _ in range(min(args.warmup, 1)):
        oracle_sample_run(cfg, 2)
    times = []
    for _ in range(args.steps):
        dt, frac, threads, used = oracle_sample_run(cfg, n_pairs)
        times.append(dt / frac)
    sec = sum(times) / len(times)
    value = tokens / sec
    sample = (f"layer 0 of {cfg.n_layers}, all {cfg.n_scales} scales, {used} of "
              f"{cfg.batch * cfg.n_heads} (batch, head) pairs; time scaled by 1/{frac:.6f}")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"config {cfg.index}: {cfg.name}", "tokens_per_step": tokens,
                   "budget": cfg.budget_total, "budget_c": cfg.budget_c, "budget_s": cfg.budget_s},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- our arm
def run_ours(args):
    import paper_2504_09261_b200 as hb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    cfg = get_config(args.config, args.budget_frac, args.alpha)
    if args.layers:
        cfg = cfg.with_layers(args.layers)
    if args.n_obs:
        from dataclasses import replace as _replace
        cfg = _replace(cfg, n_obs=args.n_obs)
    L, K = cfg.n_layers, cfg.n_scales
    gen = sharding.rank_generator(cfg, rank, device=dev)        # each rank decodes its own images
    mask = gen.head_is_contextual
    n_ctx = [int(mask[l].sum()) for l in range(L)]
    dtype_id = hb.HACK_F32 if cfg.dtype == "f32" else hb.HACK_BF16

    def new_cache(bc, bs, policy=0):
        return hb.HackCache(L, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, dtype_id, mask.numpy(),
                            bc, bs, n_obs=cfg.n_obs, n_init_scales=cfg.n_init_scales, overflow_policy=policy,
                            device=local, merge_last=args.merge_last, obs_sampler=args.obs_sampler)

    cache = new_cache(cfg.budget_c, cfg.budget_s)
    # inputs resident in HBM: every (layer, scale) has its own Q, K, V (ranks draw different images)
    qkv = [[None] * K for _ in range(L)]
    in_bytes = 0
    for l in range(L):
        for k in range(K):
            qkv[l][k] = gen.qkv(l, k)
            in_bytes += sum(t.numel() * t.element_size() for t in qkv[l][k])
    outs = [torch.empty_like(qkv[0][k][0]) for k in range(K)]
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream

    def loop(c, scale_events=None):
        c.hack_reset()
        for k in range(K):
            for l in range(L):
                q, kk, v = qkv[l][k]
                c.hack_scale_step(l, k, q, kk, v, outs[k], sh)
            if scale_events is not None:
                scale_events[k].record(stream)

    def capture(c):
        """One CUDA graph per scale, captured from the same C-ABI calls `loop` makes.  The length
        plan of every step is fixed by the schedule and the budgets, so a replay is the complete
        decoding loop of one image batch."""
        c.hack_reset()
        graphs = []
        side = torch.cuda.Stream()
        for k in range(K):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                cs = torch.cuda.current_stream().cuda_stream
                for l in range(L):
                    q, kk, v = qkv[l][k]
                    c.hack_scale_step(l, k, q, kk, v, outs[k], cs)
            graphs.append(g)
        return graphs

    def replay(graphs, scale_events=None):
        for k in range(K):
            graphs[k].replay()
            if scale_events is not None:
                scale_events[k].record(stream)

    def timed(c, steps, warmup, per_scale=False, use_graph=True):
        for _ in range(min(warmup, 2)):
            loop(c)                       # direct calls first: one-time kernel attributes are set here
        torch.cuda.synchronize()
        graphs = capture(c) if use_graph else None
        run = (lambda ev=None: replay(graphs, ev)) if use_graph else (lambda ev=None: loop(c, ev))
        for _ in range(warmup):
            run()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        ev0 = torch.cuda.Event(enable_timing=True)
        ev1 = torch.cuda.Event(enable_timing=True)
        sev = [[torch.cuda.Event(enable_timing=True) for _ in range(K)] for _ in range(steps)] if per_scale else None
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)] if per_scale else None
        ev0.record(stream)
        for s in range(steps):
            if per_scale:
                starts[s].record(stream)
            run(sev[s] if per_scale else None)
        ev1.record(stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
        scale_ms = None
        if per_scale:
            scale_ms = [0.0] * K
            for s in range(steps):
                prev = starts[s]
                for k in range(K):
                    scale_ms[k] += prev.elapsed_time(sev[s][k]) / steps
                    prev = sev[s][k]
        del graphs
        return ms, scale_ms

    use_graph = not args.no_graph
    if args.latency_profile:
        # Attention-module latency per scale (score + select + compact + attend of every layer) for the
        # uncompressed cache and for compression ratios rho = 1 - B / T_K, budgets split 1 : 2 between
        # contextual and structural heads (Eq. 7).  The cumulative time up to the scale whose side is
        # 16 / 32 / 64 is the latency of a 256 / 512 / 1024 pixel image under this schedule: the
        # resolution axis of the paper's latency profile.  One JSON line.
        cache.close()
        t_k = cfg.total_tokens
        rows = []
        for rho, policy in ((0.0, 0), (0.3, 0), (0.5, 0), (0.7, 0), (0.9, 0), (0.9, 1)):
            if rho == 0.0:
                bc = bs = t_k
            else:
                bc, bs = hb.hack_split_budget(int((1.0 - rho) * t_k + 1e-9), cfg.alpha, hb.RULE_RATIO, 2.0, t_k)
            c = new_cache(bc, bs, policy)
            ms, scale_ms = timed(c, args.steps, args.warmup, per_scale=True, use_graph=use_graph)
            _, peak_kv, _ = c.hack_kv_bytes()
            c.close()
            cum = 0.0
            at_side = {}
            for k in range(K):
                cum += scale_ms[k]
                at_side[cfg.sides[k]] = cum
            rows.append({"rho": rho, "budget_c": bc, "budget_s": bs,
                         "overflow_policy": "keep protected" if policy == 0 else "compete",
                         "ms_per_image_batch": ms / args.steps, "ms_per_scale": [round(x, 4) for x in scale_ms],
                         "ms_up_to_side": {str(sd): round(at_side[sd], 4) for sd in (16, 32, 64) if sd in at_side},
                         "peak_kv_bytes": peak_kv})
        full = rows[0]
        for r in rows:
            r["speedup_vs_full"] = full["ms_per_image_batch"] / r["ms_per_image_batch"]
            r["speedup_last_scale"] = full["ms_per_scale"][-1] / r["ms_per_scale"][-1]
        if rank == 0:
            print(json.dumps({"metric": "attention-module latency per scale, uncompressed against compressed",
                              "unit": "ms", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                              "dtype": cfg.dtype, "data": "synthetic",
                              "config": {"workload": cfg.name, "layers": L, "sides": list(cfg.sides),
                                         "timing": "CUDA graph replay" if use_graph else "direct calls"},
                              "rows": rows}))
        if dist is not None:
            dist.destroy_process_group()
        return
    launches0 = cache.hack_launch_count()
    loop(cache)
    launches_per_step = cache.hack_launch_count() - launches0
    sampler = ClockSampler(local)
    sampler.start()
    total_ms, scale_ms = timed(cache, args.steps, args.warmup, per_scale=True, use_graph=use_graph)
    clocks = sampler.stop()
    total_ms = sharding.max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    tokens = cfg.batch * cfg.total_tokens
    value = sharding.job_throughput(world, tokens, ms_per_step)
    live, peak, reserved = cache.hack_kv_bytes()

    # ---- work model and roofline of the loop
    peaks, peak_kind = load_peaks()
    hbm = peaks["hbm_gbs"] * 1e9
    tf_burst = peaks["bf16_tflops"] * 1e12
    tf_sus = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12
    # Which measured tensor peak is like for like: the burst figure was taken at full clock, the
    # sustained one under the power cap (about two thirds of the clock).  A run whose sampled SM
    # clock stayed near the maximum with no power cap is compared with the burst peak.
    at_full_clock = bool(clocks["sm_mhz"] and clocks["sm_max_mhz"] and clocks["sm_mhz"] >= 0.9 * clocks["sm_max_mhz"]
                         and "sw_power_cap" not in clocks["reasons"])
    tf_ref = tf_burst if at_full_clock else tf_sus
    peak_note = (f"bf16_tflops ({'burst' if at_full_clock else 'sustained'}) of {peak_kind}: median SM clock "
                 f"{clocks['sm_mhz']} of {clocks['sm_max_mhz']} MHz, reasons {clocks['reasons']}")
    infos = []
    walker = hb.HackCache(1, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, dtype_id, mask[0].numpy(),
                          cfg.budget_c, cfg.budget_s, n_obs=cfg.n_obs, n_init_scales=cfg.n_init_scales,
                          device=local)
    # lengths depend on the head type only, so layer 0's plan holds for every layer
    dq = torch.zeros((cfg.batch, cfg.n_heads, max(cfg.tokens_per_scale), cfg.head_dim),
                     dtype=qkv[0][0][0].dtype, device=dev)
    for k in range(K):
        infos.append(walker.hack_step_info(0, k))
        walker.hack_scale_step(0, k, dq, dq, dq, dq, sh)
    torch.cuda.synchronize()
    walker.close()
    attend_fl = score_fl = byt = 0.0
    t_roof = 0.0
    roof_alt = {"sustained": 0.0, "burst": 0.0, "nominal": 0.0}
    per_scale = []
    for k in range(K):
        a_k = s_k = b_k = roof_k = 0.0
        for l in range(L):
            a, s, by = step_work(infos[k], cfg, n_ctx[l])
            a_k += a
            s_k += s
            b_k += by
            roof_k += max((a + s) / tf_ref, by / hbm)
            roof_alt["sustained"] += max((a + s) / tf_sus, by / hbm)
            roof_alt["burst"] += max((a + s) / tf_burst, by / hbm)
            roof_alt["nominal"] += max((a + s) / (NOMINAL_PEAKS["bf16_tflops"] * 1e12),
                                       by / (NOMINAL_PEAKS["hbm_gbs"] * 1e9))
        attend_fl += a_k
        score_fl += s_k
        byt += b_k
        t_roof += roof_k
        per_scale.append({
            "scale": k, "n_new": infos[k].n_new, "kept_c": infos[k].kept_c, "kept_s": infos[k].kept_s,
            "ms": round(scale_ms[k], 4),
            "tokens_per_s": round(cfg.batch * infos[k].n_new / (scale_ms[k] * 1e-3), 1),
            "roofline_ms": round(roof_k * 1e3, 4),
            "roofline_frac": round(roof_k * 1e3 / scale_ms[k], 4),
        })

    # ---- per-stage device time (second pass, stage events on) -> roofline of the dominant kernel
    stage = None
    roofline = None
    if rank == 0:
        cache.hack_stage_timing(True)
        n_prof = 2
        for _ in range(n_prof):
            loop(cache)
        st = cache.hack_stage_times()
        cache.hack_stage_timing(False)
        stage = {k: {"ms_per_step": v[0] / n_prof, "launches_per_step": v[1] // n_prof} for k, v in st.items()}
        # The dominant kernel is the attention launch of the last scale (the largest launch of the
        # step).  It is timed on its own launch here: the last scale runs through the staged calls
        # with CUDA events on the launching stream around hack_attend, every layer, in loop order
        # (the score / select / compact kernels of the same layer run in between, so its inputs are
        # not L2-warm from a previous attention launch).
        lim_c, lim_k = cache.cand_stride, cache.kept_stride
        bh = cfg.batch * cfg.n_heads
        sc_buf = torch.empty((bh, lim_c), dtype=torch.float32, device=dev)
        ix_buf = torch.empty((bh, lim_k), dtype=torch.int32, device=dev)
        n_rep = 3
        evs = []
        for _ in range(n_rep):
            cache.hack_reset()
            for k in range(K):
                for l in range(L):
                    q, kk, v = qkv[l][k]
                    if k < K - 1:
                        cache.hack_scale_step(l, k, q, kk, v, outs[k], sh)
                        continue
                    cache.hack_score(l, k, q, kk, sc_buf, sh)
                    cache.hack_select(l, k, sc_buf, ix_buf, None, sh)
                    cache.hack_compact(l, k, ix_buf, kk, v, sh)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    cache.hack_attend(l, k, q, outs[k], sh)
                    e1.record(stream)
                    evs.append((e0, e1))
        torch.cuda.synchronize()
        last_ms = sorted(e0.elapsed_time(e1) for e0, e1 in evs)
        last_ms = last_ms[len(last_ms) // 2]            # median launch
        last = infos[K - 1]
        n_c_heads = [cfg.batch * n for n in n_ctx]
        kept_sum = sum(nc * last.kept_c + (bh - nc) * last.kept_s for nc in n_c_heads) / L
        last_flops = 4.0 * last.n_new * cfg.head_dim * kept_sum
        last_bytes = 2 * kept_sum * cfg.head_dim * 2 + 2 * last.n_new * bh * cfg.head_dim * 2
        achieved = last_flops / (last_ms * 1e-3) / 1e12
        peak_tf = tf_ref / 1e12 if cfg.dtype != "f32" else None
        att_ms = stage["attend"]["ms_per_step"]
        att_n = max(stage["attend"]["launches_per_step"], 1)
        roofline = {
            "kernel": "attend_tc_kernel, launch of the last scale", "bound": "tensor",
            "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
            "frac": (achieved / peak_tf) if peak_tf else None,
            "traffic": measured_traffic(cfg.index),
            "peak_source": peak_note,
            "frac_of_burst": achieved / (tf_burst / 1e12), "frac_of_sustained": achieved / (tf_sus / 1e12),
            "frac_of_nominal": achieved / NOMINAL_PEAKS["bf16_tflops"],
            "flops_per_launch": last_flops, "algorithmic_bytes_per_launch": last_bytes,
            "launch_ms_median": last_ms, "launches_timed": len(evs),
            "all_attend_launches": {"tflops": attend_fl / (att_ms * 1e-3) / 1e12, "launches_per_step": att_n,
                                    "ms_per_step": att_ms},
        }

    # ---- e2e: same loop through the host-buffer entry point (pinned host memory)
    e2e = None
    if not args.no_e2e:
        host = [[tuple(t.cpu().pin_memory() for t in qkv[l][k]) for k in range(K)] for l in range(L)]
        host_out = [torch.empty_like(host[0][k][0]).pin_memory() for k in range(K)]
        c2 = new_cache(cfg.budget_c, cfg.budget_s)

        def loop_host():
            c2.hack_reset()
            for k in range(K):
                for l in range(L):
                    q, kk, v = host[l][k]
                    c2.hack_scale_step_host(l, k, q, kk, v, host_out[k], sh)

        for _ in range(2):
            loop_host()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_e2e = max(1, min(args.steps, 3))
        e0.record(stream)
        for _ in range(n_e2e):
            loop_host()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n_e2e
        ms = sharding.max_over_ranks(ms, dist, dev)
        e2e = {"value": sharding.job_throughput(world, tokens, ms), "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": in_bytes // 3}
        c2.close()
        del host, host_out

    # ---- uncompressed comparison run (same call, budgets = T_K)
    full = None
    if rank == 0 and not args.no_full:
        cf = new_cache(cfg.total_tokens, cfg.total_tokens)
        ms_f, _ = timed(cf, 2, 1, use_graph=use_graph)
        ms_f /= 2
        _, peak_f, res_f = cf.hack_kv_bytes()
        full = {"ms_per_step": ms_f, "tokens_per_s": tokens / (ms_f * 1e-3), "kv_bytes_peak": peak_f,
                "speedup_of_budgeted_run": ms_f / ms_per_step}
        cf.close()

    # ---- CPU oracle on the host cores (rank 0, N = 1)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        base_cfg = get_config(args.config, args.budget_frac, args.alpha)
        dt, frac, threads, used = oracle_sample_run(base_cfg, args.oracle_pairs)
        cpu = {"value": base_cfg.batch * base_cfg.total_tokens / (dt / frac), "unit": UNIT, "cores": threads,
               "kind": "oracle", "seconds_measured": dt,
               "sample": (f"layer 0 of {base_cfg.n_layers}, all {base_cfg.n_scales} scales, {used} of "
                          f"{base_cfg.batch * base_cfg.n_heads} (batch, head) pairs; time scaled by 1/{frac:.6f}")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {
                "workload": f"config {cfg.index}: {cfg.name}", "n_layers": L, "n_heads": cfg.n_heads,
                "head_dim": cfg.head_dim, "batch": cfg.batch, "scales": list(cfg.sides),
                "tokens_per_step": tokens, "budget": cfg.budget_total, "budget_c": cfg.budget_c,
                "budget_s": cfg.budget_s, "calls_per_step": L * K,
                "launch": ("one CUDA graph per scale, captured from the hack_scale_step calls" if use_graph
                           else "direct hack_scale_step calls"),
                "l2": f"inputs larger than L2 ({in_bytes / 1e9:.2f} GB of Q/K/V walked once per step)",
                "sharding": "independent image batches per GPU, no collective in the path",
            },
            "roofline": roofline,
            "loop_roofline": {"t_roof_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms_per_step,
                              "flops": attend_fl + score_fl, "bytes": byt, "peaks": peak_kind,
                              "tensor_peak": peak_note,
                              "frac_of_sustained": roof_alt["sustained"] * 1e3 / ms_per_step,
                              "frac_of_burst": roof_alt["burst"] * 1e3 / ms_per_step,
                              "frac_of_nominal": roof_alt["nominal"] * 1e3 / ms_per_step},
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks, "stages": stage, "per_scale": per_scale,
            "kv_bytes": {"live": live, "peak": peak, "reserved": reserved,
                         "full_cache": 2 * cfg.total_tokens * cfg.head_dim * (4 if cfg.dtype == "f32" else 2)
                         * cfg.n_heads * L * cfg.batch},
            "full_cache_run": full,
        }
        if not args.quiet:
            print(json.dumps(line))
    cache.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return line if rank == 0 else None


def run_head_variance(args):
    """Separate measurement (not part of the decoding loop): the attention-variance pass of the offline
    head classification (Eq. 6) on one layer of the chosen workload, uncompressed cache, last scale.
    Prints its own JSON line.  The pass evaluates one exponential per (query, key) pair, so it is
    bound by the special-function units: 16 exp2 per clock and SM."""
    import torch
    import paper_2504_09261_b200 as hb
    from workloads import SyntheticQKV, get_config
    cfg = get_config(args.config, n_layers=1)
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    gen = SyntheticQKV(cfg, device=dev)
    mask = gen.head_is_contextual
    t_k = cfg.total_tokens
    K = cfg.n_scales
    bh = cfg.batch * cfg.n_heads
    cache = hb.HackCache(1, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides, hb.HACK_BF16, mask.numpy(), t_k, t_k,
                         n_obs=cfg.n_obs, device=0)
    qkv = [gen.qkv(0, k) for k in range(K)]
    outs = [torch.empty_like(qkv[k][0]) for k in range(K)]
    scores = torch.empty((bh, cache.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, cache.kept_stride), dtype=torch.int32, device=dev)
    sigma = torch.zeros(bh, device=dev)
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream

    def one(with_variance):
        cache.hack_reset()
        for k in range(K - 1):
            q, kk, v = qkv[k]
            cache.hack_scale_step(0, k, q, kk, v, outs[k], sh)
        q, kk, v = qkv[K - 1]
        cache.hack_score(0, K - 1, q, kk, scores, sh)
        cache.hack_select(0, K - 1, scores, idx, None, sh)
        cache.hack_compact(0, K - 1, idx, kk, v, sh)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        if with_variance:
            cache.hack_attend_variance(0, K - 1, q, outs[K - 1], sigma, sh)
        else:
            cache.hack_attend(0, K - 1, q, outs[K - 1], sh)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(0)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        one(True)
        one(False)
    both = sorted(one(True) for _ in range(max(args.steps, 5)))
    plain = sorted(one(False) for _ in range(max(args.steps, 5)))
    clocks = sampler.stop()
    ms_both, ms_plain = both[len(both) // 2], plain[len(plain) // 2]
    ms_var = ms_both - ms_plain
    n_k = cfg.tokens_per_scale[-1]
    pairs = float(bh) * n_k * t_k
    props = torch.cuda.get_device_properties(0)
    sm_mhz = clocks.get("sm_max_mhz") or 1965.0
    peak = 16.0 * props.multi_processor_count * sm_mhz * 1e6
    print(json.dumps({
        "metric": "attention-variance pass of the offline head classification (Eq. 6), (query, key) pairs per second",
        "value": pairs / (ms_var * 1e-3), "unit": "pairs/s", "n_gpus": 1, "higher_is_better": True,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"config {args.config}, one layer, uncompressed cache, last scale: "
                               f"{bh} heads x {n_k} queries x {t_k} keys, head_dim {cfg.head_dim}"},
        "ms_attend": ms_plain, "ms_attend_with_variance": ms_both, "ms_variance_kernels": ms_var,
        "roofline": {"kernel": "attn_colstats_kernel", "bound": "alu", "achieved": pairs / (ms_var * 1e-3) / 1e9,
                     "peak": peak / 1e9, "unit": "G exp2/s", "frac": pairs / (ms_var * 1e-3) / peak,
                     "peak_source": f"16 exp2 per clock and SM x {props.multi_processor_count} SMs x {sm_mhz:.0f} MHz (clocks.max.sm)",
                     "traffic": None},
        "tensor_tflops": 2.0 * pairs * cfg.head_dim / (ms_var * 1e-3) / 1e12,
        "sigma_mean_contextual": float(sigma.view(cfg.batch, cfg.n_heads)[:, mask[0].bool()].mean()),
        "sigma_mean_structural": float(sigma.view(cfg.batch, cfg.n_heads)[:, ~mask[0].bool()].mean()),
        "clocks": clocks,
    }))
    cache.close()


def run_sweep(args):
    """Every workload that has budget literals (configs 0, 1, 2 x {30, 50, 70 %}, 3, 4 x {25, 50, 75 %
    contextual} x {10, 30, 50 %}), one compact JSON line each: loop time, tokens/s, fraction of the
    loop roofline, KV bytes, and the uncompressed run of the same inputs."""
    from workloads import list_configs
    for (index, frac, alpha) in list_configs():
        a = argparse.Namespace(**vars(args))
        a.config, a.budget_frac, a.alpha = index, frac, alpha
        a.no_e2e = a.no_cpu = a.quiet = True
        a.no_full = False
        line = run_ours(a)
        torch.cuda.empty_cache()
        full = line["full_cache_run"]
        print(json.dumps({
            "workload": line["config"]["workload"], "budget_frac": frac, "alpha": alpha,
            "budget_c": line["config"]["budget_c"], "budget_s": line["config"]["budget_s"],
            "dtype": line["dtype"], "ms_per_step": round(line["ms_per_step"], 4),
            "tokens_per_s": round(line["value"], 1), "gpu_launches_per_step": line["gpu_launches"] // line["steps"],
            "loop_roofline": {k: (round(v, 4) if isinstance(v, float) else v) for k, v in line["loop_roofline"].items()
                              if k in ("t_roof_ms", "frac", "frac_of_sustained", "frac_of_burst", "frac_of_nominal")},
            "kv_bytes_peak": line["kv_bytes"]["peak"], "kv_bytes_full_cache": line["kv_bytes"]["full_cache"],
            "full_cache_run_ms": round(full["ms_per_step"], 4),
            "speedup_vs_full_cache": round(full["speedup_of_budgeted_run"], 4),
            "sm_mhz": line["clocks"]["sm_mhz"], "clock_reasons": line["clocks"]["reasons"]}), flush=True)


def spawn_ranks(n: int) -> int:
    """Started plainly with --gpus N > 1: run the same command as N ranks, one per GPU."""
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    if have < n:
        print(f"bench.py --gpus {n} needs {n} GPUs on this node; {have} visible", file=sys.stderr)
        return 2
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--budget-frac", type=float, default=None, help="point of the budget sweep of configs 2 and 4")
    ap.add_argument("--alpha", type=float, default=None, help="contextual share of config 4's sweep")
    ap.add_argument("--sweep", action="store_true",
                    help="every workload and sweep point, one compact JSON line each, instead of the default loop")
    ap.add_argument("--layers", type=int, default=0, help="restrict the stack (debugging only)")
    ap.add_argument("--oracle-pairs", type=int, default=32)
    ap.add_argument("--no-graph", action="store_true", help="time direct calls instead of graph replays")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-full", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--n-obs", type=int, default=0, help="query subset size N_obs (1..32) instead of the workload's 32")
    ap.add_argument("--obs-sampler", type=int, default=0, choices=[0, 1, 2],
                    help="query subset rule: 0 uniform (the method), 1 first n, 2 last n")
    ap.add_argument("--merge-last", action="store_true",
                    help="contextual heads fold what the last scale discards into what it keeps (off in the paper's efficiency runs' default here)")
    ap.add_argument("--latency-profile", action="store_true",
                    help="per-scale latency of the uncompressed cache and of compression ratios 30-90 %% instead of the loop")
    ap.add_argument("--head-variance", action="store_true",
                    help="time the attention-variance pass of the offline head classification instead of the loop")
    args = ap.parse_args()
    args.quiet = False
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1 and args.impl == "ours":
        sys.exit(spawn_ranks(args.gpus))
    if world_env is not None and int(world_env) != args.gpus and args.impl == "ours":
        sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world_env}")
    if args.sweep:
        run_sweep(args)
    elif args.head_variance:
        run_head_variance(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
