"""Teacher-forced comparison of the CUDA path (through the C ABI) with the CPU oracle.

Per (layer, scale) step, on the same seeded inputs:
  (i)   the oracle's own fp64 scores vs the GPU's fp32 scores: |d| <= 1e-4*max(|s|,|s^|) + 1e-7;
  (ii)  the oracle's selection fed the GPU's fp32 scores must give the identical index list;
  (iii) stored K/V rows and positions after compaction are byte-equal;
  (iv)  attention output within 1e-5 (fp32) / 2e-2 (bf16) max-abs.
Feeding the GPU's scores to the oracle's selection keeps near-ties from cascading into different
cache contents; the selection itself is still decided by the oracle's own code.
With fused=True a second cache is driven through hack_scale_step on the same inputs; its stored
positions must equal the staged path's and its outputs must meet (iv) as well.
With free_running=True a second oracle decides every selection from its own fp64 scores (no teacher
forcing); the Jaccard overlap of its stored positions with the GPU's is recorded per step.  It is
information, not a pass criterion: one near-tie decided the other way changes all later steps.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import hack_oracle as ho
from workloads import SyntheticQKV, WorkloadConfig

SCORE_RTOL, SCORE_ATOL = 1e-4, 1e-7
OUT_TOL = {"f32": 1e-5, "bf16": 2e-2}


@dataclass
class ParityReport:
    workload: str
    steps: int = 0
    heads_checked: int = 0
    compressed_heads: int = 0
    max_score_err: float = 0.0          # max of |d| / (max(|s|,|s^|) + atol/rtol)
    max_out_abs: float = 0.0
    max_out_abs_fused: float = 0.0
    jaccard: List[float] = field(default_factory=list)   # free-running oracle vs GPU, per compressed (step, head)
    problems: List[str] = field(default_factory=list)

    def summary(self) -> str:
        return (f"{self.workload}: steps={self.steps} heads={self.heads_checked} "
                f"compressed={self.compressed_heads} score_err={self.max_score_err:.2e} "
                f"out_abs={self.max_out_abs:.2e} fused_out_abs={self.max_out_abs_fused:.2e} "
                + (f"jaccard(min/mean)={min(self.jaccard):.4f}/{sum(self.jaccard) / len(self.jaccard):.4f} "
                   if self.jaccard else "")
                + f"problems={len(self.problems)}")

    def ok(self) -> bool:
        return not self.problems


def _torch_dtype(cfg: WorkloadConfig):
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def make_cache(cfg: WorkloadConfig, mask: np.ndarray, policy: int = 0, budget_c: Optional[int] = None,
               budget_s: Optional[int] = None, device: int = 0, obs_sampler: int = 0, obs_rows=None):
    from paper_2504_09261_b200 import HACK_BF16, HACK_F32, HackCache
    cache = HackCache(cfg.n_layers, cfg.n_heads, cfg.head_dim, cfg.batch, cfg.sides,
                      HACK_F32 if cfg.dtype == "f32" else HACK_BF16, mask,
                      cfg.budget_c if budget_c is None else budget_c,
                      cfg.budget_s if budget_s is None else budget_s,
                      n_obs=cfg.n_obs, n_init_scales=cfg.n_init_scales, overflow_policy=policy,
                      device=device, obs_sampler=obs_sampler)
    if obs_rows is not None:
        for k, rows in enumerate(obs_rows):
            cache.hack_set_obs_rows(k, rows)
    return cache


def sample_heads(cfg: WorkloadConfig, layer: int, n: Optional[int]) -> List[Tuple[int, int]]:
    pairs = [(b, h) for b in range(cfg.batch) for h in range(cfg.n_heads)]
    if n is None or n >= len(pairs):
        return pairs
    rng = np.random.default_rng(1000 + layer)
    sel = rng.choice(len(pairs), size=n, replace=False)
    return [pairs[i] for i in sorted(sel.tolist())]


def _rows_bytes(arr64: np.ndarray, tdt) -> bytes:
    t = torch.from_numpy(np.ascontiguousarray(arr64)).to(tdt).contiguous()
    return t.view(torch.uint8).numpy().tobytes() if t.numel() else b""


def run_parity(cfg: WorkloadConfig, layers: Sequence[int], fused: bool = False,
               heads_per_layer: Optional[int] = None, policy: int = 0,
               budget_c: Optional[int] = None, budget_s: Optional[int] = None,
               scales: Optional[int] = None, check_rows: bool = True,
               obs_sampler: int = 0, obs_rows=None, pairs_of=None, gen_on_gpu: bool = False,
               free_running: bool = False, staged_cache=None) -> ParityReport:
    """pairs_of: {layer: [(b, h), ...]} overrides the per-layer sample; gen_on_gpu: the seeded
    generator runs on the device and the oracle reads a host copy of the same bytes (the large
    workloads would spend minutes in the CPU generator otherwise); staged_cache: a cache of the
    same configuration to run the staged calls on (it is reset first and left open)."""
    dev = torch.device("cuda:0")
    tdt = _torch_dtype(cfg)
    gen = SyntheticQKV(cfg, device=dev if gen_on_gpu else "cpu")
    mask = gen.head_is_contextual.numpy()
    b_c = cfg.budget_c if budget_c is None else budget_c
    b_s = cfg.budget_s if budget_s is None else budget_s
    orc = ho.HackOracle(cfg.n_layers, cfg.n_heads, cfg.batch, cfg.head_dim, cfg.sides, mask, b_c, b_s,
                        n_obs=cfg.n_obs, n_init_scales=cfg.n_init_scales, overflow_policy=policy,
                        obs_sampler=obs_sampler, obs_rows=obs_rows)
    if staged_cache is not None:
        staged = staged_cache
        staged.hack_reset()
    else:
        staged = make_cache(cfg, mask, policy, b_c, b_s, obs_sampler=obs_sampler, obs_rows=obs_rows)
    twin = make_cache(cfg, mask, policy, b_c, b_s, obs_sampler=obs_sampler, obs_rows=obs_rows) if fused else None
    rep = ParityReport(cfg.name)
    bh = cfg.batch * cfg.n_heads
    H = cfg.n_heads
    n_scales = cfg.n_scales if scales is None else scales
    if pairs_of is None:
        pairs_of = {l: sample_heads(cfg, l, heads_per_layer) for l in layers}
    free = None
    if free_running:
        free = ho.HackOracle(cfg.n_layers, cfg.n_heads, cfg.batch, cfg.head_dim, cfg.sides, mask, b_c, b_s,
                             n_obs=cfg.n_obs, n_init_scales=cfg.n_init_scales, overflow_policy=policy,
                             obs_sampler=obs_sampler, obs_rows=obs_rows)
    out_tol = OUT_TOL[cfg.dtype]
    scores = torch.empty((bh, staged.cand_stride), dtype=torch.float32, device=dev)
    idx = torch.empty((bh, staged.kept_stride), dtype=torch.int32, device=dev)
    kept = torch.empty((bh,), dtype=torch.int32, device=dev)

    def note(msg):
        if len(rep.problems) < 20:
            rep.problems.append(msg)

    for k in range(n_scales):
        for l in layers:
            q, kk, v = gen.qkv(l, k)
            qd, kd, vd = q.to(dev), kk.to(dev), v.to(dev)
            q, kk, v = q.cpu(), kk.cpu(), v.cpu()
            out = torch.full_like(qd, float("nan"))
            info = staged.hack_step_info(l, k)
            scores.fill_(float("nan"))
            idx.fill_(-1)
            kept.fill_(-1)
            staged.hack_score(l, k, qd, kd, scores)
            staged.hack_select(l, k, scores, idx, kept)
            staged.hack_compact(l, k, idx, kd, vd)
            staged.hack_attend(l, k, qd, out)
            if fused:
                out_f = torch.full_like(qd, float("nan"))
                twin.hack_scale_step(l, k, qd, kd, vd, out_f)
            torch.cuda.synchronize()
            staged.hack_poll_status()
            s_h = scores.cpu().numpy()
            idx_h = idx.cpu().numpy()
            kept_h = kept.cpu().numpy()
            pairs = pairs_of[l]
            override = {}
            for (b, h) in pairs:
                ctx = int(mask[l, h])
                trig = info.triggered_c if ctx else info.triggered_s
                cand = info.cand_c if ctx else info.cand_s
                if trig:
                    override[(b, h)] = s_h[b * H + h, :cand].astype(np.float64)
            if 2 * len(pairs) < bh:
                # only the sampled heads are widened (the rest of the arrays is never read)
                q64, k64, v64 = (np.zeros(tuple(t.shape)) for t in (q, kk, v))
                for (b, h) in pairs:
                    q64[b, h], k64[b, h], v64[b, h] = (t[b, h].to(torch.float64).numpy() for t in (q, kk, v))
            else:
                q64, k64, v64 = (t.to(torch.float64).numpy() for t in (q, kk, v))
            o_ref, recs = orc.scale_step(l, k, q64, k64, v64, scores_override=override, heads=pairs)
            if free is not None:
                free.scale_step(l, k, q64, k64, v64, heads=pairs, need_output=False)
            lengths = staged.hack_get_lengths(l)
            for (b, h) in pairs:
                tag = f"layer {l} scale {k} b {b} h {h}"
                r = b * H + h
                ctx = int(mask[l, h])
                rec = recs[(b, h)]
                trig = bool(info.triggered_c if ctx else info.triggered_s)
                cand = info.cand_c if ctx else info.cand_s
                n_keep = info.kept_c if ctx else info.kept_s
                rep.heads_checked += 1
                if rec.n_candidates != cand or rec.compressed != trig:
                    note(f"{tag}: plan mismatch (cand {cand} vs {rec.n_candidates}, trig {trig} vs {rec.compressed})")
                    continue
                if trig:
                    rep.compressed_heads += 1
                    sg = s_h[r, :cand].astype(np.float64)
                    if not np.all(np.isfinite(sg)):
                        note(f"{tag}: non-finite GPU scores")
                        continue
                    den = SCORE_RTOL * np.maximum(np.abs(sg), np.abs(rec.scores)) + SCORE_ATOL
                    err = float(np.max(np.abs(sg - rec.scores) / den))
                    rep.max_score_err = max(rep.max_score_err, err)
                    if err > 1.0:
                        note(f"{tag}: score error {err:.3f} x tolerance")
                if kept_h[r] != len(rec.keep) or n_keep != len(rec.keep) or lengths[r] != len(rec.keep):
                    note(f"{tag}: kept count gpu {kept_h[r]} plan {n_keep} oracle {len(rec.keep)}")
                    continue
                if not np.array_equal(idx_h[r, :n_keep].astype(np.int64), rec.keep):
                    bad = int(np.sum(idx_h[r, :n_keep].astype(np.int64) != rec.keep))
                    note(f"{tag}: index list differs in {bad} of {n_keep} places")
                if check_rows:
                    st = orc.state[l][b][h]
                    pos_g = np.frombuffer(staged.hack_read_head(l, b, h, 2), dtype=np.int32)
                    if not np.array_equal(pos_g.astype(np.int64), st.pos):
                        note(f"{tag}: stored positions differ")
                    if free is not None and trig:
                        pf = free.state[l][b][h].pos
                        inter = np.intersect1d(pos_g.astype(np.int64), pf).shape[0]
                        rep.jaccard.append(inter / max(pos_g.shape[0] + pf.shape[0] - inter, 1))
                    if staged.hack_read_head(l, b, h, 0) != _rows_bytes(st.k, tdt):
                        note(f"{tag}: stored K rows are not byte-equal")
                    if staged.hack_read_head(l, b, h, 1) != _rows_bytes(st.v, tdt):
                        note(f"{tag}: stored V rows are not byte-equal")
                    if fused:
                        pos_f = np.frombuffer(twin.hack_read_head(l, b, h, 2), dtype=np.int32)
                        if not np.array_equal(pos_f, pos_g):
                            note(f"{tag}: fused path kept a different set")
                d = float(np.max(np.abs(out[b, h].to(torch.float64).cpu().numpy() - o_ref[b, h])))
                if not np.isfinite(d):
                    d = float("inf")
                rep.max_out_abs = max(rep.max_out_abs, d)
                if d > out_tol:
                    note(f"{tag}: attention output off by {d:.3e} (tol {out_tol})")
                if fused:
                    df = float(np.max(np.abs(out_f[b, h].to(torch.float64).cpu().numpy() - o_ref[b, h])))
                    if not np.isfinite(df):
                        df = float("inf")
                    rep.max_out_abs_fused = max(rep.max_out_abs_fused, df)
                    if df > out_tol:
                        note(f"{tag}: fused attention output off by {df:.3e} (tol {out_tol})")
            rep.steps += 1
    if staged_cache is None:
        staged.close()
    if twin is not None:
        twin.close()
    return rep
