"""CPU oracle for the HACK per-scale decoding step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, double-precision restatement of what one (layer, scale) step of head-aware
KV-cache compression computes in a next-scale visual autoregressive transformer: append the new
scale's keys/values (Eq. 3), score every candidate key with a small query subset (Eq. 9), pick a
budgeted subset per head with the contextual rule (Eq. 10) or the structural rule (Eq. 11),
gather the survivors, and attend over them (Eq. 4 applied to the compressed cache, Eq. 5/8).
One (batch, head) at a time, no blocking, no fusion; numpy matmul / argsort / exp serve as steps.

It shares no code with the CUDA path and must never be imported by the product package: only
the tests, the smoke check and the CPU-baseline leg of the benchmark may use it.

Parity pins (see tests/test_oracle_*.py): full-budget == vanilla attention (Eq. 3-4), softmax
row sums, brute-force subset selection, protected-scale invariants, the closed forms of the
complexity analysis (Eq. 12-22), convexity and permutation invariance of the attention output.
The final-scale merge of contextual heads (merge_assign, merge_apply) follows one sentence of the
paper; the similarity measure, the weights and the treatment of V are a reading: parity unpinned
(pins cover only what the reading itself fixes: special cases, an explicit loop, convexity).
Offline head classification (Eq. 6) is here too: attention_variance and classify_heads, pinned by
closed forms (identity and uniform attention) and by recovering a planted head mask.
Parity unpinned (the paper is silent; only self-consistency is tested): the overflow rule when
B_S < N_init + N_k, the exact stride of the "uniform" query sample, the budget rounding rule.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

KEEP_PROTECTED = 0   # overflow policy 0: every protected entry stays even if that exceeds B_S
COMPETE = 1          # overflow policy 1: only the initial scales are protected


# --------------------------------------------------------------------------- budgets (Eq. 7)
def split_budget(budget: int, alpha: float, rule: str, param: float, total_tokens: int) -> Tuple[int, int]:
    """Per-type budgets (B_C, B_S) with alpha*B_C + (1-alpha)*B_S <= B  (Eq. 7).

    rule "fraction": B_C = floor(param * T_K) is given directly (the class-conditional setting);
                     B_S = floor((B - alpha*B_C) / (1 - alpha)).
    rule "ratio":    B_C : B_S = 1 : param (the text-to-image setting, param = 2);
                     B_C = floor(B / (alpha + param*(1-alpha))), B_S = param * B_C.
    B_S is clamped to T_K, both are at least 1.
    """
    if not (0.0 < alpha < 1.0):
        raise ValueError("alpha must lie strictly between 0 and 1")
    if rule == "fraction":
        b_c = int(math.floor(param * total_tokens + 1e-9))
        b_s = int(math.floor((budget - alpha * b_c) / (1.0 - alpha) + 1e-9))
    elif rule == "ratio":
        b_c = int(math.floor(budget / (alpha + param * (1.0 - alpha)) + 1e-9))
        b_s = int(round(param * b_c))
    else:
        raise ValueError(rule)
    b_s = min(b_s, total_tokens)
    return max(b_c, 1), max(b_s, 1)


# --------------------------------------------------------------------------- step pieces
UNIFORM, INIT, RECENT, CALLER, FULL = 0, 1, 2, 3, 4   # query-subset rules of the sampling ablation


def observation_rows(n_k: int, n_obs: int, sampler: int = UNIFORM,
                     caller_rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Indices of the query subset Q~ of Eq. 9, n = min(N_obs, N_k) rows of the current scale.

    UNIFORM (the method's rule): floor(m * N_k / n).  INIT: the first n tokens.  RECENT: the last n
    tokens.  CALLER: rows drawn outside (the ablation's random sampling), n distinct indices given in
    `caller_rows`, used in the order given.  FULL: every query of the scale, whatever N_obs (the
    ablation's "full attention" reference).  These are the alternatives the paper's query-subset
    ablation compares the uniform rule with."""
    if sampler == FULL:
        return np.arange(n_k, dtype=np.int64)
    n = min(n_obs, n_k)
    if sampler == UNIFORM:
        return np.array([(m * n_k) // n for m in range(n)], dtype=np.int64)
    if sampler == INIT:
        return np.arange(n, dtype=np.int64)
    if sampler == RECENT:
        return np.arange(n_k - n, n_k, dtype=np.int64)
    if sampler == CALLER:
        rows = np.asarray(caller_rows, dtype=np.int64)
        if rows.shape != (n,) or rows.min() < 0 or rows.max() >= n_k or len(set(rows.tolist())) != n:
            raise ValueError("caller_rows must hold min(N_obs, N_k) distinct rows of the current scale")
        return rows
    raise ValueError(sampler)


def softmax_rows(z: np.ndarray) -> np.ndarray:
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=1, keepdims=True)


def subset_attention_scores(q_obs: np.ndarray, k_cand: np.ndarray, sm_scale: float) -> np.ndarray:
    """s_j = sum_i Softmax(sm_scale * Q~ K^T)[i, j]  (Eq. 9 and the TOPK argument of Eq. 10/11)."""
    a = softmax_rows(sm_scale * (q_obs @ k_cand.T))
    return a.sum(axis=0)


def top_indices(s: np.ndarray, n: int) -> np.ndarray:
    """The n entries with the largest score; ties go to the lower index.  Returned ascending."""
    if n <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.argsort(-s, kind="stable")      # score descending, index ascending among equals
    return np.sort(order[:n])


def select_contextual(s: np.ndarray, budget_c: int) -> np.ndarray:
    """Eq. 10: keep the B_C candidates with the highest cumulative attention."""
    return top_indices(s, min(budget_c, s.shape[0]))


def select_structural(s: np.ndarray, scale_id: np.ndarray, k: int, n_init_scales: int,
                      budget_s: int, policy: int = KEEP_PROTECTED) -> np.ndarray:
    """Eq. 11: keep the initial scales and the latest scale, fill the rest (M) by score.

    scale_id[j] is the 1-based scale that produced candidate j, k the scale being decoded.
    """
    if policy == KEEP_PROTECTED:
        prot = (scale_id <= n_init_scales) | (scale_id == k)
    else:
        prot = scale_id <= n_init_scales
    m = budget_s - int(prot.sum())
    free = np.nonzero(~prot)[0]
    chosen = free[top_indices(s[free], min(max(m, 0), free.shape[0]))]
    return np.sort(np.concatenate([np.nonzero(prot)[0], chosen]))


def attend(q: np.ndarray, k_hat: np.ndarray, v_hat: np.ndarray, sm_scale: float) -> np.ndarray:
    """Eq. 4 on the compressed cache: O = Softmax(sm_scale * Q K^T) V, no mask inside a scale."""
    return softmax_rows(sm_scale * (q @ k_hat.T)) @ v_hat


# --------------------------------------------------------------------------- final-scale merge
def merge_assign(k_evicted: np.ndarray, k_kept: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Nearest retained counterpart of every discarded key, and its weight.

    The paper gives the merge one sentence (contextual-head strategy, after Eq. 10): discarded KV
    tokens of the last step are folded into their nearest retained counterparts by similarity-weighted
    averaging.  Reading taken here (the paper is silent on all three points): nearness is the cosine
    similarity between keys; the counterpart is the retained key with the largest similarity, the
    lowest index among equals; the weight is that similarity, or 0 if it is negative.
    Returns (index into the kept list, weight) per discarded entry."""
    ne = np.linalg.norm(k_evicted, axis=1, keepdims=True)
    nk = np.linalg.norm(k_kept, axis=1, keepdims=True)
    cos = (k_evicted @ k_kept.T) / np.maximum(ne * nk.T, 1e-300)
    assign = np.argmax(cos, axis=1).astype(np.int64)
    weight = np.maximum(cos[np.arange(cos.shape[0]), assign], 0.0)
    return assign, weight


def merge_apply(k_kept: np.ndarray, v_kept: np.ndarray, k_evicted: np.ndarray, v_evicted: np.ndarray,
                assign: np.ndarray, weight: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Similarity-weighted average of every retained entry with the discarded entries assigned to it:
    k_c <- (k_c + sum_e w_e k_e) / (1 + sum_e w_e), the same weights for v_c (the retained entry
    itself has similarity 1).  Entries without assignments are unchanged."""
    num_k, num_v = k_kept.copy(), v_kept.copy()
    den = np.ones(k_kept.shape[0])
    for e in range(k_evicted.shape[0]):
        c = int(assign[e])
        num_k[c] += weight[e] * k_evicted[e]
        num_v[c] += weight[e] * v_evicted[e]
        den[c] += weight[e]
    return num_k / den[:, None], num_v / den[:, None]


# --------------------------------------------------------------------------- state
@dataclass
class HeadCache:
    k: np.ndarray
    v: np.ndarray
    pos: np.ndarray        # global token position of each stored entry
    sid: np.ndarray        # 1-based scale that produced each stored entry


@dataclass
class StepRecord:
    """What one (batch, head) did in one step; candidate indices refer to [stored ; new]."""
    compressed: bool
    n_candidates: int
    scores: Optional[np.ndarray]      # fp64 scores the oracle computed (None if not triggered)
    keep: np.ndarray                  # ascending candidate indices that survive
    pos: np.ndarray                   # their global token positions
    evicted: Optional[np.ndarray] = None        # final-scale merge: ascending candidate indices discarded
    merge_assign: Optional[np.ndarray] = None   # ... index into `keep` each of them was folded into
    merge_weight: Optional[np.ndarray] = None   # ... and its weight
    evicted_k: Optional[np.ndarray] = None      # ... the discarded rows themselves
    evicted_v: Optional[np.ndarray] = None
    kept_k_before: Optional[np.ndarray] = None  # ... and the retained rows before the fold
    kept_v_before: Optional[np.ndarray] = None


@dataclass
class Counters:
    attention_pairs: int = 0          # sum N_k * |stored|
    score_pairs: int = 0              # sum n * T'
    peak_entries: int = 0             # peak of sum |stored| over the whole stack
    overflows: int = 0                # steps in which a head kept more than its budget


class HackOracle:
    """Per-(layer, batch, head) cache state plus the step-by-step algorithm."""

    def __init__(self, n_layers: int, n_heads: int, batch: int, head_dim: int,
                 sides: Sequence[int], head_is_contextual: np.ndarray,
                 budget_c: int, budget_s: int, n_obs: int = 32, n_init_scales: int = 2,
                 sm_scale: Optional[float] = None, overflow_policy: int = KEEP_PROTECTED,
                 obs_sampler: int = UNIFORM, obs_rows: Optional[Sequence[Sequence[int]]] = None,
                 merge_last: bool = False):
        self.L, self.H, self.b, self.D = n_layers, n_heads, batch, head_dim
        self.sides = tuple(int(s) for s in sides)
        self.N = tuple(s * s for s in self.sides)
        self.T = tuple(int(x) for x in np.cumsum(self.N))
        self.is_ctx = np.asarray(head_is_contextual, dtype=bool).reshape(n_layers, n_heads)
        self.budget_c, self.budget_s = int(budget_c), int(budget_s)
        self.n_obs, self.n_init_scales = int(n_obs), int(n_init_scales)
        self.sm_scale = float(sm_scale) if sm_scale else 1.0 / math.sqrt(head_dim)
        self.policy = overflow_policy
        self.obs_sampler = obs_sampler
        self.obs_rows = obs_rows            # CALLER: one row list per scale
        self.merge_last = bool(merge_last)  # contextual heads fold what the last scale evicts into what it keeps
        self.counters = Counters()
        self.reset()

    def reset(self) -> None:
        D = self.D
        self.state: List[List[List[HeadCache]]] = [
            [[HeadCache(np.zeros((0, D)), np.zeros((0, D)), np.zeros(0, np.int64), np.zeros(0, np.int64))
              for _ in range(self.H)] for _ in range(self.b)] for _ in range(self.L)]
        self.next_scale = [0] * self.L
        self._live = 0

    def budget_of(self, layer: int, head: int) -> int:
        return self.budget_c if self.is_ctx[layer, head] else self.budget_s

    def stored_lengths(self, layer: int) -> np.ndarray:
        return np.array([[self.state[layer][b][h].k.shape[0] for h in range(self.H)]
                         for b in range(self.b)], dtype=np.int64)

    # ----------------------------------------------------------------------- one head
    def head_step(self, layer: int, scale: int, b: int, h: int, q: np.ndarray, k_new: np.ndarray,
                  v_new: np.ndarray, scores_override: Optional[np.ndarray] = None,
                  need_output: bool = True,
                  assign_override: Optional[np.ndarray] = None) -> Tuple[Optional[np.ndarray], StepRecord]:
        """One (batch, head) of one step.  `scale` is 0-based here, the paper's k is scale + 1.

        scores_override: fp32/fp64 scores over the candidates to be used for the selection in
        place of the oracle's own (teacher forcing, so near-ties cannot cascade).
        assign_override: with the final-scale merge, the counterpart of every discarded entry to be
        used in place of the oracle's own argmax (same reason); the weights are then the similarities
        to those counterparts.
        """
        k1 = scale + 1
        n_k = self.N[scale]
        st = self.state[layer][b][h]
        # 1. candidates = stored ++ new (Eq. 3; the key set of the detailed complexity analysis)
        k_c = np.concatenate([st.k, k_new], axis=0)
        v_c = np.concatenate([st.v, v_new], axis=0)
        pos_c = np.concatenate([st.pos, self.T[scale] - n_k + np.arange(n_k, dtype=np.int64)])
        sid_c = np.concatenate([st.sid, np.full(n_k, k1, dtype=np.int64)])
        t_cand = k_c.shape[0]
        budget = self.budget_of(layer, h)
        scores = None
        # 2. compression happens before attention, only when the cache exceeds the budget
        if t_cand <= budget:
            keep = np.arange(t_cand, dtype=np.int64)
            compressed = False
        else:
            compressed = True
            obs = observation_rows(n_k, self.n_obs, self.obs_sampler,
                                   self.obs_rows[scale] if self.obs_sampler == CALLER else None)
            scores = subset_attention_scores(q[obs], k_c, self.sm_scale)
            self.counters.score_pairs += obs.shape[0] * t_cand
            s_sel = scores if scores_override is None else np.asarray(scores_override, dtype=np.float64)
            assert s_sel.shape[0] == t_cand
            if self.is_ctx[layer, h]:
                keep = select_contextual(s_sel, budget)
            else:
                keep = select_structural(s_sel, sid_c, k1, self.n_init_scales, budget, self.policy)
            if keep.shape[0] > budget:
                self.counters.overflows += 1
        # 3. gather survivors in ascending position
        self._live += keep.shape[0] - st.k.shape[0]
        st.k, st.v, st.pos, st.sid = k_c[keep], v_c[keep], pos_c[keep], sid_c[keep]
        # 3b. only at the final scale, only in contextual heads: fold the discarded entries of this
        # step into their nearest retained counterparts
        evicted = m_assign = m_weight = ev_k = ev_v = kk_before = kv_before = None
        if self.merge_last and compressed and scale == len(self.N) - 1 and self.is_ctx[layer, h]:
            gone = np.ones(t_cand, dtype=bool)
            gone[keep] = False
            evicted = np.nonzero(gone)[0]
            m_assign, m_weight = merge_assign(k_c[evicted], st.k)
            if assign_override is not None:
                m_assign = np.asarray(assign_override, dtype=np.int64)
                ke, kk = k_c[evicted], st.k[m_assign]
                cos = (ke * kk).sum(axis=1) / np.maximum(np.linalg.norm(ke, axis=1) * np.linalg.norm(kk, axis=1), 1e-300)
                m_weight = np.maximum(cos, 0.0)
            ev_k, ev_v, kk_before, kv_before = k_c[evicted], v_c[evicted], st.k, st.v
            st.k, st.v = merge_apply(st.k, st.v, ev_k, ev_v, m_assign, m_weight)
        # 4. attention of all N_k queries over the compressed cache
        out = None
        if need_output:
            out = attend(q, st.k, st.v, self.sm_scale)
        self.counters.attention_pairs += n_k * keep.shape[0]
        return out, StepRecord(compressed, t_cand, scores, keep, st.pos.copy(), evicted, m_assign, m_weight,
                               ev_k, ev_v, kk_before, kv_before)

    # ----------------------------------------------------------------------- all heads
    def scale_step(self, layer: int, scale: int, q: np.ndarray, k: np.ndarray, v: np.ndarray,
                   scores_override: Optional[Dict[Tuple[int, int], np.ndarray]] = None,
                   heads: Optional[Sequence[Tuple[int, int]]] = None,
                   need_output: bool = True):
        """One (layer, scale) step on Q, K, V of shape [b, H, N_k, D] (fp64 arrays).

        Returns (O [b, H, N_k, D] fp64, records {(b, h): StepRecord}).  With `heads`, only those
        (b, h) pairs are advanced (their outputs filled, the rest left at zero).
        """
        if scale != self.next_scale[layer]:
            raise RuntimeError(f"layer {layer} expects scale {self.next_scale[layer]}, got {scale}")
        n_k = self.N[scale]
        assert q.shape == (self.b, self.H, n_k, self.D), q.shape
        out = np.zeros((self.b, self.H, n_k, self.D))
        records: Dict[Tuple[int, int], StepRecord] = {}
        pairs = heads if heads is not None else [(b, h) for b in range(self.b) for h in range(self.H)]
        for (b, h) in pairs:
            ov = None if scores_override is None else scores_override.get((b, h))
            o, rec = self.head_step(layer, scale, b, h, q[b, h], k[b, h], v[b, h], ov, need_output)
            if o is not None:
                out[b, h] = o
            records[(b, h)] = rec
        self.next_scale[layer] = scale + 1
        self.counters.peak_entries = max(self.counters.peak_entries, self._live)
        return out, records


# --------------------------------------------------------------------------- offline head classification
def attention_variance(q: np.ndarray, k: np.ndarray, sm_scale: float) -> float:
    """sigma = sum_j Var_i A[i, j] for one head (Eq. 6): A = Softmax(sm_scale * Q K^T) is the
    attention matrix of the step's queries (rows) over the cached keys (columns); the variance of a
    column is taken over the queries, as the population variance (mean of squares minus squared
    mean; the paper does not say which normalisation, and the ranking does not depend on it)."""
    a = softmax_rows(sm_scale * (q @ k.T))
    return float(np.var(a, axis=0).sum())


def classify_heads(sigma: np.ndarray, alpha: float) -> np.ndarray:
    """Head types from the variance matrix sigma [L, H] (averaged over samples by the caller): all
    heads are ranked globally by sigma and the round(alpha * L * H) lowest become contextual (1),
    the others structural (0).  Equal values are ranked by (layer, head)."""
    sigma = np.asarray(sigma, dtype=np.float64)
    flat = sigma.reshape(-1)
    n_ctx = int(math.floor(alpha * flat.shape[0] + 0.5))
    order = np.argsort(flat, kind="stable")
    mask = np.zeros(flat.shape[0], dtype=np.uint8)
    mask[order[:n_ctx]] = 1
    return mask.reshape(sigma.shape)


# --------------------------------------------------------------------------- vanilla reference
def vanilla_var_attention(q_scales: Sequence[np.ndarray], k_scales: Sequence[np.ndarray],
                          v_scales: Sequence[np.ndarray], sm_scale: float) -> List[np.ndarray]:
    """Uncompressed next-scale attention for ONE head (Eq. 3-4): scale k sees scales <= k.

    Written as the definition (one full softmax per query row), independently of HackOracle.
    """
    outs = []
    for k in range(len(q_scales)):
        keys = np.concatenate(k_scales[: k + 1], axis=0)
        vals = np.concatenate(v_scales[: k + 1], axis=0)
        o = np.zeros_like(q_scales[k])
        for i in range(q_scales[k].shape[0]):
            z = sm_scale * (keys @ q_scales[k][i])
            w = np.exp(z - z.max())
            o[i] = (w / w.sum()) @ vals
        outs.append(o)
    return outs
