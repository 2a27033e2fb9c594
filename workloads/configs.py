"""The five benchmark workloads: shapes, scale schedules, head-mask recipe and budgets.

Budgets are stored as plain data.  Each (budget_c, budget_s) pair was worked out by hand from
the paper's per-model allocation rules (asymmetric split, Eq. 7; the VAR rule fixes
B_C as a fraction of T_K, the Infinity rule fixes B_C : B_S = 1 : 2, appendix "Model-Specific
Configurations").  The oracle's and the library's budget splitters are each tested against these
literals; nothing here computes them.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Tuple

# Scale schedules (token-map side per scale).  N_k = side_k ** 2, T_k = sum_{i<=k} N_i.
SCHEDULES: Dict[str, Tuple[int, ...]] = {
    "256": (1, 2, 3, 4, 5, 6, 8, 10, 13, 16),                    # T_K = 680
    "512": (1, 2, 3, 4, 6, 9, 13, 18, 24, 32),                   # T_K = 2240
    "1024": (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64),     # T_K = 10521
}

BASE_SEED = 25040926


@dataclass(frozen=True)
class WorkloadConfig:
    index: int
    name: str
    n_layers: int
    n_heads: int
    head_dim: int
    batch: int
    sides: Tuple[int, ...]
    dtype: str                 # "f32" | "bf16"
    budget_frac: float         # B / T_K
    alpha: float               # global share of contextual heads
    mask_recipe: str           # "half" (heads 0..H/2-1 contextual in every layer) | "global_perm"
    sink_frac: float           # share of keys per scale that are sinks in contextual heads
    budget_rule: str           # "var" | "ratio12"   (which allocation rule produced the literals)
    budget_total: int          # B  = floor(budget_frac * T_K)
    budget_c: int              # B_C, entries per contextual head
    budget_s: int              # B_S, entries per structural head
    n_obs: int = 32
    n_init_scales: int = 2

    @property
    def n_scales(self) -> int:
        return len(self.sides)

    @property
    def tokens_per_scale(self) -> Tuple[int, ...]:
        return tuple(s * s for s in self.sides)

    @property
    def total_tokens(self) -> int:
        return sum(self.tokens_per_scale)

    @property
    def seed(self) -> int:
        return BASE_SEED + 1000 * self.index

    def with_layers(self, n_layers: int) -> "WorkloadConfig":
        """Same workload restricted to its first n_layers layers (layers are independent)."""
        return replace(self, n_layers=n_layers)


# (config, budget_frac, alpha) -> (B, B_C, B_S); hand-derived, see module docstring.
_BUDGETS = {
    (0, 0.30, 0.50): (204, 34, 374),
    (1, 0.50, 0.50): (340, 68, 612),
    (2, 0.30, 0.40): (672, 112, 1045),
    (2, 0.50, 0.40): (1120, 224, 1717),
    (2, 0.70, 0.40): (1568, 224, 2240),
    (3, 0.30, 0.50): (3156, 2104, 4208),
    # 8B-shaped sweep: contextual share 25/50/75 % x budget 10/30/50 %, rule B_C:B_S = 1:2
    (4, 0.10, 0.25): (1052, 601, 1202),
    (4, 0.30, 0.25): (3156, 1803, 3606),
    (4, 0.50, 0.25): (5260, 3005, 6010),
    (4, 0.10, 0.50): (1052, 701, 1402),
    (4, 0.30, 0.50): (3156, 2104, 4208),
    (4, 0.50, 0.50): (5260, 3506, 7012),
    (4, 0.10, 0.75): (1052, 841, 1682),
    (4, 0.30, 0.75): (3156, 2524, 5048),
    (4, 0.50, 0.75): (5260, 4208, 8416),
}

_BASE = {
    0: dict(name="single-layer-fp32-256", n_layers=1, n_heads=16, head_dim=64, batch=1,
            sides=SCHEDULES["256"], dtype="f32", budget_frac=0.30, alpha=0.50,
            mask_recipe="half", sink_frac=0.02, budget_rule="var"),
    1: dict(name="var-d16-256-bs16", n_layers=16, n_heads=16, head_dim=64, batch=16,
            sides=SCHEDULES["256"], dtype="bf16", budget_frac=0.50, alpha=0.50,
            mask_recipe="global_perm", sink_frac=0.02, budget_rule="var"),
    2: dict(name="var-d30-512-bs8", n_layers=30, n_heads=30, head_dim=64, batch=8,
            sides=SCHEDULES["512"], dtype="bf16", budget_frac=0.30, alpha=0.40,
            mask_recipe="global_perm", sink_frac=0.02, budget_rule="var"),
    3: dict(name="infinity-2b-1024-bs2", n_layers=32, n_heads=16, head_dim=128, batch=2,
            sides=SCHEDULES["1024"], dtype="bf16", budget_frac=0.30, alpha=0.50,
            mask_recipe="half", sink_frac=0.005, budget_rule="ratio12"),
    4: dict(name="wide-8b-1024-bs2", n_layers=40, n_heads=32, head_dim=128, batch=2,
            sides=SCHEDULES["1024"], dtype="bf16", budget_frac=0.30, alpha=0.50,
            mask_recipe="global_perm", sink_frac=0.02, budget_rule="ratio12"),
}


def get_config(index: int, budget_frac: float | None = None, alpha: float | None = None,
               n_layers: int | None = None) -> WorkloadConfig:
    """Workload `index` (0..4); budget_frac / alpha pick a point of the sweeps of configs 2 and 4."""
    base = dict(_BASE[index])
    if budget_frac is not None:
        base["budget_frac"] = float(budget_frac)
    if alpha is not None:
        base["alpha"] = float(alpha)
    key = (index, round(base["budget_frac"], 2), round(base["alpha"], 2))
    if key not in _BUDGETS:
        raise KeyError(f"no budget literals for config {index} at budget_frac="
                       f"{base['budget_frac']}, alpha={base['alpha']}")
    b, bc, bs = _BUDGETS[key]
    cfg = WorkloadConfig(index=index, budget_total=b, budget_c=bc, budget_s=bs, **base)
    if n_layers is not None:
        cfg = cfg.with_layers(n_layers)
    return cfg


def list_configs():
    """All (index, budget_frac, alpha) points that have budget literals."""
    return sorted(_BUDGETS.keys())
