"""Seeded synthetic Q/K/V with the two attention patterns the paper describes.

Contextual heads attend "vertically" (a few sink keys attract every query); structural heads
attend locally in space (a 2-D sinusoidal code of the token's grid coordinates, rescaled to each
scale, is added to both Q and K).  The generator is counter based: every element is a pure
function of (seed, layer, tensor, batch, head, global token index, dim), so a tensor for one
(layer, scale) can be produced on its own, on the CPU or on a CUDA device, from the same code.

This module generates inputs only; it contains none of the method's arithmetic.
"""
from __future__ import annotations

import math
from typing import Dict, Tuple

import torch

from .configs import WorkloadConfig

_MASK64 = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15      # splitmix64 increment
_MUL1 = 0xBF58476D1CE4E5B9       # splitmix64 finaliser multipliers
_MUL2 = 0x94D049BB133111EB

_TENSOR_Q, _TENSOR_K, _TENSOR_V, _TENSOR_U, _TENSOR_SINK, _TENSOR_MASK = range(6)


def _i64(x: int) -> int:
    """Python int (mod 2^64) as the signed 64-bit value with the same bit pattern."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _finalise(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on int64 bit patterns (wrap-around arithmetic)."""
    z = (z ^ _lsr(z, 30)) * _i64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _i64(_MUL2)
    return z ^ _lsr(z, 31)


def _finalise_int(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _MUL1) & _MASK64
    z = ((z ^ (z >> 27)) * _MUL2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, layer: int, tensor: int, extra: int = 0) -> int:
    """Key of one random stream: hash of (seed, layer, tensor, extra)."""
    z = _finalise_int(seed + _GAMMA)
    z = _finalise_int(z ^ ((layer + 1) * _GAMMA))
    z = _finalise_int(z ^ ((tensor + 1) * _MUL1))
    z = _finalise_int(z ^ ((extra + 1) * _MUL2))
    return z


def _uniform(key: int, counter: torch.Tensor) -> torch.Tensor:
    """Uniform in (0, 1) with 53 random bits, for int64 counters, stream `key`."""
    z = _finalise(counter * _i64(_GAMMA) + _i64(key))
    return (_lsr(z, 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal(key: int, counter: torch.Tensor) -> torch.Tensor:
    """Standard normal via Box-Muller on two uniforms drawn at counters 2c and 2c+1 (fp64)."""
    u1 = _uniform(key, counter * 2)
    u2 = _uniform(key, counter * 2 + 1)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def _hash_u64(key: int, counter: torch.Tensor) -> torch.Tensor:
    """Non-negative 62-bit hash, used only to rank positions."""
    return _lsr(_finalise(counter * _i64(_GAMMA) + _i64(key)), 2)


class SyntheticQKV:
    """Generator of per-(layer, scale) Q, K, V for one workload."""

    def __init__(self, cfg: WorkloadConfig, device: str | torch.device = "cpu", seed_offset: int = 0):
        self.cfg = cfg
        self.seed = cfg.seed + 7919 * seed_offset      # the head mask does not depend on the offset
        self.device = torch.device(device)
        self.tokens = cfg.tokens_per_scale
        self.starts = [0]
        for n in self.tokens:
            self.starts.append(self.starts[-1] + n)
        self.total = self.starts[-1]
        self._mask = self._make_mask()
        self._pos_code_cache: Dict[Tuple[int, str], torch.Tensor] = {}

    # ------------------------------------------------------------------ head mask
    def _make_mask(self) -> torch.Tensor:
        c = self.cfg
        L, H = c.n_layers, c.n_heads
        if c.mask_recipe == "half":
            row = torch.zeros(H, dtype=torch.uint8)
            row[: H // 2] = 1
            return row.repeat(L, 1).contiguous()
        if c.mask_recipe == "global_perm":
            # ranks of a seeded hash over the full stack of the named workload, so that a
            # layer-restricted copy of the workload sees the same masks for the layers it keeps
            full_layers = _FULL_LAYERS[c.index]
            n = full_layers * H
            h = _hash_u64(stream_key(c.seed, 0, _TENSOR_MASK), torch.arange(n, dtype=torch.int64))
            order = torch.argsort(h, stable=True)
            n_ctx = int(round(c.alpha * n))
            flat = torch.zeros(n, dtype=torch.uint8)
            flat[order[:n_ctx]] = 1
            return flat.view(full_layers, H)[:L].contiguous()
        raise ValueError(c.mask_recipe)

    @property
    def head_is_contextual(self) -> torch.Tensor:
        """uint8 [n_layers, n_heads]; 1 = contextual, 0 = structural (CPU tensor)."""
        return self._mask

    # ------------------------------------------------------------------ pieces
    def _base_normal(self, layer: int, tensor: int, scale: int) -> torch.Tensor:
        """iid N(0,1) of shape [b, H, N_k, D] in fp64; counter = flat index in [b, H, T_K, D]."""
        c = self.cfg
        dev = self.device
        n_k, t0 = self.tokens[scale], self.starts[scale]
        b = torch.arange(c.batch, dtype=torch.int64, device=dev).view(-1, 1, 1, 1)
        h = torch.arange(c.n_heads, dtype=torch.int64, device=dev).view(1, -1, 1, 1)
        t = torch.arange(t0, t0 + n_k, dtype=torch.int64, device=dev).view(1, 1, -1, 1)
        d = torch.arange(c.head_dim, dtype=torch.int64, device=dev).view(1, 1, 1, -1)
        counter = ((b * c.n_heads + h) * self.total + t) * c.head_dim + d
        return _normal(stream_key(self.seed + layer, layer, tensor), counter)

    def _sink_direction(self, layer: int) -> torch.Tensor:
        """Unit vector u_{l,h} per head, [H, D] fp64 (shared over batch and scales)."""
        c = self.cfg
        idx = torch.arange(c.n_heads * c.head_dim, dtype=torch.int64, device=self.device)
        g = _normal(stream_key(self.seed + layer, layer, _TENSOR_U), idx).view(c.n_heads, c.head_dim)
        return g / torch.linalg.vector_norm(g, dim=1, keepdim=True)

    def sink_positions(self, layer: int, scale: int) -> torch.Tensor:
        """bool [H, N_k]: which keys of this scale are sinks (meaningful for contextual heads)."""
        c = self.cfg
        n_k = self.tokens[scale]
        n_sink = max(1, int(round(c.sink_frac * n_k)))
        idx = torch.arange(c.n_heads * n_k, dtype=torch.int64, device=self.device)
        hsh = _hash_u64(stream_key(self.seed + layer, layer, _TENSOR_SINK, scale), idx).view(c.n_heads, n_k)
        order = torch.argsort(hsh, dim=1, stable=True)
        flag = torch.zeros(c.n_heads, n_k, dtype=torch.bool, device=self.device)
        flag.scatter_(1, order[:, :n_sink], True)
        return flag

    def _position_code(self, scale: int) -> torch.Tensor:
        """2-D sinusoidal code of the token grid of this scale, [N_k, D] fp64, |p|^2 = sqrt(D)."""
        key = (scale, str(self.device))
        if key in self._pos_code_cache:
            return self._pos_code_cache[key]
        c = self.cfg
        dev = self.device
        side, D = c.sides[scale], c.head_dim
        q = D // 4
        s_max = max(c.sides)
        r = torch.arange(side, dtype=torch.float64, device=dev)
        y = ((r + 0.5) / side).view(side, 1).expand(side, side).reshape(-1, 1)   # row coordinate
        x = ((r + 0.5) / side).view(1, side).expand(side, side).reshape(-1, 1)   # column coordinate
        m = torch.arange(q, dtype=torch.float64, device=dev)
        omega = 2.0 * math.pi * (s_max / 2.0) ** (m / max(q - 1, 1))
        p = torch.cat([torch.sin(omega * y), torch.cos(omega * y),
                       torch.sin(omega * x), torch.cos(omega * x)], dim=1)       # |p|^2 = D/2
        p = p * math.sqrt(math.sqrt(D) / (D / 2.0))
        self._pos_code_cache[key] = p
        return p

    # ------------------------------------------------------------------ public
    def qkv(self, layer: int, scale: int, as_float64: bool = False):
        """Q, K, V of shape [b, H, N_k, D] for 0-based (layer, scale), in the workload's dtype.

        With as_float64 the tensors are returned after rounding to the workload's dtype and
        widening back to fp64 (exactly the values a consumer of the rounded tensors sees).
        """
        c = self.cfg
        q = self._base_normal(layer, _TENSOR_Q, scale)
        k = self._base_normal(layer, _TENSOR_K, scale)
        v = self._base_normal(layer, _TENSOR_V, scale)
        ctx = self._mask[layer].to(self.device).bool()                            # [H]
        # contextual heads: every query and the sink keys get +4 u
        u = self._sink_direction(layer)                                           # [H, D]
        sinks = self.sink_positions(layer, scale)                                 # [H, N_k]
        add_q = (4.0 * u).view(1, c.n_heads, 1, c.head_dim) * ctx.view(1, -1, 1, 1)
        add_k = (4.0 * u).view(1, c.n_heads, 1, c.head_dim) * (sinks & ctx.view(-1, 1)).view(
            1, c.n_heads, -1, 1)
        # structural heads: +3 p on both sides
        p = (3.0 * self._position_code(scale)).view(1, 1, -1, c.head_dim) * (~ctx).view(1, -1, 1, 1)
        q = q + add_q + p
        k = k + add_k + p
        tdt = torch.float32 if c.dtype == "f32" else torch.bfloat16
        out = tuple(t.to(tdt).contiguous() for t in (q, k, v))
        if as_float64:
            out = tuple(t.to(torch.float64) for t in out)
        return out


# Layer count of the named workloads (the global head permutation is drawn over the full stack).
_FULL_LAYERS = {0: 1, 1: 16, 2: 30, 3: 32, 4: 40}


def random_observation_rows(cfg: WorkloadConfig, seed: int = 0) -> list:
    """Per scale, min(N_obs, N_k) distinct query rows drawn without replacement (the random-sampling
    arm of the query-subset ablation).  The draw is an input of the method, so it is made here, once,
    and handed to both the CPU oracle and the GPU library."""
    import numpy as np
    rng = np.random.default_rng(cfg.seed * 1000003 + seed)
    rows = []
    for side in cfg.sides:
        n_k = side * side
        n = min(cfg.n_obs, n_k)
        rows.append([int(r) for r in rng.choice(n_k, size=n, replace=False)])
    return rows
