"""ctypes binding of libhack_b200.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/hack.h).  Tensors are passed
as raw device pointers; torch is used by callers for device memory and streams, never here for
arithmetic.  There is no fallback: if the shared library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

# HACK_B200_CHECKED=1 selects the checked build of the same sources (bounds checks in the kernels,
# guard rows in the planes); HackCache.close() then also verifies the guard rows.
_CHECKED = os.environ.get("HACK_B200_CHECKED", "0") == "1"
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib",
                         "libhack_b200_checked.so" if _CHECKED else "libhack_b200.so")

HACK_OK, HACK_ERR_INVALID_ARG, HACK_ERR_UNSUPPORTED, HACK_ERR_OOM, HACK_ERR_CUDA, HACK_ERR_STATE, \
    HACK_ERR_TIMEOUT = range(7)
HACK_F32, HACK_BF16 = 0, 1
HACK_OVERFLOW_KEEP_PROTECTED, HACK_OVERFLOW_COMPETE = 0, 1
HACK_OBS_UNIFORM, HACK_OBS_INIT, HACK_OBS_RECENT, HACK_OBS_CALLER, HACK_OBS_FULL = 0, 1, 2, 3, 4
RULE_FRACTION, RULE_RATIO = 0, 1

EXPORTS = (
    "hack_split_budget", "hack_init_cache", "hack_free_cache", "hack_reset", "hack_set_obs_rows", "hack_get_limits",
    "hack_step_info", "hack_score", "hack_select", "hack_compact", "hack_attend", "hack_attend_variance",
    "hack_classify_heads", "hack_scale_step",
    "hack_scale_step_host", "hack_score_noalloc", "hack_get_lengths", "hack_read_head", "hack_kv_bytes",
    "hack_launch_count", "hack_stage_timing", "hack_stage_times", "hack_poll_status", "hack_set_wait_limit",
    "hack_debug_build", "hack_debug_check", "hack_last_error",
)


class HackConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("batch", C.c_int32),
        ("n_scales", C.c_int32), ("scale_sides", C.POINTER(C.c_int32)), ("dtype", C.c_int32),
        ("head_is_contextual", C.POINTER(C.c_uint8)), ("budget_c", C.c_int32), ("budget_s", C.c_int32),
        ("n_obs", C.c_int32), ("n_init_scales", C.c_int32), ("sm_scale", C.c_float),
        ("overflow_policy", C.c_int32), ("device", C.c_int32), ("obs_sampler", C.c_int32),
        ("merge_last", C.c_int32),
    ]


class HackStepInfo(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_new", "stored_c", "stored_s", "cand_c", "cand_s", "kept_c", "kept_s",
        "triggered_c", "triggered_s", "n_obs_rows")]


class HackLimits(C.Structure):
    _fields_ = [("cand_stride", C.c_int32), ("kept_stride", C.c_int32), ("max_new", C.c_int32)]


class HackError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"hack status {status}: {text}")
        self.status = status


def _load() -> C.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python paper_2504_09261_b200/build.py` "
            "(there is no fallback implementation)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32 = C.c_void_p, C.c_int32
    lib.hack_last_error.restype = C.c_char_p
    lib.hack_last_error.argtypes = []
    sigs = {
        "hack_split_budget": [i32, C.c_double, i32, C.c_double, i32, C.POINTER(i32), C.POINTER(i32)],
        "hack_init_cache": [C.POINTER(HackConfig), C.POINTER(vp)],
        "hack_free_cache": [vp],
        "hack_reset": [vp],
        "hack_set_obs_rows": [vp, i32, C.POINTER(i32), i32],
        "hack_get_limits": [vp, C.POINTER(HackLimits)],
        "hack_step_info": [vp, i32, i32, C.POINTER(HackStepInfo)],
        "hack_score": [vp, i32, i32, vp, vp, vp, vp],
        "hack_select": [vp, i32, i32, vp, vp, vp, vp],
        "hack_compact": [vp, i32, i32, vp, vp, vp, vp],
        "hack_attend": [vp, i32, i32, vp, vp, vp],
        "hack_attend_variance": [vp, i32, i32, vp, vp, vp, vp],
        "hack_classify_heads": [C.POINTER(C.c_double), i32, i32, C.c_double, C.POINTER(C.c_uint8)],
        "hack_scale_step": [vp, i32, i32, vp, vp, vp, vp, vp],
        "hack_scale_step_host": [vp, i32, i32, vp, vp, vp, vp, vp],
        "hack_score_noalloc": [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, C.c_float, vp],
        "hack_get_lengths": [vp, i32, C.POINTER(i32)],
        "hack_read_head": [vp, i32, i32, i32, i32, vp, C.c_size_t],
        "hack_kv_bytes": [vp, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)],
        "hack_launch_count": [vp, C.POINTER(C.c_uint64)],
        "hack_poll_status": [vp, vp],
        "hack_set_wait_limit": [vp, C.c_int64],
        "hack_debug_check": [vp, C.POINTER(i32)],
        "hack_stage_timing": [vp, i32],
        "hack_stage_times": [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint64)],
    }
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.hack_debug_build.argtypes = []
    lib.hack_debug_build.restype = C.c_int32
    return lib


lib = _load()


def hack_last_error() -> str:
    return lib.hack_last_error().decode()


def _check(status: int) -> None:
    if status != HACK_OK:
        raise HackError(status, hack_last_error())


def hack_split_budget(budget: int, alpha: float, rule: int, param: float, total_tokens: int):
    bc, bs = C.c_int32(), C.c_int32()
    _check(lib.hack_split_budget(budget, alpha, rule, param, total_tokens, C.byref(bc), C.byref(bs)))
    return bc.value, bs.value


def hack_classify_heads(sigma, n_layers: int, n_heads: int, alpha: float):
    """Head mask (list of n_layers lists of 0/1, 1 = contextual) from the variance matrix."""
    flat = [float(v) for row in sigma for v in (row if hasattr(row, "__iter__") else [row])]
    if len(flat) != n_layers * n_heads:
        raise ValueError("sigma must have n_layers*n_heads entries")
    arr = (C.c_double * len(flat))(*flat)
    out = (C.c_uint8 * len(flat))()
    _check(lib.hack_classify_heads(arr, n_layers, n_heads, alpha, out))
    return [[int(out[l * n_heads + h]) for h in range(n_heads)] for l in range(n_layers)]


def hack_score_noalloc(q, k_cand, scores, n_rows: int, n_queries: int, n_cand: int, score_stride: int,
                       head_dim: int, dtype: int, n_obs: int = 32, sm_scale: float = 0.0, stream=None):
    """Scores on dense device tensors with no device allocation (fixed in-library scratch)."""
    _check(lib.hack_score_noalloc(_ptr(q), _ptr(k_cand), _ptr(scores), n_rows, n_queries, n_cand,
                                  score_stride, head_dim, dtype, n_obs, sm_scale, _ptr(stream)))


def _ptr(x) -> Optional[int]:
    """Raw address of a torch tensor / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


class HackCache:
    """Owner of one hack_cache_t.  Methods mirror the C entry points of the same name."""

    def __init__(self, n_layers: int, n_heads: int, head_dim: int, batch: int, sides: Sequence[int],
                 dtype: int, head_is_contextual, budget_c: int, budget_s: int, n_obs: int = 32,
                 n_init_scales: int = 2, sm_scale: float = 0.0,
                 overflow_policy: int = HACK_OVERFLOW_KEEP_PROTECTED, device: int = 0,
                 obs_sampler: int = HACK_OBS_UNIFORM, merge_last: bool = False):
        self._h = C.c_void_p()
        sides_arr = (C.c_int32 * len(sides))(*[int(s) for s in sides])
        flat = [int(v) for v in (head_is_contextual.reshape(-1).tolist()
                                 if hasattr(head_is_contextual, "reshape") else head_is_contextual)]
        mask_arr = (C.c_uint8 * len(flat))(*flat)
        if len(flat) != n_layers * n_heads:
            raise ValueError("head_is_contextual must have n_layers*n_heads entries")
        cfg = HackConfig(n_layers, n_heads, head_dim, batch, len(sides), sides_arr, dtype, mask_arr,
                         budget_c, budget_s, n_obs, n_init_scales, sm_scale, overflow_policy, device,
                         obs_sampler, 1 if merge_last else 0)
        _check(lib.hack_init_cache(C.byref(cfg), C.byref(self._h)))
        self.n_layers, self.n_heads, self.head_dim, self.batch = n_layers, n_heads, head_dim, batch
        self.dtype = dtype
        self.elt = 4 if dtype == HACK_F32 else 2
        lim = HackLimits()
        _check(lib.hack_get_limits(self._h, C.byref(lim)))
        self.cand_stride, self.kept_stride, self.max_new = lim.cand_stride, lim.kept_stride, lim.max_new

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            problem = None
            if lib.hack_debug_build():
                # checked build: no kernel may have tripped a bounds check or touched a guard row
                if lib.hack_poll_status(self._h, None) != HACK_OK:
                    problem = hack_last_error()
                bad = C.c_int32()
                if lib.hack_debug_check(self._h, C.byref(bad)) == HACK_OK and bad.value and problem is None:
                    problem = f"{bad.value} guard rows overwritten: {hack_last_error()}"
            lib.hack_free_cache(self._h)
            self._h = C.c_void_p()
            if problem:
                raise HackError(HACK_ERR_STATE, problem)

    def hack_debug_check(self) -> int:
        bad = C.c_int32()
        _check(lib.hack_debug_check(self._h, C.byref(bad)))
        return bad.value

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def hack_set_obs_rows(self, scale: int, rows: Sequence[int]) -> None:
        arr = (C.c_int32 * len(rows))(*[int(r) for r in rows])
        _check(lib.hack_set_obs_rows(self._h, scale, arr, len(rows)))

    def hack_reset(self) -> None:
        _check(lib.hack_reset(self._h))

    def hack_step_info(self, layer: int, scale: int) -> HackStepInfo:
        info = HackStepInfo()
        _check(lib.hack_step_info(self._h, layer, scale, C.byref(info)))
        return info

    def hack_score(self, layer, scale, q, k_new, scores, stream=None) -> None:
        _check(lib.hack_score(self._h, layer, scale, _ptr(q), _ptr(k_new), _ptr(scores), _ptr(stream)))

    def hack_select(self, layer, scale, scores, idx, kept_out=None, stream=None) -> None:
        _check(lib.hack_select(self._h, layer, scale, _ptr(scores), _ptr(idx), _ptr(kept_out), _ptr(stream)))

    def hack_compact(self, layer, scale, idx, k_new, v_new, stream=None) -> None:
        _check(lib.hack_compact(self._h, layer, scale, _ptr(idx), _ptr(k_new), _ptr(v_new), _ptr(stream)))

    def hack_attend(self, layer, scale, q, out, stream=None) -> None:
        _check(lib.hack_attend(self._h, layer, scale, _ptr(q), _ptr(out), _ptr(stream)))

    def hack_attend_variance(self, layer, scale, q, out, sigma, stream=None) -> None:
        _check(lib.hack_attend_variance(self._h, layer, scale, _ptr(q), _ptr(out), _ptr(sigma), _ptr(stream)))

    def hack_scale_step(self, layer, scale, q, k, v, out, stream=None) -> None:
        _check(lib.hack_scale_step(self._h, layer, scale, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(stream)))

    def hack_scale_step_host(self, layer, scale, q, k, v, out, stream=None) -> None:
        _check(lib.hack_scale_step_host(self._h, layer, scale, _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                        _ptr(stream)))

    def hack_get_lengths(self, layer: int):
        n = self.batch * self.n_heads
        arr = (C.c_int32 * n)()
        _check(lib.hack_get_lengths(self._h, layer, arr))
        return list(arr)

    def hack_read_head(self, layer: int, b: int, h: int, which: int) -> bytes:
        length = self.hack_get_lengths(layer)[b * self.n_heads + h]
        nbytes = length * (4 if which == 2 else self.head_dim * self.elt)
        buf = C.create_string_buffer(max(nbytes, 1))
        _check(lib.hack_read_head(self._h, layer, b, h, which, buf, nbytes))
        return buf.raw[:nbytes]

    def hack_kv_bytes(self):
        live, peak, res = C.c_size_t(), C.c_size_t(), C.c_size_t()
        _check(lib.hack_kv_bytes(self._h, C.byref(live), C.byref(peak), C.byref(res)))
        return live.value, peak.value, res.value

    def hack_launch_count(self) -> int:
        n = C.c_uint64()
        _check(lib.hack_launch_count(self._h, C.byref(n)))
        return n.value

    def hack_stage_timing(self, enable: bool) -> None:
        _check(lib.hack_stage_timing(self._h, 1 if enable else 0))

    def hack_stage_times(self):
        ms = (C.c_double * 4)()
        n = (C.c_uint64 * 4)()
        _check(lib.hack_stage_times(self._h, ms, n))
        names = ("score", "select", "compact", "attend")
        return {k: (ms[i], n[i]) for i, k in enumerate(names)}

    def hack_set_wait_limit(self, cycles: int) -> None:
        _check(lib.hack_set_wait_limit(self._h, cycles))

    def hack_poll_status(self, stream=None) -> None:
        _check(lib.hack_poll_status(self._h, _ptr(stream)))
