"""ctypes binding of liblazyev.so: the same names as the C ABI, argument
marshalling only.  `Engine` bundles a handle with the torch tensors that own
its device memory; every step of the method runs inside the library's kernels.

There is no fallback: if the shared library is missing and cannot be built, or
no CUDA device is present when one is needed, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

from . import build as _build

OK, EINVAL, ESTATE, ECAPACITY, EDEVICE, ECUDA = 0, -1, -2, -3, -4, -5
SCORE_H1_PLUS_H2, SCORE_H1_ONLY, SCORE_H2_ONLY, SCORE_H1_PLUS_H2_DECREASING = 0, 1, 2, 3
PROMPT_TILED, PROMPT_REPLAY = 0, 1


class Info(C.Structure):
    _fields_ = [(n, C.c_int) for n in (
        "layers", "batch", "q_heads", "kv_heads", "head_dim", "units", "budget", "budget_now", "window",
        "n_recent", "n_initial", "capacity", "pages_per_unit", "t", "n", "prefill", "splits", "stages",
        "groups", "tail_units", "tail_splits", "grid", "smem_bytes")] + [("launches", C.c_longlong), ("evictions", C.c_longlong),
                                                                           ("host_ranges", C.c_int)]


class Counters(C.Structure):
    _fields_ = [("device_status", C.c_int), ("select_radix_units", C.c_int), ("select_zero_cut_units", C.c_int)]


class Profile(C.Structure):
    _fields_ = [(n, C.c_double) for n in (
        "append_ms", "decode_ms", "select_ms", "compact_ms", "decode_bytes", "select_bytes", "compact_bytes",
        "compact_rows")] + [(n, C.c_longlong) for n in (
            "append_launches", "decode_launches", "select_launches", "compact_launches")]


class Dump(C.Structure):
    _fields_ = [("unit_begin", C.c_int), ("unit_count", C.c_int), ("t", C.c_int), ("n", C.c_int),
                ("capacity", C.c_int), ("device_status", C.c_int),
                ("pos", C.c_void_p), ("ts", C.c_void_p), ("mri", C.c_void_p), ("pbar", C.c_void_p),
                ("score", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p)]


_PROTOS = {
    "lazyev_create": [C.POINTER(C.c_void_p), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float],
    "lazyev_set_batch": [C.c_void_p, C.c_int],
    "lazyev_set_protect": [C.c_void_p, C.c_int, C.c_int],
    "lazyev_set_max_prefill": [C.c_void_p, C.c_int],
    "lazyev_set_budget": [C.c_void_p, C.c_int],
    "lazyev_set_auto_evict": [C.c_void_p, C.c_int],
    "lazyev_set_score_mode": [C.c_void_p, C.c_int],
    "lazyev_set_splits": [C.c_void_p, C.c_int],
    "lazyev_set_stages": [C.c_void_p, C.c_int],
    "lazyev_set_groups": [C.c_void_p, C.c_int],
    "lazyev_set_fused_append": [C.c_void_p, C.c_int],
    "lazyev_query_sizes": [C.c_void_p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)],
    "lazyev_bind": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "lazyev_set_page_table": [C.c_void_p, C.c_void_p],
    "lazyev_prefill": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int],
    "lazyev_reset": [C.c_void_p],
    "lazyev_prefill_observed": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p],
    "lazyev_set_prompt_mode": [C.c_void_p, C.c_int],
    "lazyev_set_prompt_dump": [C.c_void_p, C.c_void_p, C.c_int, C.c_int],
    "lazyev_set_wait_limit": [C.c_void_p, C.c_double],
    "lazyev_debug_starve_page_ring": [C.c_void_p, C.c_int],
    "lazyev_decode_step": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "lazyev_decode_step_host": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "lazyev_decode_step_host_async": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
    "lazyev_host_wait": [C.c_void_p, C.c_int],
    "lazyev_copy_state": [C.c_void_p, C.c_void_p],
    "lazyev_evict": [C.c_void_p, C.POINTER(C.c_int)],
    "lazyev_evict_static": [C.c_void_p, C.POINTER(C.c_int)],
    "lazyev_get_info": [C.c_void_p, C.POINTER(Info)],
    "lazyev_get_counters": [C.c_void_p, C.POINTER(Counters)],
    "lazyev_dump_state": [C.c_void_p, C.POINTER(Dump)],
    "lazyev_load_state": [C.c_void_p, C.POINTER(Dump), C.c_int],
    "lazyev_mri_histogram": [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int],
    "lazyev_mri_quantile": [C.c_void_p, C.c_int, C.c_int, C.c_double, C.POINTER(C.c_int), C.POINTER(C.c_longlong)],
    "lazyev_set_profiling": [C.c_void_p, C.c_int],
    "lazyev_get_profile": [C.c_void_p, C.POINTER(Profile), C.c_int],
    "lazyev_synchronize": [C.c_void_p],
    "lazyev_destroy": [C.c_void_p],
}

_lib = None


def debug_bounds_requested() -> bool:
    """LAZYEV_DEBUG_BOUNDS=1 in the environment selects the range-checked build of the library."""
    return os.environ.get("LAZYEV_DEBUG_BOUNDS", "0") == "1"


def lib() -> C.CDLL:
    """Load (building first if the sources are newer) the shared library."""
    global _lib
    if _lib is None:
        path = _build.build(debug_bounds=debug_bounds_requested())
        _lib = C.CDLL(path)
        _lib.lazyev_build_flags.argtypes, _lib.lazyev_build_flags.restype = [], C.c_int
        if bool(_lib.lazyev_build_flags() & 1) != debug_bounds_requested():
            raise RuntimeError(f"{path} is not the build flavour that was asked for")
        for name, args in _PROTOS.items():
            fn = getattr(_lib, name)
            fn.argtypes, fn.restype = args, C.c_int
        _lib.lazyev_strerror.argtypes, _lib.lazyev_strerror.restype = [C.c_int], C.c_char_p
        _lib.lazyev_last_error.argtypes, _lib.lazyev_last_error.restype = [C.c_void_p], C.c_char_p
    return _lib


class LazyEvError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"lazyev error {code} ({lib().lazyev_strerror(code).decode()}): {message}")
        self.code = code


def _ptr(x) -> int:
    """Address of a torch tensor's or numpy array's first element."""
    if x is None:
        return 0
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.is_contiguous()
    return x.data_ptr()


class Engine:
    """A handle plus the device memory it is bound to (allocated through torch)."""

    def __init__(self, layers: int, q_heads: int, kv_heads: int, head_dim: int, budget: int, window: int,
                 threshold: float, batch: int = 1, n_recent: Optional[int] = None, n_initial: int = 0,
                 max_prefill: Optional[int] = None, device="cuda", stream=None):
        import torch
        self._torch = torch
        self._h = C.c_void_p()
        self._check(lib().lazyev_create(C.byref(self._h), layers, q_heads, kv_heads, head_dim, budget, window,
                                        threshold), create=True)
        self._check(lib().lazyev_set_batch(self._h, batch))
        if n_recent is not None or n_initial:
            self._check(lib().lazyev_set_protect(self._h, window if n_recent is None else n_recent, n_initial))
        if max_prefill is not None:
            self._check(lib().lazyev_set_max_prefill(self._h, max_prefill))
        kv, st, sc = C.c_size_t(), C.c_size_t(), C.c_size_t()
        self._check(lib().lazyev_query_sizes(self._h, C.byref(kv), C.byref(st), C.byref(sc)))
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.kv_pool = torch.empty(kv.value, dtype=torch.uint8, device=self.device)
            self.state = torch.empty(st.value, dtype=torch.uint8, device=self.device)
            self.scratch = torch.empty(sc.value, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self._check(lib().lazyev_bind(self._h, self.kv_pool.data_ptr(), self.state.data_ptr(),
                                          self.scratch.data_ptr(), self.stream.cuda_stream))

    # -- plumbing -----------------------------------------------------------------
    def _check(self, code: int, create: bool = False) -> None:
        if code != OK:
            msg = "" if create else lib().lazyev_last_error(self._h).decode()
            raise LazyEvError(code, msg)

    def close(self) -> None:
        if self._h:
            lib().lazyev_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, same names ------------------------------------------------------
    def set_budget(self, budget_now: int) -> None:
        self._check(lib().lazyev_set_budget(self._h, budget_now))

    def set_auto_evict(self, on: bool) -> None:
        self._check(lib().lazyev_set_auto_evict(self._h, int(on)))

    def set_score_mode(self, mode: int) -> None:
        self._check(lib().lazyev_set_score_mode(self._h, mode))

    def set_splits(self, splits: int) -> None:
        self._check(lib().lazyev_set_splits(self._h, splits))

    def set_stages(self, stages: int) -> None:
        self._check(lib().lazyev_set_stages(self._h, stages))

    def set_groups(self, groups: int) -> None:
        self._check(lib().lazyev_set_groups(self._h, groups))

    def set_fused_append(self, on: bool) -> None:
        self._check(lib().lazyev_set_fused_append(self._h, int(on)))

    def set_page_table(self, table) -> None:
        arr = np.ascontiguousarray(np.asarray(table, dtype=np.int32))
        self._check(lib().lazyev_set_page_table(self._h, arr.ctypes.data))

    def prefill(self, k, v) -> None:
        self._check(lib().lazyev_prefill(self._h, _ptr(k), _ptr(v), k.shape[-2]))

    def reset(self) -> None:
        self._check(lib().lazyev_reset(self._h))

    def set_prompt_mode(self, mode: int) -> None:
        self._check(lib().lazyev_set_prompt_mode(self._h, mode))

    def set_prompt_dump(self, rows, unit_begin: int = 0, unit_count: int = 0) -> None:
        """lazyev_set_prompt_dump: rows = float32 CUDA tensor [unit_count, P, P] or None."""
        self._check(lib().lazyev_set_prompt_dump(self._h, _ptr(rows), unit_begin, unit_count))

    def debug_starve_page_ring(self, pages: int) -> None:
        self._check(lib().lazyev_debug_starve_page_ring(self._h, pages))

    def set_wait_limit(self, seconds: float) -> None:
        self._check(lib().lazyev_set_wait_limit(self._h, seconds))

    def prefill_observed(self, q, k, v, out) -> None:
        """lazyev_prefill_observed: q, out [P, layers, batch, q_heads, D]; k, v as for prefill."""
        self._check(lib().lazyev_prefill_observed(self._h, _ptr(q), _ptr(k), _ptr(v), k.shape[-2], _ptr(out)))

    def decode_step(self, q, k_new, v_new, out) -> None:
        self._check(lib().lazyev_decode_step(self._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out)))

    def decode_step_host(self, q, k_new, v_new, out) -> None:
        self._check(lib().lazyev_decode_step_host(self._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out)))

    def decode_step_host_async(self, q, k_new, v_new, out) -> None:
        self._check(lib().lazyev_decode_step_host_async(self._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out)))

    def host_wait(self, in_flight_allowed: int = 0) -> None:
        self._check(lib().lazyev_host_wait(self._h, in_flight_allowed))

    def copy_state_from(self, src: "Engine") -> None:
        """lazyev_copy_state(self, src): this handle becomes a copy of src's cached sequences."""
        self._check(lib().lazyev_copy_state(self._h, src._h))

    def evict(self) -> int:
        n = C.c_int()
        self._check(lib().lazyev_evict(self._h, C.byref(n)))
        return n.value

    def evict_static(self) -> int:
        """lazyev_evict_static: the same eviction with its work lists in the library's built-in
        array instead of the bound scratch region (for callers that cannot allocate)."""
        n = C.c_int()
        self._check(lib().lazyev_evict_static(self._h, C.byref(n)))
        return n.value

    def load_state(self, snap: dict, prefill: int) -> None:
        """lazyev_load_state from a dict as returned by dump_state(kv=True) over all units."""
        cnt, n = snap["pos"].shape
        d = Dump(unit_begin=0, unit_count=cnt, t=snap["t"], n=n, capacity=n)
        keep = {}
        for name, dt in (("pos", np.int32), ("ts", np.int32), ("mri", np.int32), ("pbar", np.float32),
                         ("k", np.uint16), ("v", np.uint16)):
            if name in snap:
                keep[name] = np.ascontiguousarray(snap[name], dtype=dt)
                setattr(d, name, keep[name].ctypes.data)
        self._check(lib().lazyev_load_state(self._h, C.byref(d), prefill))

    def mri_histogram(self, bins: int, unit_begin: int = 0, unit_count: Optional[int] = None):
        """lazyev_mri_histogram: int64 counts per MRI value (last bin: everything larger)."""
        cnt = self.info().units - unit_begin if unit_count is None else unit_count
        hist = np.zeros(bins, dtype=np.int64)
        self._check(lib().lazyev_mri_histogram(self._h, unit_begin, cnt, hist.ctypes.data, bins))
        return hist

    def mri_quantile(self, fraction: float, unit_begin: int = 0, unit_count: Optional[int] = None):
        """lazyev_mri_quantile: (value, number of re-activated tokens)."""
        cnt = self.info().units - unit_begin if unit_count is None else unit_count
        value, total = C.c_int(), C.c_longlong()
        self._check(lib().lazyev_mri_quantile(self._h, unit_begin, cnt, fraction, C.byref(value), C.byref(total)))
        return value.value, total.value

    def synchronize(self) -> None:
        self._check(lib().lazyev_synchronize(self._h))

    def set_profiling(self, on: bool) -> None:
        self._check(lib().lazyev_set_profiling(self._h, int(on)))

    def get_profile(self, reset: bool = False) -> Profile:
        out = Profile()
        self._check(lib().lazyev_get_profile(self._h, C.byref(out), int(reset)))
        return out

    def counters(self) -> Counters:
        out = Counters()
        self._check(lib().lazyev_get_counters(self._h, C.byref(out)))
        return out

    def info(self) -> Info:
        out = Info()
        self._check(lib().lazyev_get_info(self._h, C.byref(out)))
        return out

    def dump_state(self, unit_begin: int = 0, unit_count: Optional[int] = None, kv: bool = False,
                   score: bool = False) -> dict:
        """Snapshot of units [unit_begin, unit_begin + unit_count) as numpy arrays
        trimmed to the n valid slots."""
        inf = self.info()
        cnt = inf.units - unit_begin if unit_count is None else unit_count
        cap = inf.capacity
        d = Dump(unit_begin=unit_begin, unit_count=cnt)
        arrs = {"pos": np.zeros((cnt, cap), np.int32), "ts": np.zeros((cnt, cap), np.int32),
                "mri": np.zeros((cnt, cap), np.int32), "pbar": np.zeros((cnt, cap), np.float32)}
        if score:
            arrs["score"] = np.zeros((cnt, cap), np.float64)
        if kv:
            arrs["k"] = np.zeros((cnt, cap, inf.head_dim), np.uint16)
            arrs["v"] = np.zeros((cnt, cap, inf.head_dim), np.uint16)
        for name, a in arrs.items():
            setattr(d, name, a.ctypes.data)
        self._check(lib().lazyev_dump_state(self._h, C.byref(d)))
        out = {name: a[:, : d.n] for name, a in arrs.items()}
        out.update(t=d.t, n=d.n, capacity=d.capacity, device_status=d.device_status)
        return out
