"""ctypes binding of libfcsim.so: the C-ABI entry points under their own names.

Argument marshalling only -- every step of the simulation runs in the CUDA library.  PyTorch
provides device memory (the caller-owned buffers) and streams.  There is no CPU fallback: if the
library cannot be loaded the import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional

import numpy as np

from . import build as _build

FCSIM_OK = 0
COUNTER_NAMES = (
    "steps_done", "status", "arrived", "dropped", "admitted", "completed", "evictions",
    "overflow_steps", "gate_blocked_steps", "budget_blocked_steps", "acap_blocked_steps",
    "tokens_generated", "prefill_tokens", "completed_tokens", "wasted_tokens", "sum_lat", "max_lat",
    "sum_U", "max_U", "sum_N", "max_Q", "sum_w_completed", "n_logged", "q_final", "p_final",
    "resid_age", "resid_j", "mmpp_state")
N_COUNTERS = len(COUNTER_NAMES)
SUMMARY_FLOATS = ("mean_latency", "p95_latency", "p99_latency", "mean_utilisation", "request_throughput",
                  "token_throughput")


class fcsim_table(C.Structure):
    _fields_ = [("n", C.c_uint32), ("vmin", C.c_int32), ("cdf", C.POINTER(C.c_uint32))]


class fcsim_arrivals(C.Structure):
    _fields_ = [("n_states", C.c_uint32), ("count", fcsim_table * 2), ("switch_thr", C.c_uint32 * 2)]


class fcsim_group(C.Structure):
    _fields_ = [("policy", C.c_int32), ("b_fp", C.c_uint32), ("chunk", C.c_int32),
                ("arrivals_id", C.c_int32), ("rng_replica_base", C.c_uint32), ("n_replicas", C.c_int32),
                ("m_admit", C.c_int32), ("b_class", C.POINTER(C.c_int32)), ("mc_worst_case", C.c_int32),
                ("preempt_keep", C.c_int32)]


class fcsim_config(C.Structure):
    _fields_ = [("M", C.c_int32), ("K", C.c_int32), ("T_max", C.c_int32), ("Qcap", C.c_int32),
                ("Acap", C.c_int32), ("seed", C.c_uint64), ("n_classes", C.c_int32),
                ("class_law", fcsim_table), ("prompt", C.POINTER(fcsim_table)),
                ("decode", C.POINTER(fcsim_table)), ("n_arrivals", C.c_int32),
                ("arrivals", C.POINTER(fcsim_arrivals)), ("n_groups", C.c_int32),
                ("groups", C.POINTER(fcsim_group)), ("trace_stride", C.c_int32), ("hist_bins", C.c_int32),
                ("hist_shift", C.c_int32), ("complog_cap", C.c_int32), ("trace_bulk", C.c_int32)]


class fcsim_counters(C.Structure):
    _fields_ = [(n, C.c_int64) for n in COUNTER_NAMES]


class fcsim_summary(C.Structure):
    _fields_ = ([("total", fcsim_counters)] + [(n, C.c_double) for n in SUMMARY_FLOATS]
                + [("percentile_source", C.c_int32), ("reserved", C.c_int32)])


PCT_NONE, PCT_HISTOGRAM, PCT_EXACT = 0, 1, 2


def _summary_dicts(summ):
    out = []
    for s in summ:
        d = {n: int(getattr(s.total, n)) for n in COUNTER_NAMES}
        d.update({n: float(getattr(s, n)) for n in SUMMARY_FLOATS})
        d["percentile_source"] = int(s.percentile_source)
        out.append(d)
    return out


class fcsim_buffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("workspace", "counters", "trace", "hist", "complog", "scratch")]


class fcsim_sizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("workspace", "counters", "trace", "hist", "complog", "scratch")]


class fcsim_launch_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("grid", "block", "warps_per_block", "blocks_per_sm", "sm_count",
                                          "smem_per_block", "smem_per_warp", "max_steps_per_launch")]


EXPORTS = ("fcsim_query_sizes", "fcsim_create", "fcsim_run", "fcsim_stats", "fcsim_destroy",
           "fcsim_steps_done", "fcsim_get_launch_info", "fcsim_last_cuda_error", "fcsim_last_cuda_error_name",
           "fcsim_strerror", "fcsim_simulate_host", "fcsim_debug_read", "fcsim_is_checked_build",
           "fcsim_stats_noalloc")

_lib = None


def load():
    """Load (building if needed) the CUDA library; raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    if os.environ.get("FCSIM_LIB"):           # explicit library path (diagnostic builds)
        path = os.environ["FCSIM_LIB"]
    elif os.environ.get("FCSIM_CHECKED"):     # index-checked diagnostic build
        path = _build.build(checked=True)      # compiled if missing or older than the sources
    else:
        path = _build.LIB
        if not os.path.exists(path) or os.environ.get("FCSIM_REBUILD"):
            path = _build.build()
    lib = C.CDLL(path)
    vp = C.c_void_p
    lib.fcsim_query_sizes.argtypes = [C.POINTER(fcsim_config), C.POINTER(fcsim_sizes)]
    lib.fcsim_create.argtypes = [C.POINTER(fcsim_config), C.POINTER(fcsim_buffers), C.POINTER(vp)]
    lib.fcsim_run.argtypes = [vp, C.c_int32, vp]
    lib.fcsim_stats.argtypes = [vp, vp, C.POINTER(fcsim_counters), C.POINTER(fcsim_summary)]
    lib.fcsim_destroy.argtypes = [vp]
    lib.fcsim_steps_done.argtypes = [vp]
    lib.fcsim_steps_done.restype = C.c_int32
    lib.fcsim_get_launch_info.argtypes = [vp, C.POINTER(fcsim_launch_info)]
    lib.fcsim_last_cuda_error.argtypes = [vp]
    lib.fcsim_strerror.argtypes = [C.c_int]
    lib.fcsim_strerror.restype = C.c_char_p
    lib.fcsim_simulate_host.argtypes = [C.POINTER(fcsim_config), C.c_int32, C.POINTER(fcsim_counters), vp, vp, vp,
                                        C.POINTER(fcsim_summary)]
    lib.fcsim_last_cuda_error_name.argtypes = [vp]
    lib.fcsim_last_cuda_error_name.restype = C.c_char_p
    lib.fcsim_debug_read.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.fcsim_is_checked_build.argtypes = []
    lib.fcsim_stats_noalloc.argtypes = [vp, vp, C.POINTER(fcsim_summary)]
    for name in EXPORTS:
        if name not in ("fcsim_strerror", "fcsim_steps_done", "fcsim_last_cuda_error_name"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


class FcsimError(RuntimeError):
    def __init__(self, code, where, handle=None):
        self.code = int(code)
        msg = load().fcsim_strerror(int(code)).decode()
        if handle and code == -5:
            msg += " [%s]" % load().fcsim_last_cuda_error_name(C.c_void_p(handle)).decode()
        super().__init__(f"{where}: {msg} (code {code})")


def _check(code, where, handle=None):
    if code != FCSIM_OK:
        raise FcsimError(code, where, handle)


# ----------------------------------------------------------------------------- marshalling
def _mk_table(tab, keep):
    arr = np.ascontiguousarray(tab.cdf, dtype=np.uint32)
    keep.append(arr)
    return fcsim_table(arr.shape[0], int(tab.vmin), arr.ctypes.data_as(C.POINTER(C.c_uint32)))


def marshal_config(cfg):
    """workloads.SimConfig -> (fcsim_config, keepalive)."""
    keep = []
    prompt = (fcsim_table * len(cfg.prompt))(*[_mk_table(t, keep) for t in cfg.prompt])
    decode = (fcsim_table * len(cfg.decode))(*[_mk_table(t, keep) for t in cfg.decode])
    arrs = (fcsim_arrivals * max(1, len(cfg.arrivals)))()
    for i, a in enumerate(cfg.arrivals):
        arrs[i].n_states = len(a.count)
        for s, t in enumerate(a.count[:2]):
            arrs[i].count[s] = _mk_table(t, keep)
        arrs[i].switch_thr[0] = int(a.switch_thr[0])
        arrs[i].switch_thr[1] = int(a.switch_thr[1])
    groups = (fcsim_group * max(1, len(cfg.groups)))()
    for i, g in enumerate(cfg.groups):
        bc = getattr(g, "b_class", ())
        bptr = None
        if len(bc):
            arr = np.ascontiguousarray(bc, dtype=np.int32)
            keep.append(arr)
            bptr = arr.ctypes.data_as(C.POINTER(C.c_int32))
        groups[i] = fcsim_group(int(g.policy), int(g.b_fp), int(g.chunk), int(g.arrivals_id),
                                int(g.rng_replica_base), int(g.n_replicas), int(getattr(g, "m_admit", 0)), bptr,
                                int(getattr(g, "mc_worst_case", 0)),
                                int(getattr(g, "preempt_keep", 0)))
    c = fcsim_config(int(cfg.M), int(cfg.K), int(cfg.T_max), int(cfg.Qcap), int(cfg.Acap), int(cfg.seed),
                     len(cfg.prompt), _mk_table(cfg.class_law, keep), prompt, decode, len(cfg.arrivals), arrs,
                     len(cfg.groups), groups, int(cfg.trace_stride), int(cfg.hist_bins), int(cfg.hist_shift),
                     int(cfg.complog_cap), int(getattr(cfg, "trace_bulk", 0)))
    keep += [prompt, decode, arrs, groups]
    return c, keep


def _stream_ptr(stream):
    if stream is None:
        return None
    if isinstance(stream, int):
        return C.c_void_p(stream)
    return C.c_void_p(stream.cuda_stream)   # torch.cuda.Stream


# ----------------------------------------------------------------------------- the entry points
def fcsim_query_sizes(cfg) -> dict:
    c, keep = marshal_config(cfg)
    sz = fcsim_sizes()
    _check(load().fcsim_query_sizes(C.byref(c), C.byref(sz)), "fcsim_query_sizes")
    return {n: int(getattr(sz, n)) for n, _ in fcsim_sizes._fields_}


def fcsim_create(cfg, buffers: dict) -> int:
    """``buffers``: name -> torch CUDA tensor (or raw device address, or None). Returns the handle."""
    c, keep = marshal_config(cfg)
    b = fcsim_buffers()
    for n, _ in fcsim_buffers._fields_:
        v = buffers.get(n)
        setattr(b, n, None if v is None else (v if isinstance(v, int) else v.data_ptr()))
    h = C.c_void_p()
    _check(load().fcsim_create(C.byref(c), C.byref(b), C.byref(h)), "fcsim_create")
    return h.value


def fcsim_run(handle: int, n_steps: int, stream=None) -> None:
    _check(load().fcsim_run(C.c_void_p(handle), int(n_steps), _stream_ptr(stream)), "fcsim_run", handle)


def fcsim_stats(handle: int, n_replicas: int, n_groups: int, stream=None, want_counters=True, want_summary=True):
    """Returns (counters [R, 28] int64 numpy or None, list of per-group summary dicts or None)."""
    cnt = np.zeros((n_replicas, N_COUNTERS), dtype=np.int64) if want_counters else None
    summ = (fcsim_summary * n_groups)() if want_summary else None
    _check(load().fcsim_stats(C.c_void_p(handle), _stream_ptr(stream),
                              cnt.ctypes.data_as(C.POINTER(fcsim_counters)) if want_counters else None,
                              summ), "fcsim_stats", handle)
    return cnt, (_summary_dicts(summ) if want_summary else None)


def fcsim_stats_noalloc(handle: int, n_groups: int, stream=None):
    """Per-group summaries without any allocation by the library: for processes that cannot get device
    memory any more (their allocator owns the GPU) or must not pay an allocation's device-wide stall.
    The group rows use a fixed 1 MiB array inside the library, shared by all calls: do not overlap calls."""
    summ = (fcsim_summary * n_groups)()
    _check(load().fcsim_stats_noalloc(C.c_void_p(handle), _stream_ptr(stream), summ), "fcsim_stats_noalloc", handle)
    return _summary_dicts(summ)


def fcsim_destroy(handle: int) -> None:
    _check(load().fcsim_destroy(C.c_void_p(handle)), "fcsim_destroy")


def fcsim_steps_done(handle: int) -> int:
    return int(load().fcsim_steps_done(C.c_void_p(handle)))


def fcsim_get_launch_info(handle: int) -> dict:
    info = fcsim_launch_info()
    _check(load().fcsim_get_launch_info(C.c_void_p(handle), C.byref(info)), "fcsim_get_launch_info")
    return {n: int(getattr(info, n)) for n, _ in fcsim_launch_info._fields_}


def fcsim_last_cuda_error(handle: int) -> int:
    return int(load().fcsim_last_cuda_error(C.c_void_p(handle)))


def fcsim_debug_read(handle: int) -> List[int]:
    out = (C.c_uint32 * 8)()
    _check(load().fcsim_debug_read(C.c_void_p(handle), out), "fcsim_debug_read", handle)
    return [int(x) for x in out]


def fcsim_is_checked_build() -> bool:
    return bool(load().fcsim_is_checked_build())


def fcsim_strerror(code: int) -> str:
    return load().fcsim_strerror(int(code)).decode()


def host_output_arrays(cfg, trace=True, hist=True, complog=True, pinned=False) -> dict:
    """Host arrays shaped for fcsim_simulate_host; ``pinned`` takes page-locked memory from torch."""
    R = cfg.n_replicas
    n_rec = cfg.T_max // cfg.trace_stride if cfg.trace_stride > 0 else 0

    def alloc(shape, dtype):
        if not pinned:
            return np.zeros(shape, dtype=dtype)
        import torch
        tdt = {np.int32: torch.int32, np.int64: torch.int64}[dtype]
        return torch.zeros(shape, dtype=tdt, pin_memory=True).numpy()
    return {"counters": alloc((R, N_COUNTERS), np.int64),
            "trace": alloc((R, n_rec, 2), np.int32) if (trace and n_rec) else None,
            "hist": alloc((R, cfg.hist_bins), np.int32) if (hist and cfg.hist_bins) else None,
            "complog": alloc((R, cfg.complog_cap, 2), np.int32) if (complog and cfg.complog_cap) else None}


def fcsim_simulate_host(cfg, n_steps: Optional[int] = None, trace=True, hist=True, complog=True,
                        out: Optional[dict] = None) -> dict:
    """Whole job with host (numpy) outputs; device memory is managed inside the library.
    ``out``: arrays from host_output_arrays to fill (allocated here when None)."""
    c, keep = marshal_config(cfg)
    n_steps = cfg.T_max if n_steps is None else int(n_steps)
    G = len(cfg.groups)
    if out is None:
        out = host_output_arrays(cfg, trace, hist, complog)
    summ = (fcsim_summary * G)()

    def ptr(a):
        return None if a is None else C.c_void_p(a.ctypes.data)
    _check(load().fcsim_simulate_host(C.byref(c), n_steps, out["counters"].ctypes.data_as(C.POINTER(fcsim_counters)),
                                      ptr(out["trace"]), ptr(out["hist"]), ptr(out["complog"]), summ),
           "fcsim_simulate_host")
    out["summary"] = _summary_dicts(summ)
    return out


# ----------------------------------------------------------------------------- convenience owner of the buffers
class Simulation:
    """Allocates the caller-owned device buffers with torch and drives the entry points."""

    def __init__(self, cfg, device="cuda:0"):
        import torch
        self.torch = torch
        self.cfg = cfg
        self.device = torch.device(device)
        self.sizes = fcsim_query_sizes(cfg)
        with torch.cuda.device(self.device):
            self.buffers = {n: (torch.empty(max(b, 16), dtype=torch.uint8, device=self.device) if b > 0 else None)
                            for n, b in self.sizes.items()}
            self.handle = fcsim_create(cfg, self.buffers)
        self.R = cfg.n_replicas
        self.G = len(cfg.groups)

    def run(self, n_steps, stream=None):
        with self.torch.cuda.device(self.device):
            fcsim_run(self.handle, n_steps, stream)

    def stats(self, stream=None, want_counters=True, want_summary=True):
        with self.torch.cuda.device(self.device):
            return fcsim_stats(self.handle, self.R, self.G, stream, want_counters, want_summary)

    @property
    def steps_done(self):
        return fcsim_steps_done(self.handle)

    def launch_info(self):
        return fcsim_get_launch_info(self.handle)

    def _view(self, name, dtype, shape):
        buf = self.buffers[name]
        if buf is None:
            return None
        n = int(np.prod(shape)) * np.dtype(dtype).itemsize
        tdt = {np.int32: self.torch.int32, np.int64: self.torch.int64}[dtype]
        return buf[:n].view(tdt).view(*shape)

    def counters(self):
        return self._view("counters", np.int64, (self.R, N_COUNTERS))

    def trace(self):
        n_rec = self.cfg.T_max // self.cfg.trace_stride if self.cfg.trace_stride > 0 else 0
        return self._view("trace", np.int32, (self.R, n_rec, 2)) if n_rec else None

    def hist(self):
        return self._view("hist", np.int32, (self.R, self.cfg.hist_bins)) if self.cfg.hist_bins else None

    def complog(self):
        return (self._view("complog", np.int32, (self.R, self.cfg.complog_cap, 2))
                if self.cfg.complog_cap else None)

    def close(self):
        if self.handle:
            fcsim_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
