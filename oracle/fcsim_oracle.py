"""TEST INFRASTRUCTURE: ctypes front end of the CPU checker (fcsim_oracle.cpp).

Takes any simulation description with the attribute names of the workload module
(duck-typed; nothing from the CUDA path is imported) and returns numpy arrays.
Also derives the fp64 summaries of Section 2.2 (token throughput, prompt throughput,
mean and tail latency) and the mean KV utilisation from the int64 counters.
"""
from __future__ import annotations

import ctypes as C
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from . import build as _build

COUNTER_NAMES = (
    "steps_done", "status", "arrived", "dropped", "admitted", "completed", "evictions",
    "overflow_steps", "gate_blocked_steps", "budget_blocked_steps", "acap_blocked_steps",
    "tokens_generated", "prefill_tokens", "completed_tokens", "wasted_tokens", "sum_lat", "max_lat",
    "sum_U", "max_U", "sum_N", "max_Q", "sum_w_completed", "n_logged", "q_final", "p_final",
    "resid_age", "resid_j", "mmpp_state")
N_COUNTERS = len(COUNTER_NAMES)
CIDX = {n: i for i, n in enumerate(COUNTER_NAMES)}
# how a counter combines across the replicas of a group
MAX_FIELDS = ("max_lat", "max_U", "max_Q")
OR_FIELDS = ("status",)


class _Table(C.Structure):
    _fields_ = [("n", C.c_uint32), ("vmin", C.c_int32), ("cdf", C.POINTER(C.c_uint32))]


class _Arrivals(C.Structure):
    _fields_ = [("n_states", C.c_uint32), ("count", _Table * 2), ("switch_thr", C.c_uint32 * 2)]


class _Group(C.Structure):
    _fields_ = [("policy", C.c_int32), ("b_fp", C.c_uint32), ("chunk", C.c_int32),
                ("arrivals_id", C.c_int32), ("rng_replica_base", C.c_uint32), ("n_replicas", C.c_int32),
                ("m_admit", C.c_int32), ("b_class", C.POINTER(C.c_int32)), ("mc_worst_case", C.c_int32),
                ("preempt_keep", C.c_int32)]


class _Config(C.Structure):
    _fields_ = [("M", C.c_int32), ("K", C.c_int32), ("T_max", C.c_int32), ("Qcap", C.c_int32),
                ("Acap", C.c_int32), ("seed", C.c_uint64), ("n_classes", C.c_int32),
                ("class_law", _Table), ("prompt", C.POINTER(_Table)), ("decode", C.POINTER(_Table)),
                ("n_arrivals", C.c_int32), ("arrivals", C.POINTER(_Arrivals)),
                ("n_groups", C.c_int32), ("groups", C.POINTER(_Group)),
                ("trace_stride", C.c_int32), ("hist_bins", C.c_int32), ("hist_shift", C.c_int32),
                ("complog_cap", C.c_int32)]


class _Outputs(C.Structure):
    _fields_ = [("counters", C.POINTER(C.c_int64)), ("trace", C.POINTER(C.c_int32)),
                ("hist", C.POINTER(C.c_int32)), ("complog", C.POINTER(C.c_int32)),
                ("arrlog", C.POINTER(C.c_int32)), ("arrcls", C.POINTER(C.c_int32)),
                ("admlog", C.POINTER(C.c_int32)),
                ("admlog_cap", C.c_int64), ("n_admlog", C.POINTER(C.c_int64))]


_lib = None


def lib(sanitize: bool = False):
    global _lib
    if sanitize:
        return _bind(C.CDLL(_build.build(sanitize=True)))
    if _lib is None:
        _lib = _bind(C.CDLL(_build.build()))
    return _lib


def _bind(l):
    l.fcsim_oracle_run.restype = C.c_int
    l.fcsim_oracle_run.argtypes = [C.POINTER(_Config), C.c_int64, C.c_int64, C.c_int32, C.POINTER(_Outputs)]
    l.fcsim_oracle_run_ex.restype = C.c_int
    l.fcsim_oracle_run_ex.argtypes = [C.POINTER(_Config), C.c_int64, C.c_int64, C.c_int32, C.POINTER(_Outputs),
                                      C.c_int, C.POINTER(C.c_int64)]
    l.fcsim_oracle_philox.restype = None
    l.fcsim_oracle_philox.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
    l.fcsim_oracle_sample.restype = C.c_int32
    l.fcsim_oracle_sample.argtypes = [C.POINTER(_Table), C.c_uint32]
    return l


def _mk_table(tab, keep):
    arr = np.ascontiguousarray(tab.cdf, dtype=np.uint32)
    keep.append(arr)
    return _Table(arr.shape[0], int(tab.vmin), arr.ctypes.data_as(C.POINTER(C.c_uint32)))


def marshal(cfg):
    """Build the C description; returns (struct, keepalive list)."""
    keep = []
    prompt = (_Table * len(cfg.prompt))(*[_mk_table(t, keep) for t in cfg.prompt])
    decode = (_Table * len(cfg.decode))(*[_mk_table(t, keep) for t in cfg.decode])
    arrs = (_Arrivals * len(cfg.arrivals))()
    for i, a in enumerate(cfg.arrivals):
        arrs[i].n_states = len(a.count)
        for s, t in enumerate(a.count):
            arrs[i].count[s] = _mk_table(t, keep)
        arrs[i].switch_thr[0] = int(a.switch_thr[0])
        arrs[i].switch_thr[1] = int(a.switch_thr[1])
    groups = (_Group * len(cfg.groups))()
    for i, g in enumerate(cfg.groups):
        bc = getattr(g, "b_class", ())
        bptr = None
        if len(bc):
            arr = np.ascontiguousarray(bc, dtype=np.int32)
            keep.append(arr)
            bptr = arr.ctypes.data_as(C.POINTER(C.c_int32))
        groups[i] = _Group(int(g.policy), int(g.b_fp), int(g.chunk), int(g.arrivals_id),
                           int(g.rng_replica_base), int(g.n_replicas), int(getattr(g, "m_admit", 0)), bptr,
                           int(getattr(g, "mc_worst_case", 0)), int(getattr(g, "preempt_keep", 0)))
    c = _Config(int(cfg.M), int(cfg.K), int(cfg.T_max), int(cfg.Qcap), int(cfg.Acap), int(cfg.seed),
                len(cfg.prompt), _mk_table(cfg.class_law, keep), prompt, decode, len(cfg.arrivals), arrs,
                len(cfg.groups), groups, int(cfg.trace_stride), int(cfg.hist_bins), int(cfg.hist_shift),
                int(cfg.complog_cap))
    keep += [prompt, decode, arrs, groups]
    return c, keep


def philox(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().fcsim_oracle_philox(c, k, o)
    return tuple(int(x) for x in o)


def sample(tab, u):
    keep = []
    t = _mk_table(tab, keep)
    return int(lib().fcsim_oracle_sample(C.byref(t), int(u) & 0xFFFFFFFF))


def _p(arr, typ):
    return arr.ctypes.data_as(C.POINTER(typ)) if arr is not None else None


def _run_range(cfg, first, n, n_steps, trace, hist, complog, arrlog, admlog_cap, sanitize, arrcls=False,
               mc_mode=0):
    c, keep = marshal(cfg)
    out = {"counters": np.zeros((n, N_COUNTERS), dtype=np.int64)}
    n_rec = n_steps // cfg.trace_stride if cfg.trace_stride > 0 else 0
    out["trace"] = np.zeros((n, n_rec, 2), dtype=np.int32) if (trace and n_rec > 0) else None
    out["hist"] = np.zeros((n, cfg.hist_bins), dtype=np.int32) if (hist and cfg.hist_bins > 0) else None
    out["complog"] = (np.zeros((n, cfg.complog_cap, 2), dtype=np.int32)
                      if (complog and cfg.complog_cap > 0) else None)
    out["arrlog"] = np.zeros((n, n_steps), dtype=np.int32) if arrlog else None
    out["arrcls"] = np.zeros((n, n_steps, len(cfg.prompt)), dtype=np.int32) if arrcls else None
    out["admlog"] = np.zeros((n, admlog_cap, 4), dtype=np.int32) if admlog_cap > 0 else None
    out["n_admlog"] = np.zeros(n, dtype=np.int64) if admlog_cap > 0 else None
    o = _Outputs(_p(out["counters"], C.c_int64), _p(out["trace"], C.c_int32), _p(out["hist"], C.c_int32),
                 _p(out["complog"], C.c_int32), _p(out["arrlog"], C.c_int32), _p(out["arrcls"], C.c_int32),
                 _p(out["admlog"], C.c_int32),
                 int(admlog_cap), _p(out["n_admlog"], C.c_int64))
    n_tests = C.c_int64(0)
    rc = lib(sanitize).fcsim_oracle_run_ex(C.byref(c), int(first), int(n), int(n_steps), C.byref(o), int(mc_mode),
                                           C.byref(n_tests))
    if rc != 0:
        raise RuntimeError(f"fcsim_oracle_run failed with code {rc}")
    del keep
    out["n_mc_tests"] = np.array([n_tests.value], dtype=np.int64)
    return out


def run(cfg, first_replica=0, n_replicas=None, n_steps=None, *, trace=True, hist=True, complog=True,
        arrlog=False, admlog_cap=0, threads=1, sanitize=False, arrcls=False, mc_mode=0):
    """Simulate replicas [first_replica, first_replica+n_replicas) for slots 1..n_steps.

    Returns a dict of numpy arrays: counters [n,28] int64, and (when enabled in ``cfg`` and
    requested) trace [n, n_steps//stride, 2], hist [n, bins], complog [n, cap, 2]; diagnostic
    arrlog [n, n_steps] and admlog [n, admlog_cap, 4] with n_admlog [n].
    ``mc_mode``: evaluation of the MC benchmark's future-memory test (Section 4.1): 0 = every future slot is
    summed (the definition, default), 1 = only the last slots of the requests (shortcut), 2 = both, failing
    on the first disagreement; ``n_mc_tests`` in the result counts the tests made (one entry per thread).
    """
    total = sum(g.n_replicas for g in cfg.groups)
    if n_replicas is None:
        n_replicas = total - first_replica
    if n_steps is None:
        n_steps = cfg.T_max
    threads = max(1, min(int(threads), n_replicas)) if n_replicas > 0 else 1
    if threads == 1:
        return _run_range(cfg, first_replica, n_replicas, n_steps, trace, hist, complog, arrlog,
                          admlog_cap, sanitize, arrcls, mc_mode)
    bounds = np.linspace(0, n_replicas, threads + 1).astype(np.int64)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        futs = [ex.submit(_run_range, cfg, first_replica + int(bounds[i]), int(bounds[i + 1] - bounds[i]),
                          n_steps, trace, hist, complog, arrlog, admlog_cap, sanitize, arrcls, mc_mode)
                for i in range(threads)]
        parts = [f.result() for f in futs]
    out = {}
    for k in parts[0]:
        out[k] = None if parts[0][k] is None else np.concatenate([p[k] for p in parts], axis=0)
    return out


def percentile_from_hist(hist64, n, q, shift, max_lat):
    """Smallest bin k whose cumulative count reaches ceil(q*n/100); reported as the bin's
    largest latency ((k+1) << shift) - 1, or max_lat when k is the open last bin."""
    if n <= 0:
        return 0.0
    target = (q * int(n) + 99) // 100
    cum = np.cumsum(hist64.astype(np.int64))
    k = int(np.searchsorted(cum, target, side="left"))
    k = min(k, hist64.shape[0] - 1)
    if k == hist64.shape[0] - 1:
        return float(max_lat)
    return float(((k + 1) << shift) - 1)


def percentile_from_latencies(latencies, q):
    """The ceil(q*n/100)-th smallest of the n latencies (1-based rank), by a plain sort."""
    lat = np.sort(np.asarray(latencies, dtype=np.int64))
    n = lat.shape[0]
    if n == 0:
        return 0.0
    target = (q * n + 99) // 100
    return float(lat[target - 1])


def summarize(cfg, counters, hist, n_steps, complog=None):
    """Per-group int64 sums and fp64 summaries; ``counters``/``hist``/``complog`` cover all replicas.
    Tail latencies (Section 2.2 latency; the "95% latency" of Section 4.1): with a completion log that no replica
    of the group overflowed, the exact order statistic of the logged latencies (percentile_source 2); otherwise
    from the group's histogram (1); 0 when nothing completed or neither exists (0)."""
    res = []
    first = 0
    for g in cfg.groups:
        blk = counters[first:first + g.n_replicas]
        sums = {}
        for name, i in CIDX.items():
            col = blk[:, i]
            if name in MAX_FIELDS:
                sums[name] = int(col.max())
            elif name in OR_FIELDS:
                sums[name] = int(np.bitwise_or.reduce(col))
            elif name == "steps_done":
                sums[name] = int(col.max())
            else:
                sums[name] = int(col.sum(dtype=np.int64))
        n = g.n_replicas
        T = int(n_steps)
        done = sums["completed"]
        s = dict(sums)
        s["mean_latency"] = (sums["sum_lat"] / done) if done > 0 else 0.0
        s["mean_utilisation"] = sums["sum_U"] / (float(n) * T * cfg.M) if T > 0 else 0.0
        s["request_throughput"] = done / (float(n) * T) if T > 0 else 0.0
        s["token_throughput"] = sums["tokens_generated"] / (float(n) * T) if T > 0 else 0.0
        s["p95_latency"] = 0.0
        s["p99_latency"] = 0.0
        s["percentile_source"] = 0
        if complog is not None and cfg.complog_cap > 0 and done > 0 and not (sums["status"] & 2):
            n_log = blk[:, CIDX["n_logged"]]
            lats = np.concatenate([complog[first + r, :n_log[r], 1] for r in range(g.n_replicas)])
            assert lats.shape[0] == done
            s["p95_latency"] = percentile_from_latencies(lats, 95)
            s["p99_latency"] = percentile_from_latencies(lats, 99)
            s["percentile_source"] = 2
        elif hist is not None and cfg.hist_bins > 0 and done > 0:
            h = hist[first:first + g.n_replicas].astype(np.int64).sum(axis=0)
            s["p95_latency"] = percentile_from_hist(h, done, 95, cfg.hist_shift, sums["max_lat"])
            s["p99_latency"] = percentile_from_hist(h, done, 99, cfg.hist_shift, sums["max_lat"])
            s["percentile_source"] = 1
        res.append(s)
        first += g.n_replicas
    return res
