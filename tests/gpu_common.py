"""Helpers for the GPU parity tests: run a configuration through the C ABI and compare with the CPU checker."""
from __future__ import annotations

import numpy as np

from oracle import fcsim_oracle as orc


def run_gpu(cfg, n_steps=None, pieces=None):
    """Run on cuda:0 through the binding.  ``pieces``: list of step counts (resumed launches)."""
    from paper_2604_11001_b200 import binding as fb
    n_steps = cfg.T_max if n_steps is None else n_steps
    sim = fb.Simulation(cfg)
    for s in (pieces or [n_steps]):
        sim.run(s)
    counters, summary = sim.stats()
    out = {"counters": counters, "summary": summary}
    for name in ("trace", "hist", "complog"):
        v = getattr(sim, name)()
        out[name] = None if v is None else v.cpu().numpy()
    out["launch"] = sim.launch_info()
    sim.close()
    return out


def assert_same(cfg, gpu, ref, n_steps, what=""):
    """Bit-exact comparison of every output word (integer work: no tolerance)."""
    gc, rc = gpu["counters"], ref["counters"]
    if not (gc == rc).all():
        bad = np.argwhere(gc != rc)
        r, f = bad[0]
        raise AssertionError(f"{what} counters differ at replica {r} field {orc.COUNTER_NAMES[f]}: "
                             f"gpu {gc[r, f]} ref {rc[r, f]} ({len(bad)} words differ)")
    if ref.get("trace") is not None:
        n_rec = n_steps // cfg.trace_stride
        g = gpu["trace"][:, :n_rec]
        if not (g == ref["trace"]).all():
            bad = np.argwhere(g != ref["trace"])
            r, t, w = bad[0]
            raise AssertionError(f"{what} trace differs at replica {r} record {t} word {w}: gpu {g[r, t, w]} "
                                 f"ref {ref['trace'][r, t, w]} ({len(bad)} words differ)")
    if ref.get("hist") is not None:
        assert (gpu["hist"] == ref["hist"]).all(), f"{what} histogram differs"
    if ref.get("complog") is not None:
        n = ref["counters"][:, orc.CIDX["n_logged"]]
        for r in range(rc.shape[0]):
            assert (gpu["complog"][r, :n[r]] == ref["complog"][r, :n[r]]).all(), f"{what} completion log differs (replica {r})"


def assert_summary_close(cfg, gpu_summary, counters, hist, n_steps, complog=None, rtol=1e-9):
    """fp64 summaries derived from int64 sums: relative 1e-9.  With the checker's completion log the tail
    latencies must be the exact order statistics, and say so."""
    ref = orc.summarize(cfg, counters, hist, n_steps, complog)
    for g, (a, b) in enumerate(zip(gpu_summary, ref)):
        for k in orc.COUNTER_NAMES:
            assert a[k] == b[k], (g, k, a[k], b[k])
        for k in ("mean_latency", "p95_latency", "p99_latency", "mean_utilisation", "request_throughput",
                  "token_throughput"):
            assert abs(a[k] - b[k]) <= rtol * max(abs(b[k]), 1e-300), (g, k, a[k], b[k])
        if complog is not None or cfg.complog_cap == 0:
            assert a["percentile_source"] == b["percentile_source"], (g, a["percentile_source"], b["percentile_source"])
