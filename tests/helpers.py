"""Shared test helpers: fixture parsing and small configuration builders (no simulator logic)."""
from __future__ import annotations

import os

import numpy as np

from paper_2604_11001_b200 import workloads as wl

POLICIES = {"flow": wl.POLICY_FLOW, "greedy": wl.POLICY_GREEDY, "chunked": wl.POLICY_CHUNKED,
            "alpha": wl.POLICY_ALPHA, "mc": wl.POLICY_MC}


def degenerate_config(n, l, o, policy, b, K, c, M, T, Qcap=64, Acap=64, replicas=1, ma=0, keep=0, n2=None,
                      thr0=0, thr1=0, **extra):
    """Constant arrival count n per slot, constant lengths (l, o).  With ``n2`` the arrival law has two states:
    n arrivals per slot in state 0, n2 in state 1, switching thresholds (thr0, thr1)."""
    pol = POLICIES[policy] if isinstance(policy, str) else policy
    arrivals = wl.Arrivals((wl.constant_table(n),))
    if n2 is not None:
        arrivals = wl.Arrivals((wl.constant_table(n), wl.constant_table(n2)), (int(thr0), int(thr1)))
    return wl.SimConfig(
        M=M, K=K, T_max=T, Qcap=Qcap, Acap=Acap, seed=extra.pop("seed", 7),
        class_law=wl.constant_table(0), prompt=(wl.constant_table(l),), decode=(wl.constant_table(o),),
        arrivals=(arrivals,),
        groups=(wl.Group(pol, b_fp=wl.b_to_fp(b), chunk=c, n_replicas=replicas, m_admit=ma, preempt_keep=keep),),
        trace_stride=1, hist_bins=extra.pop("hist_bins", 16), hist_shift=0, complog_cap=4 * T, **extra)


def read_fixture(path):
    fx = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split(":", 1)
            fx[key.strip()] = val.strip()
    params = {}
    for tok in fx.pop("params").split():
        k, v = tok.split("=")
        params[k] = v if k == "policy" else (float(v) if k == "b" else int(v))
    out = {"params": params, "U": [int(x) for x in fx.pop("U").split()],
           "Q": [int(x) for x in fx.pop("Q").split()],
           "completions": [tuple(int(y) for y in x.split(":")) for x in fx.pop("completions", "").split()]}
    out["counters"] = {k: int(v) for k, v in fx.items()}
    return out


def trace_fixtures(golden_dir):
    return sorted(p for p in os.listdir(golden_dir) if p.startswith("trace_") and p.endswith(".txt"))


def scaled_presets():
    """The five preset workloads cut down to sizes the CPU checker finishes in seconds."""
    return [
        wl.config1(replicas=16, T=2000),
        wl.config2(replicas=3, T=4000),
        wl.config3(n_rates=3, n_b=3, reps=2, T=4000),
        wl.config4(replicas=3, T=4000, trace_stride=4),
        wl.config5(replicas=3, T=6000),
        wl.config6(replicas=3, T=3000),
    ]
