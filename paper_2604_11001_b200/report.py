"""Policy comparison on the paper's synthetic setting (Section 4.1): average latency, 95 % latency, request
throughput and token throughput (the metrics of Section 2.2) for every policy group of preset 6, at the
horizons T = 1000, 2000, .., 10000, from one resumable GPU run.

    python -m paper_2604_11001_b200.report [--replicas 1024] [--rate 15] [--keep-tokens]
"""
from __future__ import annotations

import argparse
import dataclasses

from . import binding as fb
from . import workloads as wl

NAMES = ("Algorithm 2, b=12", "greedy + LIFO eviction", "alpha-protection greedy", "Algorithm 1, b=(4,4,4)",
         "MC, known lengths", "MC, worst-case lengths")


def run(replicas: int = 1024, horizons=range(1000, 10001, 1000), device: str = "cuda:0", total_rate: float = 5.0,
        keep_tokens: bool = False):
    cfg = wl.config6(replicas=replicas, T=max(horizons), total_rate=total_rate)
    if keep_tokens:  # evicted requests keep their generated tokens as prompt (not the paper's rule); MC never evicts
        cfg = cfg.with_(groups=tuple(g if g.policy == wl.POLICY_MC else dataclasses.replace(g, preempt_keep=1)
                                     for g in cfg.groups))
    sim = fb.Simulation(cfg, device=device)
    rows = []
    for T in horizons:
        sim.run(T - sim.steps_done)
        _, summary = sim.stats(want_counters=False)
        for g, s in enumerate(summary):
            rows.append(dict(T=T, policy=NAMES[g], mean_latency=s["mean_latency"], p95_latency=s["p95_latency"],
                             request_throughput=s["request_throughput"], token_throughput=s["token_throughput"],
                             evictions=s["evictions"], overflow_steps=s["overflow_steps"], dropped=s["dropped"]))
    sim.close()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--replicas", type=int, default=1024)
    ap.add_argument("--rate", type=float, default=5.0, help="total arrivals per slot (5 = total, 15 = 5 per class)")
    ap.add_argument("--keep-tokens", action="store_true",
                    help="evicted requests keep their generated tokens as prompt instead of being refreshed")
    args = ap.parse_args()
    rows = run(args.replicas, total_rate=args.rate, keep_tokens=args.keep_tokens)
    print("%6s  %-26s %12s %12s %14s %14s %10s %10s" % ("T", "policy", "mean lat", "p95 lat", "requests/slot",
                                                          "tokens/slot", "evictions", "dropped"))
    for r in rows:
        if r["T"] in (1000, 5000, 10000):
            print("%6d  %-26s %12.2f %12.0f %14.4f %14.3f %10d %10d" % (
                r["T"], r["policy"], r["mean_latency"], r["p95_latency"], r["request_throughput"],
                r["token_throughput"], r["evictions"], r["dropped"]))


if __name__ == "__main__":
    main()
