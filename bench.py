#!/usr/bin/env python
"""Benchmark of the batched Monte-Carlo simulator: simulated replica-steps per second.

A bench step advances every replica of the workload by ``--chunk`` slots (one fcsim_run call).
W warm-up steps bring the replicas from the empty system into their loaded regime, then exactly K
steps are timed with CUDA events on the launching stream, bracketed by synchronisation (and a
barrier when several ranks run).  One JSON line is printed by rank 0.

  python bench.py                         # 1 GPU, preset 5 (large bursty run)
  python bench.py --workload 3            # another preset
  python bench.py --impl reference        # the CPU checker timed on the host cores (bounded sample)
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "simulated replica-steps/s"
UNIT = "replica-steps/s"

# Executed warp-instructions and DRAM bytes per replica-step of the step kernels come from ncu captures and are
# kept, with the SHA-256 of the kernel sources they were taken on, in profiles/kernel_constants.json
# (written by paper_2604_11001_b200/profile_constants.py).  When the sources have changed since, the figures that
# depend on them are printed as null and the line says that the constants are stale.

DEFAULT_CHUNK = {1: 200, 2: 1000, 3: 2000, 4: 2000, 5: 4000, 6: 500}
NAMES = {1: "cfg1-tiny-flow", 2: "cfg2-policy-comparison", 3: "cfg3-stability-sweep", 4: "cfg4-heavy-tail",
         5: "cfg5-large-bursty", 6: "cfg6-paper-section-4.1"}
SIDE_WORKLOADS = (1, 2, 3, 4, 6)     # reported next to the headline workload in the default run


def make_config(workload: int, total_steps: int, rank: int = 0, replicas: int = 0):
    from paper_2604_11001_b200 import workloads as wl
    kw = {"T": total_steps}
    if replicas and workload != 3:
        kw["replicas"] = replicas
    if replicas and workload == 3:
        kw["reps"] = max(1, replicas // 4096)
    cfg = wl.PRESETS[workload](**kw)
    if rank:
        from paper_2604_11001_b200 import sharding
        cfg = sharding.shard_for_rank(cfg, rank)
    return cfg


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def wait_first_sample(self, timeout_s: float = 3.0):
        """Block until nvidia-smi has written its first line (its start-up takes longer than a short timed region)."""
        t0 = time.perf_counter()
        while self.proc is not None and time.perf_counter() - t0 < timeout_s:
            if os.path.getsize(self.tmp.name) > 0:
                return
            time.sleep(0.02)

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, reasons, smax, power = [], set(), None, []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax = float(f[1])
                power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=smax, reasons=sorted(reasons), samples=len(sm),
                       power_w_max=max(power) if power else None)
        return out


def oracle_sample(workload: int, slots: int, n_rep: int):
    """The CPU checker, as it stands, on a bounded sample of the workload: n_rep replicas spread evenly
    over the groups (the first replicas of each) for slots 1..slots, one thread per host core.
    Returns (replica-steps/s, cores, description, seconds)."""
    from oracle import fcsim_oracle as orc
    from paper_2604_11001_b200 import workloads as wl
    cores = os.cpu_count() or 1
    if workload == 3:
        reps = max(1, n_rep // 64)
        sub = wl.config3(n_rates=8, n_b=8, reps=reps, T=slots)   # an 8 x 8 sub-grid of the sweep
    else:
        cfg = wl.PRESETS[workload]()
        per = max(1, n_rep // len(cfg.groups))
        groups = tuple(dataclasses.replace(g, n_replicas=min(g.n_replicas, per)) for g in cfg.groups)
        sub = cfg.with_(groups=groups, T_max=slots)
    n = sub.n_replicas
    orc.lib()
    t0 = time.perf_counter()
    orc.run(sub, 0, n, slots, threads=cores, trace=False, complog=False)
    dt = time.perf_counter() - t0
    desc = f"{n} replicas (evenly over {len(sub.groups)} groups) x slots 1..{slots}, {cores} threads"
    return n * slots / dt, cores, desc, dt


def sized_oracle_sample(workload: int, slots: int, target_s: float):
    """Probe briefly, then run a sample sized to about target_s seconds of host time."""
    cores = os.cpu_count() or 1
    v, _, _, _ = oracle_sample(workload, slots, 2 * cores)
    n = int(max(2 * cores, min(32768, v * target_s / slots)))
    return oracle_sample(workload, slots, n)


def run_reference(args):
    """--impl reference: the CPU checker timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    slots = 2000 if args.workload == 1 else 3000
    n_all = max(1, args.steps + args.warmup)
    per_step_s = min(20.0, 150.0 / n_all)
    cores = os.cpu_count() or 1
    v, _, _, _ = oracle_sample(args.workload, slots, 2 * cores)
    n = int(max(2 * cores, min(32768, v * per_step_s / slots)))
    times, vals, desc = [], [], ""
    for i in range(args.warmup + args.steps):
        v, cores, desc, dt = oracle_sample(args.workload, slots, n)
        if i >= args.warmup:
            times.append(dt)
            vals.append(v)
    value = sum(vals) / max(1, len(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / max(1, len(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": NAMES[args.workload], "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


def run_workload(args, workload, steps, warmup, chunk, cpu_seconds, ctx):
    """One workload through the device-buffer path (timed with CUDA events), the host-buffer path (wall clock) and
    the CPU checker (bounded sample); returns the fields of a bench line."""
    import torch
    from paper_2604_11001_b200 import binding as fb
    from paper_2604_11001_b200 import profile_constants as pc
    rank, world, local_rank, dist = ctx["rank"], ctx["world"], ctx["local_rank"], ctx["dist"]
    total_steps = (warmup + steps) * chunk
    cfg = make_config(workload, total_steps, rank, args.replicas)

    # CPU baseline first (rank 0 only): no GPU work is in flight while the host cores are timed
    cpu_baseline = None
    if rank == 0 and world == 1 and cpu_seconds > 0:
        v, cores, desc, dt = sized_oracle_sample(workload, 2000 if workload == 1 else 3000, cpu_seconds)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                        "seconds": round(dt, 2)}

    sim = fb.Simulation(cfg, device=f"cuda:{local_rank}")
    info = sim.launch_info()
    stream = torch.cuda.current_stream()
    R = cfg.n_replicas

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # Clock record: sampled during the timed region.  A workload whose whole run is shorter than the sampler's
    # period (presets 1 and 2: milliseconds) is sampled over warm-up and timed steps together, repeated until the
    # window holds samples, and the record says so.
    est_ms = R * chunk * steps / 3.0e6          # at about 3e9 replica-steps/s
    short = est_ms < 400.0
    sampler = None
    if rank == 0 and short:
        sampler = ClockSampler(local_rank)
        sampler.wait_first_sample()
    for _ in range(warmup):
        sim.run(chunk, stream)
    barrier()
    if rank == 0 and not short:
        sampler = ClockSampler(local_rank)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record(stream)
    for i in range(steps):
        sim.run(chunk, stream)
        ev[i + 1].record(stream)
    barrier()
    if sampler is not None and short:
        time.sleep(0.25)                        # at least two sampler periods inside the window
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["window"] = ("warm-up and timed steps plus 0.25 s (the run is shorter than the sampler's period)"
                            if short else "timed steps")
    ms_total = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    if dist is not None:
        tmax = torch.tensor([ms_total], device="cuda", dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        ms_total = float(tmax.item())
    value = world * R * chunk * steps / (ms_total * 1e-3)
    n_policies = len({g.policy for g in cfg.groups})   # one kernel per policy, side by side on forked streams
    launches_per_step = -(-chunk // info["max_steps_per_launch"]) * n_policies

    # sanity of the timed state: the counters must show the work was done
    counters, summary = sim.stats(stream)
    assert int(counters[:, 0].min()) == total_steps, "replicas did not advance"
    done_steps = int(counters[:, 0].sum())
    sizes = fb.fcsim_query_sizes(cfg)
    sim.close()
    del sim
    torch.cuda.empty_cache()

    # end to end through the host-buffer entry point: tables from host memory, every output back to host
    e2e = None
    out_bytes = sizes["counters"] + sizes["trace"] + sizes["hist"] + sizes["complog"]
    if not args.no_e2e and out_bytes > 16e9:
        e2e = {"value": None, "unit": UNIT,
               "skipped": "outputs of %.1f GB are not copied to host buffers in the default run" % (out_bytes / 1e9)}
    elif not args.no_e2e:
        # every rank runs its own shard through the host-buffer entry point; the time is the maximum over ranks
        host = fb.host_output_arrays(cfg, pinned=True)   # page-locked result buffers, allocated outside the timing
        barrier()
        t0 = time.perf_counter()
        out = fb.fcsim_simulate_host(cfg, total_steps, out=host)
        dt = time.perf_counter() - t0
        assert (out["counters"] == counters).all(), "host-buffer run differs from the device-buffer run"
        del host, out
        if dist is not None:
            tm = torch.tensor([dt], device="cuda", dtype=torch.float64)
            dist.all_reduce(tm, op=dist.ReduceOp.MAX)
            dt = float(tm.item())
        table_bytes = 4 * (cfg.class_law.n + sum(t.n for t in cfg.prompt) + sum(t.n for t in cfg.decode)
                           + sum(t.n for a in cfg.arrivals for t in a.count))
        n_all = warmup + steps
        e2e = {"value": world * R * total_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": world * table_bytes / n_all,
               "d2h_bytes_per_step": world * (out_bytes + sizes["scratch"]) / n_all,
               "what": "fcsim_simulate_host: tables H2D + all %d slots from the empty system + every output "
                       "copied to pinned host buffers, wall clock (max over ranks); bytes amortised over %d steps"
                       % (total_steps, n_all),
               "seconds": round(dt, 3)}

    peaks, peak_kind = measured_peaks()
    sm_mhz = (clocks or {}).get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
    peak_ginst = info["sm_count"] * 4 * sm_mhz * 1e6 / 1e9       # warp-instructions/s the schedulers can issue
    consts = pc.load()
    k = None if (consts["stale"] or args.replicas) else consts["presets"].get(str(workload))
    ipr = k["inst_per_replica_step"] if k else None
    dbr = k["dram_bytes_per_replica_step"] if k else None
    kernel_ms = statistics.mean(per_step) / (launches_per_step // n_policies)
    roofline = {
        "bound": "alu",
        "kernel": "fcsim_step_kernel<policy, ctas, rec>: %d concurrent launch(es) per step, one per policy; figures "
                  "are sums over them" % n_policies,
        "achieved": (ipr * value / world / 1e9) if ipr else None,
        "peak": peak_ginst, "unit": "Gwarp-inst/s",
        "frac": (ipr * value / world / 1e9 / peak_ginst) if ipr else None,
        "traffic": (dbr * R * min(chunk, info["max_steps_per_launch"])) if dbr else None,
        "inst_per_replica_step": ipr,
        "ncu_issue_active_pct": [round(x["issue_active_pct"], 1) for x in k["kernels"]] if k else None,
        "constants": {"file": "profiles/kernel_constants.json", "sha256_at_capture": consts.get("sha256"),
                      "sha256_now": pc.source_hash(), "stale": bool(consts["stale"]),
                      "captured_on": ({"replicas": k["replicas"], "slots": k["slots"]} if k else None)},
        "constants_stale": bool(consts["stale"]),
        "peak_basis": "%d SMs x 4 schedulers x %.0f MHz (median SM clock sampled during the timed region)"
                      % (info["sm_count"], sm_mhz),
        "kernel_ms_per_launch": kernel_ms, "launches_per_step": launches_per_step, "policies": n_policies,
        "hbm_peak_gbs": peaks.get("hbm_gbs"), "hbm_peak_kind": peak_kind,
    }
    if cfg.trace_stride > 0:
        rec_bytes = 8.0 / cfg.trace_stride
        roofline["trace_stream_gbs"] = value / world * rec_bytes / 1e9
        roofline["trace_stream_frac_of_hbm"] = roofline["trace_stream_gbs"] / peaks.get("hbm_gbs", 6650.0)
    return {
        "value": value, "ms_per_step": ms_total / steps, "steps": steps, "warmup": warmup,
        "config": {"workload": NAMES[workload], "replicas_per_gpu": R, "slots_per_step": chunk,
                   "warm_slots": warmup * chunk, "groups": len(cfg.groups), "M": cfg.M, "K": cfg.K,
                   "Qcap": cfg.Qcap, "Acap": cfg.Acap,
                   "l2": ("replica state %.0f MB exceeds the 126 MB L2; no explicit flush" % (sizes["workspace"] / 1e6)
                          if sizes["workspace"] > 126e6 else
                          "replica state %.0f MB fits the 126 MB L2 (small preset); its %.0f MB of per-slot outputs do "
                          "not; no explicit flush" % (sizes["workspace"] / 1e6,
                                                     (sizes["trace"] + sizes["complog"] + sizes["hist"]) / 1e6)),
                   "launch": info, "parallelism": "replicas only, %d per GPU" % R},
        "clocks": clocks, "e2e": e2e, "gpu_launches": steps * launches_per_step,
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "check": {"replica_steps_done": done_steps, "completed": int(counters[:, 5].sum()),
                  "mean_latency": [round(s["mean_latency"], 3) for s in summary[:4]],
                  "p95_latency": [s["p95_latency"] for s in summary[:4]],
                  "percentile_source": [s["percentile_source"] for s in summary[:4]]},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=5, choices=[1, 2, 3, 4, 5, 6])
    ap.add_argument("--chunk", type=int, default=0, help="slots per bench step (0 = preset default)")
    ap.add_argument("--replicas", type=int, default=0, help="replicas per group (0 = the preset's; profiling aid)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-side-workloads", action="store_true",
                    help="only the headline workload (the default run also reports the other presets)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    ctx = {"rank": rank, "world": world, "local_rank": local_rank, "dist": dist}

    chunk = args.chunk or DEFAULT_CHUNK[args.workload]
    if args.workload == 5 and not args.chunk:
        # the horizon of the large bursty run is 100 000 slots: with the default 5 + 20 steps the run is exactly that
        chunk = min(chunk, max(1, 100000 // max(1, args.warmup + args.steps)))
    head = run_workload(args, args.workload, args.steps, args.warmup, chunk,
                        0.0 if args.no_cpu_baseline else 15.0, ctx)

    # the other presets, three timed steps each after five warm-up steps (1 GPU, headline workload only)
    side = None
    if args.workload == 5 and world == 1 and not args.no_side_workloads and not args.replicas:
        side = {}
        for w in SIDE_WORKLOADS:
            r = run_workload(args, w, 3, 5, DEFAULT_CHUNK[w], 0.0 if args.no_cpu_baseline else 5.0, ctx)
            rf = r["roofline"]
            side[NAMES[w]] = {
                "value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"], "steps": 3, "warmup": 5,
                "slots_per_step": DEFAULT_CHUNK[w], "replicas": r["config"]["replicas_per_gpu"],
                "frac": rf["frac"], "inst_per_replica_step": rf["inst_per_replica_step"],
                "ncu_issue_active_pct": rf["ncu_issue_active_pct"], "constants_stale": rf["constants_stale"],
                "trace_stream_gbs": rf.get("trace_stream_gbs"),
                "trace_stream_frac_of_hbm": rf.get("trace_stream_frac_of_hbm"),
                "e2e": r["e2e"], "cpu_baseline": r["cpu_baseline"], "clocks": r["clocks"],
                "gpu_launches": r["gpu_launches"], "check": r["check"]}

    if rank != 0:
        dist.destroy_process_group()
        return
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": head["config"], "clocks": head["clocks"], "e2e": head["e2e"],
        "gpu_launches": head["gpu_launches"], "roofline": head["roofline"], "cpu_baseline": head["cpu_baseline"],
        "check": head["check"],
    }
    if side is not None:
        line["workloads"] = side
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
