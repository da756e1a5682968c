"""Roofline constants of the step kernels, taken from ncu counter captures.

The benchmark reports the step kernels against the issue-slot roofline as
(executed warp-instructions per replica-step) x (measured replica-steps/s) / (SMs x 4 x SM clock).
The first factor cannot be measured inside a timed run; it comes from an ncu capture of the launches of
one bench step (one kernel per policy present):

    ncu --metrics smsp__inst_executed.sum,smsp__issue_active.avg.pct_of_peak_sustained_active,\
gpu__time_duration.sum,dram__bytes_read.sum,dram__bytes_write.sum --clock-control none \
        -k regex:fcsim_step -s <launches of the warm-up steps> -c <launches of one step> \
        --csv --log-file light_w<N>.csv python bench.py --workload <N> --steps 2 --warmup 5 \
        --no-cpu-baseline --no-e2e --no-side-workloads [--replicas R]

This module turns such logs into ``profiles/kernel_constants.json``, stamped with the SHA-256 of the kernel
sources, so that the benchmark can tell whether the constants still describe the code it times:

    python -m paper_2604_11001_b200.profile_constants 5:light_w5.csv:32768 3:light_w3.csv:2048 2:light_w2.csv ...

(preset : ncu log : replicas per group given to bench.py, when not the preset's own).
"""
from __future__ import annotations

import collections
import csv
import datetime
import hashlib
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SOURCES = ("paper_2604_11001_b200/csrc/fcsim_device.cuh", "paper_2604_11001_b200/csrc/fcsim_step_kernels.cu",
           "paper_2604_11001_b200/csrc/fcsim.cu")
CONSTANTS = os.path.join(ROOT, "profiles", "kernel_constants.json")
METRICS = ("smsp__inst_executed.sum,smsp__issue_active.avg.pct_of_peak_sustained_active,gpu__time_duration.sum,"
           "dram__bytes_read.sum,dram__bytes_write.sum")


def source_hash() -> str:
    """SHA-256 over the kernel source files, in the order of SOURCES."""
    h = hashlib.sha256()
    for rel in SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def load() -> dict:
    """The stored constants plus ``stale``: whether the sources have changed since they were captured."""
    if not os.path.exists(CONSTANTS):
        return {"presets": {}, "sha256": None, "stale": True}
    with open(CONSTANTS) as f:
        d = json.load(f)
    d["stale"] = d.get("sha256") != source_hash()
    return d


def parse_ncu_log(path: str):
    """Per captured launch, in order: (kernel name, {metric: value})."""
    with open(path) as f:
        rows = list(csv.reader(line for line in f if line.startswith('"')))
    hdr = rows[0]
    ii, ki, mi, vi = (hdr.index(n) for n in ("ID", "Kernel Name", "Metric Name", "Metric Value"))
    per = collections.OrderedDict()
    for r in rows[1:]:
        per.setdefault((r[ii], r[ki]), {})[r[mi]] = float(r[vi].replace(",", ""))
    return [(k[1], m) for k, m in per.items()]


def constants_of(preset: int, log: str, replicas: int = 0) -> dict:
    import bench  # the chunk sizes and the preset construction are the benchmark's
    chunk = bench.DEFAULT_CHUNK[preset]
    cfg = bench.make_config(preset, 8 * chunk, 0, replicas)
    launches = parse_ncu_log(log)
    n_pol = len({g.policy for g in cfg.groups})
    if len(launches) != n_pol:
        raise SystemExit(f"preset {preset}: {len(launches)} launches captured, one bench step has {n_pol}")
    rs = cfg.n_replicas * chunk
    inst = sum(m["smsp__inst_executed.sum"] for _, m in launches)
    dram = sum(m["dram__bytes_read.sum"] + m["dram__bytes_write.sum"] for _, m in launches)
    cmd = ("ncu --metrics %s --clock-control none -k regex:fcsim_step -s S -c %d --csv --log-file %s python bench.py "
           "--workload %d --steps 2 --warmup 5 --no-cpu-baseline --no-e2e --no-side-workloads%s"
           % (METRICS, n_pol, os.path.basename(log), preset, (" --replicas %d" % replicas) if replicas else ""))
    return {
        "inst_per_replica_step": inst / rs,
        "dram_bytes_per_replica_step": dram / rs,
        "replicas": cfg.n_replicas, "slots": chunk,
        "kernels": [{"name": k.replace("void ", "").replace("(Params)", "").replace("fcsim_dev::", ""),
                     "duration_ms": m["gpu__time_duration.sum"] / 1e6,
                     "warp_instructions": m["smsp__inst_executed.sum"],
                     "issue_active_pct": m["smsp__issue_active.avg.pct_of_peak_sustained_active"],
                     "dram_bytes": m["dram__bytes_read.sum"] + m["dram__bytes_write.sum"]} for k, m in launches],
        "command": cmd,
    }


def main(argv):
    if not argv:
        raise SystemExit(__doc__)
    sys.path.insert(0, ROOT)
    old = load()
    presets = {} if old.get("stale") else dict(old.get("presets", {}))
    for spec in argv:
        parts = spec.split(":")
        preset, log = int(parts[0]), parts[1]
        replicas = int(parts[2]) if len(parts) > 2 else 0
        presets[str(preset)] = constants_of(preset, log, replicas)
    out = {"sources": list(SOURCES), "sha256": source_hash(),
           "captured": datetime.datetime.now(datetime.timezone.utc).strftime("%Y-%m-%d"),
           "what": "executed warp-instructions and DRAM bytes per replica-step of the step kernels, summed over the "
                   "launches of one bench step (one kernel per policy present), from ncu; valid for the sources "
                   "whose SHA-256 is given",
           "presets": presets}
    os.makedirs(os.path.dirname(CONSTANTS), exist_ok=True)
    with open(CONSTANTS, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")
    for p, c in sorted(presets.items()):
        print("preset %s: %.1f warp-instructions, %.1f DRAM bytes per replica-step; issue active %s"
              % (p, c["inst_per_replica_step"], c["dram_bytes_per_replica_step"],
                 ", ".join("%.1f %%" % k["issue_active_pct"] for k in c["kernels"])))


if __name__ == "__main__":
    main(sys.argv[1:])
