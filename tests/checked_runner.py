"""Runs a spread of configurations through the index-checked build of the CUDA library (every shared-memory and
output index of the step kernels is compared with its bound; the first violation is recorded instead of performed)
and prints the number of recorded violations.  Started by test_gpu_parity.py in a process of its own, because a
process loads one build of the library."""
import os
import sys

os.environ["FCSIM_CHECKED"] = "1"
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2604_11001_b200 import binding as fb  # noqa: E402
from paper_2604_11001_b200 import workloads as wl  # noqa: E402


def main():
    assert fb.fcsim_is_checked_build()
    bad = []

    def run(cfg, pieces=None):
        sim = fb.Simulation(cfg)
        for s in (pieces or [cfg.T_max]):
            sim.run(s)
        sim.stats()
        rec = fb.fcsim_debug_read(sim.handle)
        if rec[0] != 0:
            bad.append((cfg.name, rec[:4]))
        sim.close()

    for seed in range(24):
        run(wl.random_small_config(seed))
    for seed in range(12):
        cfg = wl.random_medium_config(seed)
        cut = 1 + (seed * 97) % (cfg.T_max - 1)
        run(cfg, [cut, cfg.T_max - cut])
    run(wl.config2(replicas=32, T=3000))
    run(wl.config3(n_rates=4, n_b=4, reps=2, T=3000))
    run(wl.config4(replicas=32, T=3000))
    run(wl.config5(replicas=128, T=5000), [2000, 3000])
    run(wl.config6(replicas=16, T=1500, total_rate=15.0))
    for name, rec in bad:
        print("violation", name, rec)
    print("violations:", len(bad))


if __name__ == "__main__":
    main()
