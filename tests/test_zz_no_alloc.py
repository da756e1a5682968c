"""The allocation-free statistics entry point against the ordinary one (collected last on purpose).

fcsim_stats_noalloc serves hosts that cannot allocate device memory when they ask for statistics, for
instance a serving process whose own memory manager already holds the whole GPU, or a thread that must
not cause the device-wide stall of an allocation.  It keeps its per-group rows in a fixed array inside
the library, which every call shares and which still holds the previous call's rows; so the check runs
two calls in a row, on different data, and compares each with fcsim_stats on the same state.
"""
import pytest

from paper_2604_11001_b200 import workloads as wl

pytestmark = pytest.mark.gpu
FLOATS = ("mean_latency", "p95_latency", "p99_latency", "mean_utilisation", "request_throughput",
          "token_throughput")


def _same(a, b):
    from paper_2604_11001_b200 import binding as fb
    assert len(a) == len(b)
    for ga, gb in zip(a, b):
        for k in fb.COUNTER_NAMES:            # int64 sums: exact
            assert ga[k] == gb[k], k
        for k in FLOATS:                      # fp64 summaries: relative 1e-9 as everywhere else
            assert abs(ga[k] - gb[k]) <= 1e-9 * max(abs(gb[k]), 1e-300), k
        assert ga["percentile_source"] == gb["percentile_source"]


def test_two_calls_in_a_row_match_fcsim_stats():
    from paper_2604_11001_b200 import binding as fb
    first = fb.Simulation(wl.config3(n_rates=3, n_b=4, reps=5, T=900).with_(Qcap=64, Acap=256))
    second = fb.Simulation(wl.config1(replicas=40, T=500))   # other shape: 1 group, other bin count meaning
    first.run(600)
    ref1 = first.stats()[1]
    got1 = fb.fcsim_stats_noalloc(first.handle, first.G)
    _same(got1, ref1)
    assert sum(g["completed"] for g in got1) > 0
    # second call on other data, then the first handle again after more slots: stale rows must not leak
    second.run(500)
    _same(fb.fcsim_stats_noalloc(second.handle, second.G), second.stats()[1])
    first.run(300)
    ref2 = first.stats()[1]
    got2 = fb.fcsim_stats_noalloc(first.handle, first.G)
    _same(got2, ref2)
    assert got2[0]["steps_done"] == 900 and got2 != got1
    first.close()
    second.close()


def test_rows_beyond_the_fixed_scratch_are_refused():
    from paper_2604_11001_b200 import binding as fb
    cfg = wl.config3(n_rates=16, n_b=16, reps=1, T=32).with_(Qcap=32, Acap=64)   # 256 groups x (28 + 1024) words
    sim = fb.Simulation(cfg)
    sim.run(32)
    with pytest.raises(fb.FcsimError) as e:
        fb.fcsim_stats_noalloc(sim.handle, sim.G)
    assert e.value.code == -7
    assert "scratch" in fb.fcsim_strerror(-7)
    sim.close()
