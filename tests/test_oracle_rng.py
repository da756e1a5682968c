"""Pins for the checker's random numbers: Philox4x32-10 known answers and the inverse-CDF rule."""
import os

import numpy as np
import pytest

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl
from pyref import philox_py, sample_py


def _kat(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "philox_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            c, k, o = [[int(x, 16) for x in part.split()] for part in line.split("|")]
            rows.append((c, k, o))
    return rows


def test_philox_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for c, k, o in rows:
        assert list(orc.philox(c, k)) == o
        assert list(philox_py(c, k)) == o


def test_philox_matches_python_definition():
    rng = np.random.default_rng(123)
    for _ in range(2000):
        c = rng.integers(0, 2 ** 32, size=4)
        k = rng.integers(0, 2 ** 32, size=2)
        assert orc.philox(c, k) == philox_py(c, k)


def test_philox_counter_words_are_not_interchangeable():
    # a transposed counter word or key word must change the output
    base = orc.philox((1, 2, 3, 4), (5, 6))
    assert orc.philox((2, 1, 3, 4), (5, 6)) != base
    assert orc.philox((1, 2, 4, 3), (5, 6)) != base
    assert orc.philox((1, 2, 3, 4), (6, 5)) != base


def test_philox_words_uniform():
    # 4 x 20000 words: mean and bit balance of a uniform 32-bit source
    words = np.array([orc.philox((i, 9, 1, 0), (11, 0)) for i in range(20000)], dtype=np.float64)
    assert abs(words.mean() / 2 ** 32 - 0.5) < 0.005
    for col in range(4):
        assert abs((words[:, col] >= 2 ** 31).mean() - 0.5) < 0.02


def test_sample_is_the_literal_scan():
    rng = np.random.default_rng(5)
    tabs = [wl.poisson_table(2.0), wl.uniform_table(16, 128), wl.geometric_table(64.0, 512),
            wl.constant_table(9), wl.table_from_pmf(3, [0.5, 0.0, 0.0, 0.5]),
            wl.Table(0, np.array([1431655765, 2863311530, 0xFFFFFFFF], dtype=np.uint32))]
    for tab in tabs:
        us = list(rng.integers(0, 2 ** 32, size=300)) + [0, 2 ** 32 - 1]
        us += [int(x) for x in tab.cdf[:5]] + [max(int(x) - 1, 0) for x in tab.cdf[:5]]
        for u in us:
            assert orc.sample(tab, int(u)) == sample_py(tab, int(u))


def test_sample_threshold_semantics():
    # thresholds 2^31 and 3*2^30: u < cdf[0] -> vmin; cdf[0] <= u < cdf[1] -> vmin+1; else catch-all
    tab = wl.Table(10, np.array([2 ** 31, 3 * 2 ** 30, 0], dtype=np.uint32))
    assert orc.sample(tab, 0) == 10
    assert orc.sample(tab, 2 ** 31 - 1) == 10
    assert orc.sample(tab, 2 ** 31) == 11
    assert orc.sample(tab, 3 * 2 ** 30 - 1) == 11
    assert orc.sample(tab, 3 * 2 ** 30) == 12
    assert orc.sample(tab, 2 ** 32 - 1) == 12   # last entry is a catch-all whatever its value


def test_tables_realise_their_laws():
    # quantised tables reproduce the intended moments (input generator sanity, fp64)
    m, _ = wl.table_moments(wl.poisson_table(2.0))
    assert abs(m - 2.0) < 1e-6
    m, _ = wl.table_moments(wl.uniform_table(16, 128))
    assert abs(m - 72.0) < 1e-6
    m, _ = wl.table_moments(wl.geometric_table(64.0, 512))
    p = 1 / 64.0
    expect = (1 - (1 - p) ** 512) / p   # E[min(G, 512)] for a geometric law on {1,2,..}
    assert abs(m - expect) < 1e-5
    v, pm = wl.table_pmf(wl.pareto_table(1.5, 16.0, 16, 8192))
    assert v[0] == 16 and v[-1] == 8192 and abs(pm.sum() - 1) < 1e-12
    assert abs(pm[-1] - (16 / 8191.5) ** 1.5) < 1e-8


def test_drawn_counts_follow_the_arrival_law():
    # the n_t sequence logged by the checker is the table applied to word 0 of the step stream
    cfg = wl.config1(replicas=2, T=400)
    out = orc.run(cfg, arrlog=True)
    key = (cfg.seed & 0xFFFFFFFF, cfg.seed >> 32)
    for r in range(2):
        for t in range(1, 401):
            w = philox_py((t, r, 0, 0), key)
            assert out["arrlog"][r, t - 1] == sample_py(cfg.arrivals[0].count[0], w[0])
    big = orc.run(wl.config1(replicas=64, T=2000), arrlog=True, trace=False, hist=False, complog=False)
    assert abs(big["arrlog"].mean() - 0.5) < 0.01
