"""The checker against hand-evaluated instances of the model (tests/golden/trace_*.txt)."""
import os

import numpy as np
import pytest

from helpers import degenerate_config, read_fixture, trace_fixtures
from oracle import fcsim_oracle as orc
from pyref import brute_force

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


@pytest.mark.parametrize("name", trace_fixtures(GOLDEN))
def test_hand_trace(name):
    fx = read_fixture(os.path.join(GOLDEN, name))
    cfg = degenerate_config(**fx["params"])
    out = orc.run(cfg)
    T = fx["params"]["T"]
    assert out["trace"][0, :, 0].tolist() == fx["U"]
    assert out["trace"][0, :, 1].tolist() == fx["Q"]
    n = int(out["counters"][0, orc.CIDX["n_logged"]])
    assert [tuple(x) for x in out["complog"][0, :n].tolist()] == fx["completions"]
    assert int(out["counters"][0, orc.CIDX["completed"]]) == len(fx["completions"])
    for k, v in fx["counters"].items():
        assert int(out["counters"][0, orc.CIDX[k]]) == v, k
    # latency histogram (shift 0): one count per completion in bin min(lat, bins-1)
    hist = np.zeros(cfg.hist_bins, dtype=np.int64)
    for _, lat in fx["completions"]:
        hist[min(lat, cfg.hist_bins - 1)] += 1
    assert out["hist"][0].tolist() == hist.tolist()
    # the independent Python evaluator agrees with the hand values as well
    bf = brute_force(cfg, 0, T)
    assert bf["U"] == fx["U"] and bf["Q"] == fx["Q"] and bf["completions"] == fx["completions"]


def test_workload_constant_of_the_steady_state():
    # l*o + o(o+1)/2 for (l, o) = (2, 3): the per-request workload of the proof of Prop. 3.2
    fx = read_fixture(os.path.join(GOLDEN, "trace_roomy.txt"))
    assert fx["U"][-1] == 2 * 3 + 3 * 4 // 2 == sum(2 + j for j in (1, 2, 3))


def test_latency_of_an_unqueued_request_is_its_decode_length():
    cfg = degenerate_config(n=1, l=7, o=5, policy="flow", b=1, K=0, c=0, M=10 ** 6, T=40)
    out = orc.run(cfg)
    n = int(out["counters"][0, orc.CIDX["n_logged"]])
    assert n == 36
    assert set(out["complog"][0, :n, 1].tolist()) == {5}
    assert int(out["counters"][0, orc.CIDX["sum_w_completed"]]) == 36 * (7 * 5 + 15)
