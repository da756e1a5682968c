"""Special cases in which two different settings of the checker must coincide exactly."""
import numpy as np
import pytest

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl

I = orc.CIDX
# counters that describe the trajectory itself (blocked-step bookkeeping differs by construction)
TRAJ = [n for n in orc.COUNTER_NAMES if n not in ("status",)]


def _same(a, b, skip=()):
    for k in ("trace", "hist", "complog"):
        if a[k] is not None:
            assert (a[k] == b[k]).all(), k
    for n in TRAJ:
        if n not in skip:
            assert (a["counters"][:, I[n]] == b["counters"][:, I[n]]).all(), n


@pytest.mark.parametrize("maker", [lambda: wl.config1(replicas=4, T=1500),
                                   lambda: wl.config5(replicas=2, T=3000).with_(trace_stride=1)],
                         ids=["cfg1", "cfg5"])
def test_large_b_is_greedy(maker):
    # Section 3.3: as b grows the flow-controlled policy degenerates to greedy with LIFO eviction
    cfg = maker()
    n = cfg.groups[0].n_replicas
    flow = cfg.with_(groups=(wl.Group(wl.POLICY_FLOW, b_fp=0xFFFF0000, n_replicas=n),))
    greedy = cfg.with_(groups=(wl.Group(wl.POLICY_GREEDY, n_replicas=n),))
    _same(orc.run(flow), orc.run(greedy))


def test_chunk_at_least_max_prompt_without_budget_is_greedy():
    cfg = wl.config1(replicas=4, T=1500).with_(K=0)
    n = 4
    chunked = cfg.with_(groups=(wl.Group(wl.POLICY_CHUNKED, chunk=128, n_replicas=n),))
    greedy = cfg.with_(groups=(wl.Group(wl.POLICY_GREEDY, n_replicas=n),))
    _same(orc.run(chunked), orc.run(greedy))


def test_trajectories_do_not_depend_on_grouping_or_placement():
    cfg = wl.config1(replicas=6, T=800)
    whole = orc.run(cfg)
    split = cfg.with_(groups=(wl.Group(wl.POLICY_FLOW, b_fp=0xC000, rng_replica_base=4, n_replicas=2),
                              wl.Group(wl.POLICY_FLOW, b_fp=0xC000, rng_replica_base=0, n_replicas=4)))
    parts = orc.run(split)
    order = [4, 5, 0, 1, 2, 3]
    for k in ("counters", "trace", "hist", "complog"):
        assert (parts[k] == whole[k][order]).all()
    # a sub-range of replicas computed alone equals the same rows of the full run
    sub = orc.run(cfg, first_replica=2, n_replicas=3)
    for k in ("counters", "trace", "hist", "complog"):
        assert (sub[k] == whole[k][2:5]).all()
    # threads only split the replica range
    thr = orc.run(cfg, threads=3)
    for k in ("counters", "trace", "hist", "complog"):
        assert (thr[k] == whole[k]).all()


def test_replicas_differ_and_seeds_matter():
    cfg = wl.config1(replicas=4, T=500)
    a = orc.run(cfg)
    assert len({tuple(r) for r in a["counters"][:, [I["arrived"], I["sum_U"]]].tolist()}) == 4
    b = orc.run(cfg.with_(seed=1))
    assert (a["counters"][:, I["sum_U"]] != b["counters"][:, I["sum_U"]]).any()
    hi = orc.run(cfg.with_(seed=1 << 32))     # the high key word is used too
    assert (a["counters"][:, I["sum_U"]] != hi["counters"][:, I["sum_U"]]).any()


def test_zero_flow_rate_admits_nothing_and_fractional_rate_has_the_right_mean():
    cfg = wl.config1(replicas=8, T=3000)
    z = orc.run(cfg.with_(groups=(wl.Group(wl.POLICY_FLOW, b_fp=0, n_replicas=8),)))
    assert z["counters"][:, I["admitted"]].sum() == 0
    # b = 0.25 with a standing queue and no memory/budget limit: admissions/T -> b (E[B_t] = b, Thm. 3.6)
    roomy = cfg.with_(M=2 ** 30, K=0, Qcap=2 ** 31 - 1, Acap=1 << 20,
                      groups=(wl.Group(wl.POLICY_FLOW, b_fp=0x4000, n_replicas=8),))
    out = orc.run(roomy, complog=False, hist=False)
    rate = out["counters"][:, I["admitted"]].sum() / (8 * 3000)
    assert abs(rate - 0.25) < 0.01
    assert out["counters"][:, I["q_final"]].min() > 100   # lambda = 0.5 > b: the queue stands
