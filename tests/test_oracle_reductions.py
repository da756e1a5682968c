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


def test_alpha_protection_with_full_limit_and_no_overflow_is_greedy():
    # Section 4.1 baseline: with alpha = 0 the admission rule is the capacity itself; while no slot overflows
    # the evict-all rule never fires and the policy coincides with greedy
    cfg = wl.config6(replicas=3, T=2500)
    n = 3
    alpha0 = cfg.with_(groups=(wl.Group(wl.POLICY_ALPHA, n_replicas=n, m_admit=cfg.M),))
    greedy = cfg.with_(groups=(wl.Group(wl.POLICY_GREEDY, n_replicas=n),))
    a, g = orc.run(alpha0), orc.run(greedy)
    assert a["counters"][:, I["overflow_steps"]].sum() == 0
    _same(a, g)


def test_alpha_protection_evicts_everything_on_overflow():
    # overloaded single class: whenever a slot overflows, the active set is emptied (usage 0 in that slot)
    cfg = wl.config1(replicas=3, T=1500)
    cfg = cfg.with_(groups=(wl.Group(wl.POLICY_ALPHA, n_replicas=3, m_admit=cfg.M - 64),))
    out = orc.run(cfg, admlog_cap=0)
    c = out["counters"]
    assert c[:, I["overflow_steps"]].min() > 0
    # evictions per overflow slot = the whole active set, so evictions >> overflow slots
    assert (c[:, I["evictions"]] > 3 * c[:, I["overflow_steps"]]).all()
    zero_slots = (out["trace"][:, :, 0] == 0).sum(axis=1)
    assert (zero_slots >= c[:, I["overflow_steps"]]).all()
    # admission never takes the usage of an admission slot past the protection limit + growth of that slot:
    # max_U can exceed m_admit only through decoding growth, never beyond M
    assert (c[:, I["max_U"]] <= cfg.M).all()


def test_mc_benchmark_never_overflows_and_equals_greedy_when_memory_is_ample():
    # Section 4.1's MC benchmark admits only what provably fits until completion: no slot can overflow, so
    # nothing is ever evicted, whatever the load
    for cfg in (wl.config1(replicas=3, T=2500), wl.config5(replicas=2, T=4000).with_(trace_stride=1)):
        n = cfg.groups[0].n_replicas
        for worst in (0, 1):
            mc = cfg.with_(groups=(wl.Group(wl.POLICY_MC, n_replicas=n, mc_worst_case=worst),))
            c = orc.run(mc, complog=False)["counters"]
            assert c[:, I["evictions"]].sum() == 0 and c[:, I["overflow_steps"]].sum() == 0
            assert (c[:, I["max_U"]] <= cfg.M).all() and c[:, I["completed"]].min() > 0
    # with ample memory the projection never refuses and the policy is plain greedy
    roomy = wl.config1(replicas=3, T=1500).with_(M=1 << 24)
    mc = roomy.with_(groups=(wl.Group(wl.POLICY_MC, n_replicas=3),))
    gr = roomy.with_(groups=(wl.Group(wl.POLICY_GREEDY, n_replicas=3),))
    _same(orc.run(mc), orc.run(gr))


def test_mc_worst_case_projection_equals_known_lengths_when_lengths_are_constant():
    # the unknown-length adaptation projects with the longest output of the class; with one possible length it
    # is the known-length rule, and with variable lengths it is more conservative (never more admissions)
    cfg = wl.config6(replicas=2, T=2500).with_(M=2000)
    known = cfg.with_(groups=(wl.Group(wl.POLICY_MC, n_replicas=2, mc_worst_case=0),))
    worst = cfg.with_(groups=(wl.Group(wl.POLICY_MC, n_replicas=2, mc_worst_case=1),))
    _same(orc.run(known), orc.run(worst))
    var = wl.config1(replicas=3, T=2500)
    k = orc.run(var.with_(groups=(wl.Group(wl.POLICY_MC, n_replicas=3, mc_worst_case=0),)), complog=False)
    w = orc.run(var.with_(groups=(wl.Group(wl.POLICY_MC, n_replicas=3, mc_worst_case=1),)), complog=False)
    assert (w["counters"][:, I["sum_U"]] < k["counters"][:, I["sum_U"]]).all()


def test_mc_last_slot_shortcut_agrees_with_the_slot_by_slot_test_on_every_decision():
    # Section 4.1: a request starts only if the usage of EVERY future slot stays within M.  The checker sums
    # every future slot (mode 0); its opt-in shortcut looks at the requests' last slots only (mode 1).  Mode 2
    # evaluates both on every admission test and fails on the first disagreement.
    tests = 0
    for seed in range(40):
        cfg = wl.random_medium_config(seed)
        if not any(g.policy == wl.POLICY_MC for g in cfg.groups):
            continue
        both = orc.run(cfg, mc_mode=2, threads=2, trace=False, complog=False)
        tests += int(both["n_mc_tests"].sum())
    for seed in range(60):
        cfg = wl.random_small_config(seed, n_replicas=3, T=97)
        tests += int(orc.run(cfg, mc_mode=2)["n_mc_tests"].sum())
    cfg = wl.config6(replicas=1, T=1500)
    for rate in (5.0, 15.0):
        c6 = wl.config6(replicas=1, T=1500, total_rate=rate)
        both = orc.run(c6, mc_mode=2)
        tests += int(both["n_mc_tests"].sum())
        fast = orc.run(c6, mc_mode=1)
        for k in ("counters", "trace", "hist"):
            assert (both[k] == fast[k]).all()
    assert tests > 100000, tests
