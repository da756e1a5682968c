"""Closed forms from the paper's proofs that the checker must reproduce exactly."""
import numpy as np
import pytest

from helpers import degenerate_config
from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl

I = orc.CIDX
BIG = 2 ** 30


def roomy(cfg, b, **kw):
    """Nothing binds: huge M and queue, no token budget, integer flow rate b."""
    return cfg.with_(M=BIG, K=0, Qcap=2 ** 31 - 1, Acap=1 << 20,
                     groups=(wl.Group(wl.POLICY_FLOW, b_fp=b << 16, n_replicas=cfg.n_replicas),), **kw)


def test_waiting_queue_follows_the_lindley_recursion():
    # proof of Thm. 3.3: Q_t = (Q_{t-1} + n_t - b)^+ when memory never binds
    for lam, b in ((1.6, 2), (2.2, 2), (0.7, 1)):
        base = wl.config2(replicas=3, T=3000)
        cfg = roomy(base, b, arrivals=(wl.Arrivals((wl.poisson_table(lam),)),))
        out = orc.run(cfg, arrlog=True, hist=False, complog=False)
        for r in range(3):
            q = 0
            expect = []
            for n_t in out["arrlog"][r]:
                q = max(q + int(n_t) - b, 0)
                expect.append(q)
            assert out["trace"][r, :, 1].tolist() == expect
        assert out["counters"][:, I["evictions"]].sum() == 0
        assert out["counters"][:, I["dropped"]].sum() == 0


def test_usage_is_the_double_sum_over_the_admission_log():
    # proof of Thm. 3.6: U_t = sum_s sum_p (l_{s,p} + (t-s+1)) 1(o_{s,p} >= t-s+1) while nothing is evicted
    base = wl.config1(replicas=3, T=700)
    cfg = roomy(base, 1)
    out = orc.run(cfg, admlog_cap=4096, hist=False, complog=False)
    assert out["counters"][:, I["evictions"]].sum() == 0
    T = cfg.T_max
    for r in range(3):
        n = int(out["n_admlog"][r])
        assert n == out["counters"][r, I["admitted"]] and n < 4096
        U = np.zeros(T + 2, dtype=np.int64)
        for s, l, o, _ in out["admlog"][r, :n]:
            for q in range(1, o + 1):
                t = s + q - 1
                if t <= T:
                    U[t] += l + q
        assert out["trace"][r, :, 0].tolist() == U[1:T + 1].tolist()


def test_saturated_single_class_usage_equals_b_times_w():
    # equality case of the bound in the proof of Thm. 3.3: b activations of (l, o) every slot
    for l, o, b in ((10, 20, 4), (10, 60, 4), (3, 7, 2)):
        cfg = degenerate_config(n=b, l=l, o=o, policy="flow", b=b, K=0, c=0, M=BIG, T=3 * o, Qcap=1024, Acap=1024)
        out = orc.run(cfg)
        w = l * o + o * (o + 1) // 2
        assert (out["trace"][0, o - 1:, 0] == b * w).all()
        assert (out["trace"][0, :o - 1, 0] < b * w).all()


def test_section_4_1_parameters_satisfy_the_sufficient_condition():
    # Section 4.1: classes (10,20),(10,40),(10,60), b = (4,4,4): sum_k b_k w_k = 16240 < M = 16492 (Eq. 2);
    # the checker's saturated per-class usages add up to that number
    total = 0
    for o in (20, 40, 60):
        cfg = degenerate_config(n=4, l=10, o=o, policy="flow", b=4, K=0, c=0, M=BIG, T=2 * o, Qcap=1024, Acap=1024)
        total += int(orc.run(cfg)["trace"][0, -1, 0])
    assert total == 16240 < 16492


def test_no_eviction_when_the_flow_rate_keeps_usage_under_capacity():
    # Thm. 3.3 with one class: integer b > lambda and b*w < M  =>  no eviction, gate never binds
    l, o, b = 10, 40, 4
    w = l * o + o * (o + 1) // 2
    cfg = degenerate_config(n=1, l=l, o=o, policy="flow", b=b, K=0, c=0, M=b * w + 1, T=4000, Qcap=4096, Acap=4096,
                            replicas=4)
    cfg = cfg.with_(arrivals=(wl.Arrivals((wl.poisson_table(3.0),)),))
    out = orc.run(cfg, complog=False)
    assert out["counters"][:, I["evictions"]].sum() == 0
    assert out["counters"][:, I["gate_blocked_steps"]].sum() == 0
    assert (out["counters"][:, I["max_U"]] <= b * w).all()


def test_percentile_rule_and_summaries():
    cfg = degenerate_config(n=1, l=2, o=3, policy="flow", b=1, K=0, c=0, M=11, T=12, hist_bins=8)
    out = orc.run(cfg)
    s = orc.summarize(cfg, out["counters"], out["hist"], 12)[0]
    # latencies 3,3,4,4,5,5,6 (hand trace): mean 30/7; p95 -> ceil(.95*7)=7th value = 6; p99 the same
    assert s["mean_latency"] == 30 / 7
    assert s["p95_latency"] == 6.0 and s["p99_latency"] == 6.0
    assert s["request_throughput"] == 7 / 12
    assert s["mean_utilisation"] == sum((3, 7, 9, 8, 7, 9, 8, 7, 9, 8, 7, 9)) / (12 * 11)
    # token throughput: tokens generated per slot (Section 2.2)
    assert s["token_throughput"] == out["counters"][0, I["tokens_generated"]] / 12
    assert s["percentile_source"] == 1


def test_exact_percentiles_from_the_completion_log_differ_from_the_bin_edge():
    # same hand trace with 4-slot histogram bins: latencies 3,3 fall in bin 0 and 4,4,5,5,6 in bin 1, so the
    # histogram rule reports the edge of bin 1, (2 << 2) - 1 = 7, while the 7th smallest latency itself is 6
    cfg = degenerate_config(n=1, l=2, o=3, policy="flow", b=1, K=0, c=0, M=11, T=12, hist_bins=8).with_(hist_shift=2)
    out = orc.run(cfg)
    assert out["complog"][0, :7, 1].tolist() == [3, 3, 4, 4, 5, 5, 6]
    by_hist = orc.summarize(cfg, out["counters"], out["hist"], 12)[0]
    exact = orc.summarize(cfg, out["counters"], out["hist"], 12, out["complog"])[0]
    assert by_hist["p95_latency"] == 7.0 and by_hist["percentile_source"] == 1
    assert exact["p95_latency"] == 6.0 and exact["p99_latency"] == 6.0 and exact["percentile_source"] == 2
    # rank rule ceil(q n / 100), 1-based: 100 distinct values -> the 95th and 99th; 101 values -> ranks 96 and 100
    rng = np.random.default_rng(0)
    assert orc.percentile_from_latencies(rng.permutation(np.arange(1, 101)), 95) == 95.0
    assert orc.percentile_from_latencies(rng.permutation(np.arange(1, 101)), 99) == 99.0
    assert orc.percentile_from_latencies(rng.permutation(np.arange(1, 102)), 95) == 96.0
    assert orc.percentile_from_latencies(rng.permutation(np.arange(1, 102)), 99) == 100.0
    assert orc.percentile_from_latencies([7], 95) == 7.0 and orc.percentile_from_latencies([], 95) == 0.0
    # a log that overflowed cannot give the order statistics: the histogram rule is used and reported
    small = cfg.with_(complog_cap=3)
    o2 = orc.run(small)
    s2 = orc.summarize(small, o2["counters"], o2["hist"], 12, o2["complog"])[0]
    assert s2["percentile_source"] == 1 and s2["p95_latency"] == 7.0


# ---------------------------------------------------------------- Algorithm 1 (per-class budgets, known lengths)
def _paper_classes(T, lam, b=(4, 4, 4), M=16492, replicas=3, Qcap=2 ** 31 - 1):
    cfg = wl.config6(replicas=replicas, T=T)
    return cfg.with_(M=M, Qcap=Qcap, Acap=4096, arrivals=(wl.Arrivals((wl.poisson_table(lam),)),),
                     groups=(wl.Group(wl.POLICY_CLASSFLOW, n_replicas=replicas, b_class=tuple(b)),))


def test_algorithm1_section_4_1_never_exceeds_the_bound_of_theorem_3_3():
    # Section 4.1: (l,o) = (10,20),(10,40),(10,60), b = (4,4,4): usage <= sum_k b_k w_k = 16240 < M = 16492
    # in every slot, so no eviction ever happens and the gate never binds (proof of Thm. 3.3)
    cfg = _paper_classes(T=6000, lam=5.0)
    out = orc.run(cfg)
    c = out["counters"]
    assert (c[:, I["max_U"]] <= 16240).all()
    assert c[:, I["evictions"]].sum() == 0 and c[:, I["gate_blocked_steps"]].sum() == 0
    assert c[:, I["completed"]].min() > 25000
    # integer b_k > lambda_k = 5/3: queues are positive recurrent -- short and bounded
    assert c[:, I["max_Q"]].max() < 40


def test_algorithm1_saturated_usage_equals_sum_b_k_w_k():
    # with at least b_k waiting requests of every class in every slot the bound is attained exactly
    cfg = _paper_classes(T=400, lam=60.0)
    out = orc.run(cfg, complog=False, hist=False)
    assert (out["trace"][:, 80:, 0] == 16240).all()
    assert (out["trace"][:, :59, 0] < 16240).all()


def test_algorithm1_per_class_queues_follow_the_lindley_recursion():
    # proof of Thm. 3.3: Q_{t,k} = (Q_{t-1,k} + n_{t,k} - b_k)^+, independently for every class
    cfg = _paper_classes(T=3000, lam=5.5, b=(2, 2, 1), M=2 ** 30)
    out = orc.run(cfg, arrcls=True, complog=False, hist=False)
    assert out["counters"][:, I["evictions"]].sum() == 0
    for r in range(cfg.n_replicas):
        q = np.zeros(3, dtype=np.int64)
        expect = []
        for n_tk in out["arrcls"][r]:
            q = np.maximum(q + n_tk - np.array([2, 2, 1]), 0)
            expect.append(int(q.sum()))
        assert out["trace"][r, :, 1].tolist() == expect
        assert (out["arrcls"][r].sum(axis=1) >= 0).all()
    # class 3 has b_3 = 1 < lambda_3: its queue grows, the others stay short
    assert out["trace"][:, -1, 1].min() > 1000


def test_algorithm1_with_one_class_is_algorithm2_with_integer_budget():
    base = wl.config1(replicas=4, T=1500)
    for b in (1, 2):
        one = base.with_(groups=(wl.Group(wl.POLICY_CLASSFLOW, n_replicas=4, b_class=(b,)),))
        flow = base.with_(groups=(wl.Group(wl.POLICY_FLOW, b_fp=b << 16, n_replicas=4),))
        a, f = orc.run(one), orc.run(flow)
        for k in ("trace", "hist", "complog"):
            assert (a[k] == f[k]).all()
        assert (a["counters"] == f["counters"]).all()
