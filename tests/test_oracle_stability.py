"""The stability dichotomy (Prop. 3.5 and Thm. 3.6) observed on long runs of the checker."""
import numpy as np

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl

I = orc.CIDX


def _cfg(rho, beta, T, reps=6):
    """Single-class workload with E[w] ~ 8.7e3 at M = 32768; arrival rate rho*M/E[w], flow rate beta*M/E[w]."""
    base = wl.config1(replicas=reps, T=T).with_(M=32768, K=0, Qcap=2 ** 31 - 1, Acap=4096, trace_stride=0,
                                                 hist_bins=0, complog_cap=0)
    ew = wl.mean_workload(base)
    lam = rho * base.M / ew
    cfg = base.with_(arrivals=(wl.Arrivals((wl.poisson_table(lam),)),),
                     groups=(wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(beta * base.M / ew), n_replicas=reps),))
    return cfg, ew, lam


def test_overloaded_system_backlog_grows_linearly():
    # Prop. 3.5: lambda E[w] > M  =>  unfinished requests / T >= delta / w_max > 0, whatever the policy
    for beta in (0.9, 4.0):
        T = 20000
        cfg, ew, lam = _cfg(1.3, beta, T)
        out = orc.run(cfg, threads=6)
        backlog = (out["counters"][:, I["q_final"]] + out["counters"][:, I["p_final"]]).mean() / T
        delta = lam * ew - cfg.M
        C = 512
        w_max = 1.5 * C * C + 0.5 * C
        assert delta > 0 and backlog >= delta / w_max
        # and it keeps growing: doubling the horizon roughly doubles the backlog
        out2 = orc.run(cfg.with_(T_max=2 * T), threads=6)
        b2 = (out2["counters"][:, I["q_final"]] + out2["counters"][:, I["p_final"]]).mean()
        assert b2 > 1.6 * backlog * T


def test_underloaded_flow_control_stays_bounded_without_overflow():
    # Thm. 3.6 regime: b > lambda and b E[w] <= (1-eps) M: bounded queue, (almost) no overflow
    T = 20000
    cfg, ew, lam = _cfg(0.6, 0.8, T)
    assert cfg.groups[0].b_fp / 65536 > lam
    out = orc.run(cfg, threads=6)
    out2 = orc.run(cfg.with_(T_max=2 * T), threads=6)
    assert out2["counters"][:, I["max_Q"]].max() <= 2 * max(out["counters"][:, I["max_Q"]].max(), 8)
    assert out2["counters"][:, I["max_Q"]].max() < 60
    assert out2["counters"][:, I["overflow_steps"]].sum() == 0
    assert out2["counters"][:, I["dropped"]].sum() == 0
    # Little's law in its long-run form: mean number in system ~ arrival rate x mean latency
    c = out2["counters"].sum(axis=0).astype(np.float64)
    L = c[I["sum_N"]] / (cfg.n_replicas * 2 * T)
    W = c[I["sum_lat"]] / c[I["completed"]]
    assert abs(L - lam * W) / L < 0.02


def test_overflow_count_respects_the_bound_of_theorem_3_6():
    # Thm. 3.6: b E[w] <= (1 - eps) M, B_t <= A, lengths <= C  =>  E[#overflow slots] < T exp(-eps^2 M^2 / (2 (A^2+A) C^3)).
    # The bound is loose at these sizes (close to T); the slots in which memory binds (an eviction, or an
    # activation refused by the headroom gate) must stay below it -- here they are in fact zero.
    import math
    T = 20000
    cfg, ew, lam = _cfg(0.6, 0.8, T)
    b = cfg.groups[0].b_fp / 65536.0
    eps = 1.0 - b * ew / cfg.M
    assert eps > 0.19
    A = int(b) + 1
    C = 512
    bound = T * math.exp(-(eps * cfg.M) ** 2 / (2.0 * (A * A + A) * C ** 3))
    out = orc.run(cfg, threads=6)
    binding = (out["counters"][:, I["overflow_steps"]] + out["counters"][:, I["gate_blocked_steps"]]).mean()
    assert binding < bound
    assert binding == 0
