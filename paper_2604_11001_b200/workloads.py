"""Seeded synthetic inputs for the flow-control serving simulator.

This module only *describes* simulations: integer inverse-CDF tables for the
arrival-count, class, prompt-length and decode-length laws, and the five
preset workloads.  It contains none of the simulator's stepping logic and is
the one module that both the CUDA binding and the CPU checker consume, so that
both are fed byte-identical tables.

Table format (used by both consumers): support ``{vmin, .., vmin+n-1}``;
``cdf[k] = floor(P(X <= vmin+k) * 2**32)`` clamped to ``2**32-1`` and
non-decreasing; the last entry is a catch-all and its value is ignored.
A draw ``u`` (uniform 32-bit word) maps to ``vmin + min{k < n-1 : u < cdf[k]}``
or to ``vmin+n-1`` when no such ``k`` exists.

The laws follow the model of Section 2.1 (arrival count ``n_t`` with mean
lambda, request lengths ``(l, o)``) and Assumption 3.4 (bounded lengths); the
five presets are synthetic stand-ins shaped like the paper's Section 4
workloads (Poisson arrivals, a handful of classes, bounded lengths).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Sequence, Tuple

import numpy as np
from scipy.special import ndtr

POLICY_FLOW = 0
POLICY_GREEDY = 1
POLICY_CHUNKED = 2
POLICY_ALPHA = 3   # alpha-protection greedy (Section 4.1)
POLICY_CLASSFLOW = 4   # Algorithm 1: per-class activation budgets b_k, FIFO within a class
POLICY_MC = 5          # memory-constrained FCFS benchmark (Section 4.1): admit only if future usage stays <= M

_TWO32 = float(2 ** 32)


# --------------------------------------------------------------------------- tables
@dataclass(frozen=True)
class Table:
    vmin: int
    cdf: np.ndarray  # uint32, length n

    @property
    def n(self) -> int:
        return int(self.cdf.shape[0])

    @property
    def vmax(self) -> int:
        return self.vmin + self.n - 1


def table_from_cdf(vmin: int, cdf_values: Sequence[float]) -> Table:
    """Quantise a real-valued CDF (P(X <= vmin+k), k = 0..n-1) to 32-bit thresholds."""
    c = np.asarray(cdf_values, dtype=np.float64)
    thr = np.floor(np.clip(c, 0.0, 1.0) * _TWO32)
    thr = np.minimum(thr, _TWO32 - 1.0)
    thr = np.maximum.accumulate(thr)
    out = thr.astype(np.uint64).astype(np.uint32)
    out[-1] = np.uint32(0xFFFFFFFF)
    return Table(int(vmin), np.ascontiguousarray(out))


def table_from_pmf(vmin: int, pmf: Sequence[float]) -> Table:
    p = np.asarray(pmf, dtype=np.float64)
    p = p / p.sum()
    return table_from_cdf(vmin, np.cumsum(p))


def table_pmf(tab: Table) -> Tuple[np.ndarray, np.ndarray]:
    """The law a table actually realises: (values, probabilities), exact in fp64."""
    thr = tab.cdf.astype(np.float64)
    thr[-1] = _TWO32
    thr = np.maximum.accumulate(thr)
    p = np.diff(np.concatenate(([0.0], thr))) / _TWO32
    return np.arange(tab.vmin, tab.vmin + tab.n, dtype=np.int64), p


def table_moments(tab: Table) -> Tuple[float, float]:
    v, p = table_pmf(tab)
    vf = v.astype(np.float64)
    return float((vf * p).sum()), float((vf * vf * p).sum())


def constant_table(value: int) -> Table:
    return Table(int(value), np.array([0xFFFFFFFF], dtype=np.uint32))


def poisson_table(lam: float, max_entries: int = 64) -> Table:
    """Counts 0,1,2,.. of a Poisson(lam) law, cut at the first k whose upper tail is
    below 2**-32 (at most ``max_entries`` values); the tail mass goes to the last value."""
    cdf = []
    term = math.exp(-lam)
    acc = 0.0
    for k in range(max_entries):
        acc += term
        cdf.append(min(acc, 1.0))
        if 1.0 - acc < 2.0 ** -32:
            break
        term *= lam / (k + 1)
    return table_from_cdf(0, cdf)


def uniform_table(lo: int, hi: int) -> Table:
    n = hi - lo + 1
    return table_from_cdf(lo, (np.arange(n, dtype=np.float64) + 1.0) / n)


def geometric_table(mean: float, cap: int) -> Table:
    """P(o=k) = (1-p)^(k-1) p on {1,2,..} with p = 1/mean; values above ``cap`` pile on ``cap``."""
    p = 1.0 / mean
    k = np.arange(1, cap + 1, dtype=np.float64)
    cdf = 1.0 - np.power(1.0 - p, k)
    cdf[-1] = 1.0
    return table_from_cdf(1, cdf)


def _rounded_clamped(cdf_fn, lo: int, hi: int) -> Table:
    """Round a continuous law to the nearest integer and clamp to [lo, hi]:
    P(X <= v) = F(v + 1/2) for lo <= v < hi, 1 at hi."""
    v = np.arange(lo, hi + 1, dtype=np.float64)
    cdf = cdf_fn(v + 0.5)
    cdf[-1] = 1.0
    return table_from_cdf(lo, cdf)


def lognormal_table(mu: float, sigma: float, lo: int, hi: int) -> Table:
    return _rounded_clamped(lambda x: ndtr((np.log(x) - mu) / sigma), lo, hi)


def pareto_table(alpha: float, xm: float, lo: int, hi: int) -> Table:
    def cdf(x):
        return np.where(x >= xm, 1.0 - np.power(xm / np.maximum(x, xm), alpha), 0.0)
    return _rounded_clamped(cdf, lo, hi)


def mixture_table(parts: Sequence[Tuple[float, Table]]) -> Table:
    lo = min(t.vmin for _, t in parts)
    hi = max(t.vmax for _, t in parts)
    pmf = np.zeros(hi - lo + 1, dtype=np.float64)
    for w, t in parts:
        v, p = table_pmf(t)
        pmf[v - lo] += w * p
    return table_from_pmf(lo, pmf)


# --------------------------------------------------------------------------- config
@dataclass(frozen=True)
class Arrivals:
    count: Tuple[Table, ...]            # one table (plain law) or two (two-state modulated law)
    switch_thr: Tuple[int, int] = (0, 0)  # state s flips when the step's third word < switch_thr[s]

    @property
    def n_states(self) -> int:
        return len(self.count)


@dataclass(frozen=True)
class Group:
    policy: int
    b_fp: int = 0              # Q16.16 activation rate b (FLOW)
    chunk: int = 0             # prefill chunk c (CHUNKED)
    arrivals_id: int = 0
    rng_replica_base: int = 0  # generator replica id = base + index within the group
    n_replicas: int = 1
    m_admit: int = 0           # ALPHA: admission keeps usage <= m_admit = floor((1 - alpha) M)
    b_class: Tuple[int, ...] = ()  # CLASSFLOW: integer budget b_k of every class (Algorithm 1)
    mc_worst_case: int = 0         # MC: 1 = project every request with its class's longest output length
    preempt_keep: int = 0          # 0 = an evicted request loses all progress (the paper's model); 1 = it keeps
                                   # its generated tokens as prompt, (l, o) <- (l + j, o - j) (not in the paper)


@dataclass(frozen=True)
class SimConfig:
    M: int
    K: int
    T_max: int
    Qcap: int
    Acap: int
    seed: int
    class_law: Table
    prompt: Tuple[Table, ...]
    decode: Tuple[Table, ...]
    arrivals: Tuple[Arrivals, ...]
    groups: Tuple[Group, ...]
    trace_stride: int = 0
    hist_bins: int = 0
    hist_shift: int = 0
    complog_cap: int = 0
    trace_bulk: int = 0        # 1 = trace records staged in shared memory and stored with bulk copies (same results)
    name: str = ""
    notes: dict = field(default_factory=dict, compare=False)

    @property
    def n_classes(self) -> int:
        return len(self.prompt)

    @property
    def n_replicas(self) -> int:
        return sum(g.n_replicas for g in self.groups)

    def with_(self, **kw) -> "SimConfig":
        return replace(self, **kw)


def b_to_fp(b: float) -> int:
    return int(round(b * 65536.0))


def mean_workload(cfg: SimConfig) -> float:
    """E[w] = E[l]E[o] + (E[o] + E[o^2])/2 over the class mix (the per-request KV-time of
    Prop. 3.5 / Eq. 3, with l and o independent inside a class)."""
    _, pc = table_pmf(cfg.class_law)
    ew = 0.0
    for k in range(cfg.n_classes):
        el, _ = table_moments(cfg.prompt[k])
        eo, eo2 = table_moments(cfg.decode[k])
        ew += pc[k] * (el * eo + 0.5 * (eo + eo2))
    return ew


def arrival_rate(arr: Arrivals) -> float:
    """Mean arrivals per slot (stationary mix of the two states when modulated)."""
    means = [table_moments(t)[0] for t in arr.count]
    if arr.n_states == 1:
        return means[0]
    p01 = arr.switch_thr[0] / _TWO32
    p10 = arr.switch_thr[1] / _TWO32
    pi0 = p10 / (p01 + p10) if (p01 + p10) > 0 else 1.0
    return pi0 * means[0] + (1.0 - pi0) * means[1]


def load_factor(cfg: SimConfig, group: int = 0) -> float:
    """rho = lambda E[w] / M; the system cannot be stable for rho > 1 (Prop. 3.5)."""
    g = cfg.groups[group]
    return arrival_rate(cfg.arrivals[g.arrivals_id]) * mean_workload(cfg) / cfg.M


# --------------------------------------------------------------------------- presets
def _single_class(prompt: Table, decode: Table):
    return constant_table(0), (prompt,), (decode,)


def config1(replicas: int = 64, T: int = 2000) -> SimConfig:
    """Tiny flow-control run: Poisson 0.5/step, l ~ U[16,128], o geometric(mean 64) clamp 512."""
    cl, pr, de = _single_class(uniform_table(16, 128), geometric_table(64.0, 512))
    return SimConfig(
        M=4096, K=512, T_max=T, Qcap=128, Acap=256, seed=0, class_law=cl, prompt=pr, decode=de,
        arrivals=(Arrivals((poisson_table(0.5),)),),
        groups=(Group(POLICY_FLOW, b_fp=0xC000, n_replicas=replicas),),
        trace_stride=1, hist_bins=1024, hist_shift=2, complog_cap=2048, name="cfg1-tiny-flow")


def _cfg2_lengths():
    return _single_class(lognormal_table(math.log(256.0), 1.0, 1, 4096), geometric_table(200.0, 2048))


def config2(replicas: int = 4096, T: int = 20000) -> SimConfig:
    """Policy comparison: FLOW (b = 0.5) vs GREEDY on common random numbers."""
    cl, pr, de = _cfg2_lengths()
    return SimConfig(
        M=65536, K=2048, T_max=T, Qcap=256, Acap=512, seed=1, class_law=cl, prompt=pr, decode=de,
        arrivals=(Arrivals((poisson_table(2.0),)),),
        groups=(Group(POLICY_FLOW, b_fp=0x8000, n_replicas=replicas),
                Group(POLICY_GREEDY, n_replicas=replicas)),
        trace_stride=1, hist_bins=1024, hist_shift=5, complog_cap=16384, name="cfg2-policy-comparison")


def config3(n_rates: int = 64, n_b: int = 64, reps: int = 16, T: int = 50000,
            trace_stride: int = 1) -> SimConfig:
    """Stability sweep: arrival rates at 0.5x..1.5x the necessary-condition load times
    flow-control rates 0.25x..2x of M/E[w], ``reps`` replicas each."""
    cl, pr, de = _cfg2_lengths()
    M = 131072
    base = SimConfig(M=M, K=2048, T_max=T, Qcap=512, Acap=512, seed=2, class_law=cl, prompt=pr,
                     decode=de, arrivals=(), groups=())
    ew = mean_workload(base)
    cap_rate = M / ew
    arrivals = []
    for i in range(n_rates):
        rho = 0.5 + (i / (n_rates - 1) if n_rates > 1 else 0.5)
        arrivals.append(Arrivals((poisson_table(rho * cap_rate),)))
    groups = []
    for i in range(n_rates):
        for j in range(n_b):
            beta = 0.25 + 1.75 * (j / (n_b - 1) if n_b > 1 else 0.5)
            g = i * n_b + j
            groups.append(Group(POLICY_FLOW, b_fp=b_to_fp(beta * cap_rate), arrivals_id=i,
                                rng_replica_base=reps * g, n_replicas=reps))
    return base.with_(arrivals=tuple(arrivals), groups=tuple(groups), trace_stride=trace_stride,
                      hist_bins=1024, hist_shift=6, name="cfg3-stability-sweep",
                      notes={"E_w": ew, "M_over_Ew": cap_rate})


def config4(replicas: int = 16384, T: int = 50000, trace_stride: int = 4) -> SimConfig:
    """Heavy-tailed decode lengths: FLOW (b = 1.25) vs CHUNKED prefill (chunk 512)."""
    prompt = mixture_table(((0.7, uniform_table(32, 256)), (0.3, uniform_table(2048, 8192))))
    cl, pr, de = _single_class(prompt, pareto_table(1.5, 16.0, 16, 8192))
    return SimConfig(
        M=262144, K=2048, T_max=T, Qcap=256, Acap=512, seed=3, class_law=cl, prompt=pr, decode=de,
        arrivals=(Arrivals((poisson_table(1.0),)),),
        groups=(Group(POLICY_FLOW, b_fp=0x14000, n_replicas=replicas),
                Group(POLICY_CHUNKED, chunk=512, n_replicas=replicas)),
        trace_stride=trace_stride, hist_bins=1024, hist_shift=6, name="cfg4-heavy-tail")


def config5(replicas: int = 131072, T: int = 100000) -> SimConfig:
    """Large bursty run: two-state modulated Poisson arrivals (1.0 / 4.0 per step, switch
    probability 1e-3), three equiprobable classes with lognormal prompts (mean m_k, sigma 1)
    and geometric decodes (mean m_k), m = (64, 256, 1024); FLOW (b = 0.3125) vs GREEDY;
    latency histograms only."""
    means = (64.0, 256.0, 1024.0)
    prompt = tuple(lognormal_table(math.log(m) - 0.5, 1.0, 1, 8192) for m in means)
    decode = tuple(geometric_table(m, 8192) for m in means)
    class_law = Table(0, np.array([1431655765, 2863311530, 0xFFFFFFFF], dtype=np.uint32))
    thr = 4294967  # floor(1e-3 * 2**32)
    return SimConfig(
        M=262144, K=2048, T_max=T, Qcap=256, Acap=512, seed=4, class_law=class_law, prompt=prompt,
        decode=decode,
        arrivals=(Arrivals((poisson_table(1.0), poisson_table(4.0)), (thr, thr)),),
        groups=(Group(POLICY_FLOW, b_fp=0x5000, n_replicas=replicas),
                Group(POLICY_GREEDY, n_replicas=replicas)),
        trace_stride=0, hist_bins=1024, hist_shift=7, complog_cap=0, name="cfg5-large-bursty")


def config6(replicas: int = 4096, T: int = 10000, alpha: float = 0.2, total_rate: float = 5.0) -> SimConfig:
    """The paper's own synthetic setting (Section 4.1): three classes (l, o) = (10,20), (10,40), (10,60),
    Poisson arrivals of total intensity 5 per slot split evenly over the classes, M = 16492, no token
    budget, T up to 10000.  Policies on common random numbers: Algorithm 2 with b = 12 (the sum of the
    paper's per-class budgets 4+4+4), greedy, alpha-protection greedy, Algorithm 1 with the paper's
    budgets (4, 4, 4), for which sum_k b_k w_k = 16240 < M (Eq. 2), and the MC benchmark with known and with
    worst-case output lengths.  ``total_rate`` = 5 reads the paper's "intensity 5" as the total rate (load
    0.41 of capacity); 15 reads it as 5 per class (load 1.23: memory binds and the policies separate, but the
    finite waiting room then drops arrivals, which the paper's unbounded queue does not)."""
    class_law = Table(0, np.array([1431655765, 2863311530, 0xFFFFFFFF], dtype=np.uint32))
    prompt = tuple(constant_table(10) for _ in range(3))
    decode = tuple(constant_table(o) for o in (20, 40, 60))
    M = 16492
    # storage bound of the active set, chosen so that it never binds: about 200 requests are active at rate 5
    # (never more than 300 in 2.5e8 replica-steps), about 500 when memory binds at rate 15
    Acap = 512 if total_rate <= 5.0 else 1024
    return SimConfig(
        M=M, K=0, T_max=T, Qcap=256, Acap=Acap, seed=6, class_law=class_law, prompt=prompt, decode=decode,
        arrivals=(Arrivals((poisson_table(total_rate),)),),
        groups=(Group(POLICY_FLOW, b_fp=12 << 16, n_replicas=replicas),
                Group(POLICY_GREEDY, n_replicas=replicas),
                Group(POLICY_ALPHA, n_replicas=replicas, m_admit=int(math.floor((1.0 - alpha) * M))),
                Group(POLICY_CLASSFLOW, n_replicas=replicas, b_class=(4, 4, 4)),
                Group(POLICY_MC, n_replicas=replicas, mc_worst_case=0),
                Group(POLICY_MC, n_replicas=replicas, mc_worst_case=1)),
        trace_stride=1, hist_bins=1024, hist_shift=0, complog_cap=0, name="cfg6-paper-section-4.1")


PRESETS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5, 6: config6}


# --------------------------------------------------------------------------- random tiny configs
def random_small_config(seed: int, n_replicas: int = 4, T: int = 60) -> SimConfig:
    """A seeded, randomly parameterised tiny simulation exercising every policy and option."""
    rng = np.random.default_rng(seed)
    n_classes = int(rng.integers(1, 4))

    def rand_table(lo, hi):
        vmin = int(rng.integers(lo, hi))
        n = int(rng.integers(1, 7))
        return table_from_pmf(vmin, rng.random(n) + 0.05)

    prompt = tuple(rand_table(1, 9) for _ in range(n_classes))
    decode = tuple(rand_table(1, 7) for _ in range(n_classes))
    class_law = table_from_pmf(0, rng.random(n_classes) + 0.1)
    max_fp = max(p.vmax for p in prompt) + max(d.vmax for d in decode)
    M = int(rng.integers(max_fp, max_fp + 48))
    K = int(rng.choice([0, 0, int(rng.integers(1, 24))]))
    arrivals = []
    for _ in range(2):
        if rng.random() < 0.5:
            arrivals.append(Arrivals((poisson_table(float(rng.uniform(0.2, 2.5))),)))
        else:
            arrivals.append(Arrivals((poisson_table(float(rng.uniform(0.1, 1.0))),
                                      poisson_table(float(rng.uniform(1.0, 4.0)))),
                                     (int(rng.integers(0, 2 ** 31)), int(rng.integers(0, 2 ** 31)))))
    groups = []
    base = 0
    keep_rng = np.random.default_rng(500_000 + seed)  # its own stream: the other parameters of a seed stay put
    for pol in (POLICY_FLOW, POLICY_GREEDY, POLICY_CHUNKED, POLICY_ALPHA, POLICY_CLASSFLOW, POLICY_MC):
        groups.append(Group(pol, b_fp=int(rng.integers(0, 3 * 65536)), chunk=int(rng.integers(1, 9)),
                            arrivals_id=int(rng.integers(0, 2)), rng_replica_base=base,
                            n_replicas=n_replicas, m_admit=int(rng.integers(max(2, M // 2), M + 1)),
                            b_class=tuple(int(x) for x in rng.integers(0, 3, size=n_classes)),
                            mc_worst_case=int(rng.integers(0, 2)),
                            preempt_keep=int(keep_rng.integers(0, 2)) if pol != POLICY_MC else 0))
        base += int(rng.integers(0, 2)) * n_replicas
    stride = int(rng.choice([1, 1, 2, 3]))
    return SimConfig(
        M=M, K=K, T_max=T, Qcap=int(rng.integers(1, 12)), Acap=int(rng.integers(2, 40)),
        seed=int(rng.integers(0, 2 ** 63)), class_law=class_law, prompt=prompt, decode=decode,
        arrivals=tuple(arrivals), groups=tuple(groups), trace_stride=stride,
        hist_bins=int(rng.choice([0, 8, 16])), hist_shift=int(rng.integers(0, 3)),
        complog_cap=int(rng.choice([0, 5, 64])), name=f"random-{seed}")


def random_medium_config(seed: int, n_replicas: int = 2) -> SimConfig:
    """A seeded, randomly parameterised simulation on the length laws of presets 2, 4 or 5 with a few
    thousand slots: three random policies, random capacities, budget, arrival law and outputs."""
    rng = np.random.default_rng(10_000 + seed)
    base = (config5, config2, config4)[int(rng.integers(0, 3))](replicas=1, T=100)
    T = int(rng.integers(1500, 4000))
    lmax = max(t.vmax for t in base.prompt)
    omax = max(t.vmax for t in base.decode)
    M = int(rng.integers(lmax + omax, 6 * (lmax + omax)))
    groups = []
    keep_rng = np.random.default_rng(600_000 + seed)
    for pol in rng.permutation(6)[:3]:
        groups.append(Group(int(pol), b_fp=int(rng.integers(0, 4 * 65536)), chunk=int(rng.choice([64, 512, 3000])),
                            arrivals_id=0, rng_replica_base=int(rng.integers(0, 1000)), n_replicas=n_replicas,
                            m_admit=int(rng.integers(M // 2, M + 1)),
                            b_class=tuple(int(x) for x in rng.integers(0, 3, size=base.n_classes)),
                            mc_worst_case=int(rng.integers(0, 2)),
                            preempt_keep=int(keep_rng.integers(0, 2)) if int(pol) != POLICY_MC else 0))
    lam = float(rng.uniform(0.2, 4.0))
    if rng.random() < 0.6:
        arr = Arrivals((poisson_table(lam),))
    else:
        arr = Arrivals((poisson_table(lam * 0.3), poisson_table(lam * 1.5)),
                       (int(rng.integers(0, 2 ** 28)), int(rng.integers(0, 2 ** 28))))
    return base.with_(M=M, K=int(rng.choice([0, 0, 700, 2048])), T_max=T, Qcap=int(rng.choice([8, 40, 256])),
                      Acap=int(rng.choice([48, 96, 200, 512])), seed=int(rng.integers(0, 2 ** 62)), arrivals=(arr,),
                      groups=tuple(groups), trace_stride=int(rng.choice([1, 1, 5])), hist_bins=64, hist_shift=6,
                      complog_cap=int(rng.choice([0, 300, 20000])), name=f"medium-{seed}")
