"""Full-size presets on the GPU, run in the benchmark's launch configuration (one fcsim_run per chunk of
slots): sampled replicas are compared word for word with the CPU checker, and every replica must satisfy
the exact integer identities of the model."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl

pytestmark = pytest.mark.gpu
I = orc.CIDX


def _oracle_rows(cfg, idx, n_steps):
    def one(r):
        return orc.run(cfg, int(r), 1, n_steps)
    with ThreadPoolExecutor(max_workers=16) as ex:
        return list(ex.map(one, idx))


def _identities(cfg, c, hist, n_steps):
    col = lambda n: c[:, I[n]]
    assert (col("steps_done") == n_steps).all()
    assert (col("arrived") == col("dropped") + col("completed") + col("q_final") + col("p_final")).all()
    assert (col("admitted") == col("completed") + col("evictions") + col("p_final")).all()
    assert (col("tokens_generated") == col("completed_tokens") + col("wasted_tokens") + col("resid_j")).all()
    assert (col("max_U") <= cfg.M).all()
    assert (col("sum_w_completed") <= col("sum_U")).all() and (col("sum_U") <= cfg.M * n_steps).all()
    assert (col("sum_N") == col("sum_lat") + col("resid_age")).all()
    assert (col("acap_blocked_steps") == 0).all() and (col("status") & 1 == 0).all()
    if hist is not None:
        assert (hist == col("completed")).all()


def _run_full(cfg, chunk, sample, n_steps=None):
    import torch
    from paper_2604_11001_b200 import binding as fb
    n_steps = cfg.T_max if n_steps is None else n_steps
    sim = fb.Simulation(cfg)
    done = 0
    while done < n_steps:
        s = min(chunk, n_steps - done)
        sim.run(s)
        done += s
    counters, summary = sim.stats()
    hist_tot = sim.hist().sum(dim=1, dtype=torch.int64).cpu().numpy() if cfg.hist_bins else None
    _identities(cfg, counters, hist_tot, n_steps)
    idx = torch.as_tensor(np.asarray(sample), device="cuda")
    rows = {"trace": sim.trace()[idx].cpu().numpy() if cfg.trace_stride else None,
            "hist": sim.hist()[idx].cpu().numpy() if cfg.hist_bins else None,
            "complog": sim.complog()[idx].cpu().numpy() if cfg.complog_cap else None}
    ref = _oracle_rows(cfg, sample, n_steps)
    for k, r in enumerate(sample):
        o = ref[k]
        bad = np.flatnonzero(counters[r] != o["counters"][0])
        assert bad.size == 0, (cfg.name, r, [orc.COUNTER_NAMES[b] for b in bad])
        if rows["trace"] is not None:
            n_rec = n_steps // cfg.trace_stride
            assert (rows["trace"][k, :n_rec] == o["trace"][0]).all(), (cfg.name, r, "trace")
        if rows["hist"] is not None:
            assert (rows["hist"][k] == o["hist"][0]).all(), (cfg.name, r, "hist")
        if rows["complog"] is not None:
            n = int(o["counters"][0, I["n_logged"]])
            assert (rows["complog"][k, :n] == o["complog"][0, :n]).all(), (cfg.name, r, "complog")
    # group summaries against the int64 sums of all replicas
    first = 0
    for g, grp in enumerate(cfg.groups):
        blk = counters[first:first + grp.n_replicas]
        assert summary[g]["completed"] == int(blk[:, I["completed"]].sum())
        assert summary[g]["max_lat"] == int(blk[:, I["max_lat"]].max())
        want = blk[:, I["sum_lat"]].sum() / max(1, blk[:, I["completed"]].sum())
        assert abs(summary[g]["mean_latency"] - want) <= 1e-9 * max(want, 1e-300)
        first += grp.n_replicas
        if g > 64:
            break
    sim.close()
    return counters


def _sample(cfg, per_group, seed):
    rng = np.random.default_rng(seed)
    out, first = [], 0
    groups = list(range(len(cfg.groups)))
    if len(groups) > 8:
        groups = sorted(set([0, len(groups) - 1] + list(rng.choice(len(groups), 22, replace=False))))
    starts = np.cumsum([0] + [g.n_replicas for g in cfg.groups])
    for g in groups:
        n = cfg.groups[g].n_replicas
        pick = {0, n - 1} | set(int(x) for x in rng.integers(0, n, size=max(0, per_group - 2)))
        out += [int(starts[g] + p) for p in sorted(pick)][:per_group]
    return out


def test_config2_full():
    cfg = wl.config2()
    _run_full(cfg, 1000, _sample(cfg, 12, 2))


def test_config3_full():
    cfg = wl.config3()
    _run_full(cfg, 2000, _sample(cfg, 1, 3))


def test_config4_full():
    cfg = wl.config4()
    _run_full(cfg, 2000, _sample(cfg, 10, 4))


def test_config5_full():
    cfg = wl.config5()
    c = _run_full(cfg, 2000, _sample(cfg, 16, 5))
    # overloaded by construction: the waiting room is full and arrivals are being dropped
    assert c[:, I["dropped"]].min() > 0 and c[:, I["evictions"]].sum() > 0


def test_config5_all_replicas_first_2000_slots_against_a_stratified_sample():
    cfg = wl.config5()
    _run_full(cfg, 2000, list(range(0, cfg.n_replicas, 4099)), n_steps=2000)


def test_config6_full_paper_setting():
    cfg = wl.config6()
    c = _run_full(cfg, 500, _sample(cfg, 8, 6))
    # Section 4.1's load is light (about 0.41 of the necessary-condition load): flow control with b = 12 > lambda
    # never overflows, and nothing is dropped
    n = cfg.groups[0].n_replicas
    assert c[:n, I["overflow_steps"]].sum() == 0 and c[:, I["dropped"]].sum() == 0
    # Algorithm 1 with b = (4,4,4) (last group): usage never passes sum_k b_k w_k = 16240 < M, no eviction (Thm. 3.3)
    alg1 = c[3 * n:4 * n]
    assert (alg1[:, I["max_U"]] <= 16240).all() and alg1[:, I["evictions"]].sum() == 0
    assert alg1[:, I["gate_blocked_steps"]].sum() == 0 and alg1[:, I["completed"]].min() > 40000
    # MC benchmark (known and worst-case lengths): admissions are proved to fit, so nothing is ever evicted
    mc = c[4 * n:]
    assert mc[:, I["evictions"]].sum() == 0 and mc[:, I["overflow_steps"]].sum() == 0
    assert mc[:, I["completed"]].min() > 40000


def test_one_call_split_into_several_launches():
    # 262 144 replicas: the library splits a 10 000-slot call into launches of at most 8 192 slots
    from paper_2604_11001_b200 import binding as fb
    cfg = wl.config5(T=10000)
    sim = fb.Simulation(cfg)
    assert sim.launch_info()["max_steps_per_launch"] < 10000
    sim.close()
    _run_full(cfg, 10000, list(range(5, cfg.n_replicas, 16411)))


def test_horizon_at_the_24_bit_limit():
    # T_max = 2^24 - 1 slots: arrival times use all 24 bits of the packed entry, and the run spans 512 launches of
    # 32 768 slots whose 32-bit partial sums are folded into the int64 counters
    cfg = wl.config1(replicas=2, T=(1 << 24) - 1).with_(trace_stride=4096, complog_cap=4096, hist_shift=3)
    _run_full(cfg, (1 << 24) - 1, [0, 1])
