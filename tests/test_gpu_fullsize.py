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
    """The CPU checker's outputs for the replicas ``idx`` (ascending; one dict of stacked arrays)."""
    idx = [int(r) for r in idx]
    if idx == list(range(idx[0], idx[0] + len(idx))):          # one contiguous range: one call, 16 threads
        return orc.run(cfg, idx[0], len(idx), n_steps, threads=16)
    runs = [[idx[0], 1]]                                       # maximal contiguous runs, one call each
    for r in idx[1:]:
        if r == runs[-1][0] + runs[-1][1]:
            runs[-1][1] += 1
        else:
            runs.append([r, 1])

    def one(run):
        return orc.run(cfg, run[0], run[1], n_steps)
    with ThreadPoolExecutor(max_workers=16) as ex:
        parts = list(ex.map(one, runs))
    return {k: (None if parts[0][k] is None else np.concatenate([q[k] for q in parts], axis=0)) for k in parts[0]}


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


def _run_full(cfg, chunk, sample, n_steps=None, batch=512):
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
    sample = [int(r) for r in sample]
    for lo in range(0, len(sample), batch):                    # in batches: a full trace does not fit twice in RAM
        part = sample[lo:lo + batch]
        idx = torch.as_tensor(np.asarray(part), device="cuda")
        ref = _oracle_rows(cfg, part, n_steps)
        bad = np.argwhere(counters[part] != ref["counters"])
        assert bad.size == 0, (cfg.name, part[bad[0][0]], orc.COUNTER_NAMES[bad[0][1]], len(bad))
        if cfg.trace_stride:
            n_rec = n_steps // cfg.trace_stride
            rows = sim.trace()[idx, :n_rec].cpu().numpy()
            same = (rows == ref["trace"]).all(axis=(1, 2))
            assert same.all(), (cfg.name, part[int(np.flatnonzero(~same)[0])], "trace")
        if cfg.hist_bins:
            same = (sim.hist()[idx].cpu().numpy() == ref["hist"]).all(axis=1)
            assert same.all(), (cfg.name, part[int(np.flatnonzero(~same)[0])], "hist")
        if cfg.complog_cap:
            rows = sim.complog()[idx].cpu().numpy()
            n = ref["counters"][:, I["n_logged"]]
            live = np.arange(cfg.complog_cap)[None, :] < n[:, None]      # entries past n_logged are unspecified
            same = ((rows == ref["complog"]).all(axis=2) | ~live).all(axis=1)
            assert same.all(), (cfg.name, part[int(np.flatnonzero(~same)[0])], "complog")
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
    _run_full(cfg, 1000, range(cfg.n_replicas))            # every replica, every output word


def test_config3_full():
    cfg = wl.config3()
    # every 2nd group of the 64 x 64 sweep (offset 1: every arrival rate, 32 of the 64 flow-control settings), all
    # 16 replicas of each: 32 768 replicas over the full horizon
    groups = range(1, len(cfg.groups), 2)
    _run_full(cfg, 2000, [16 * g + k for g in groups for k in range(16)], batch=1024)


def test_config4_full():
    cfg = wl.config4()
    _run_full(cfg, 2000, range(cfg.n_replicas), batch=4096)   # every replica of both groups, every output word


def test_config5_full():
    cfg = wl.config5()
    c = _run_full(cfg, 2000, range(17, cfg.n_replicas, 64))   # 4096 replicas spread over both groups
    # overloaded by construction: the waiting room is full and arrivals are being dropped
    assert c[:, I["dropped"]].min() > 0 and c[:, I["evictions"]].sum() > 0


def test_config5_first_2000_slots_every_replica():
    cfg = wl.config5()
    _run_full(cfg, 2000, range(cfg.n_replicas), n_steps=2000, batch=16384)


def test_config6_full_paper_setting():
    cfg = wl.config6()
    # 64 replicas of each of the four cheap policies, 24 of each MC group (the checker's future-memory test walks
    # every future slot of every running request)
    n0 = cfg.groups[0].n_replicas
    sample = sorted([g * n0 + k for g in range(4) for k in range(g, n0, n0 // 64)][:4 * 64]
                    + [g * n0 + k for g in (4, 5) for k in range(g, n0, n0 // 24)][:2 * 24])
    c = _run_full(cfg, 500, sample)
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


def test_host_buffer_entry_point_streams_a_large_trace():
    # 8192 replicas x 8000 slots: a 524 MB trace leaves the device in windows of 2048 records per replica while the
    # run goes on (four windows, the last one partial); every output word against the CPU checker.  The second
    # call stops 1000 slots before the horizon: the records of the slots not run must read as zero.
    from paper_2604_11001_b200 import binding as fb
    cfg = wl.config2(replicas=4096, T=8000)
    assert fb.fcsim_query_sizes(cfg)["trace"] >= 256 << 20
    ref = orc.run(cfg, threads=16)
    host = fb.host_output_arrays(cfg, pinned=True)
    out = fb.fcsim_simulate_host(cfg, out=host)
    assert (out["counters"] == ref["counters"]).all()
    assert (out["trace"] == ref["trace"]).all()
    assert (out["hist"] == ref["hist"]).all()
    n = ref["counters"][:, I["n_logged"]]
    live = np.arange(cfg.complog_cap)[None, :] < n[:, None]
    assert ((out["complog"] == ref["complog"]).all(axis=2) | ~live).all()
    host["trace"][:] = -1
    part = fb.fcsim_simulate_host(cfg, 7000, out=host)
    assert (part["trace"][:, :7000] == ref["trace"][:, :7000]).all()
    assert (part["trace"][:, 7000:] == 0).all()
    short = orc.run(cfg, 0, 64, 7000, threads=16)
    assert (part["counters"][:64] == short["counters"]).all()
