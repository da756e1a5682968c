"""GPU parity: the CUDA library against the CPU checker, word for word, through the C ABI."""
import os

import numpy as np
import pytest

from gpu_common import assert_same, assert_summary_close, run_gpu
from helpers import degenerate_config, read_fixture, scaled_presets, trace_fixtures
from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


@pytest.mark.parametrize("name", trace_fixtures(GOLDEN))
def test_hand_traces_on_gpu(name):
    fx = read_fixture(os.path.join(GOLDEN, name))
    cfg = degenerate_config(**fx["params"])
    gpu = run_gpu(cfg)
    assert gpu["trace"][0, :, 0].tolist() == fx["U"]
    assert gpu["trace"][0, :, 1].tolist() == fx["Q"]
    n = int(gpu["counters"][0, orc.CIDX["n_logged"]])
    assert [tuple(x) for x in gpu["complog"][0, :n].tolist()] == fx["completions"]
    assert_same(cfg, gpu, orc.run(cfg), cfg.T_max, name)


@pytest.mark.parametrize("seed", range(600))
def test_random_small_configs(seed):
    cfg = wl.random_small_config(seed, n_replicas=5, T=97)
    gpu = run_gpu(cfg)
    ref = orc.run(cfg)
    assert_same(cfg, gpu, ref, cfg.T_max, cfg.name)
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], cfg.T_max, ref["complog"])


@pytest.mark.parametrize("cfg", scaled_presets(), ids=lambda c: c.name)
def test_scaled_presets(cfg):
    gpu = run_gpu(cfg)
    ref = orc.run(cfg, threads=8)
    assert_same(cfg, gpu, ref, cfg.T_max, cfg.name)
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], cfg.T_max, ref["complog"])


def test_config1_full():
    cfg = wl.config1()
    gpu = run_gpu(cfg)
    ref = orc.run(cfg, threads=8)
    assert_same(cfg, gpu, ref, cfg.T_max, "cfg1")
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], cfg.T_max, ref["complog"])


@pytest.mark.parametrize("pieces", [[1] * 40 + [60], [33, 31, 36], [7, 64, 29], [99, 1]])
def test_resumed_runs_equal_one_run(pieces):
    for seed in (3, 11, 17):
        cfg = wl.random_small_config(seed, n_replicas=4, T=100)
        whole = run_gpu(cfg)
        parts = run_gpu(cfg, pieces=pieces)
        for k in ("counters", "trace", "hist", "complog"):
            if whole[k] is not None:
                assert (whole[k] == parts[k]).all(), (seed, k)
    cfg = wl.config1(replicas=8, T=sum(pieces) * 10)
    ref = orc.run(cfg)
    parts = run_gpu(cfg, pieces=[p * 10 for p in pieces])
    assert_same(cfg, parts, ref, cfg.T_max, "cfg1 resumed")


def test_pause_counters_match_a_shorter_run():
    cfg = wl.config5(replicas=4, T=3000)
    gpu = run_gpu(cfg, n_steps=1234)
    ref = orc.run(cfg, n_steps=1234)
    assert_same(cfg, gpu, ref, 1234, "cfg5 paused")
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], 1234, ref["complog"])


def test_more_replicas_than_resident_warps_and_many_groups():
    # several replicas per warp (work queue), several launches, 24 groups
    cfg = wl.config3(n_rates=4, n_b=6, reps=3, T=1500)
    cfg = cfg.with_(Qcap=64, Acap=256)
    gpu = run_gpu(cfg)
    ref = orc.run(cfg, threads=8)
    assert_same(cfg, gpu, ref, cfg.T_max, "cfg3 grid")
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], cfg.T_max, ref["complog"])
    big = wl.config1(replicas=20000, T=64).with_(trace_stride=8, complog_cap=8)
    gpu = run_gpu(big)
    ref = orc.run(big, threads=8)
    assert_same(big, gpu, ref, big.T_max, "20000 replicas")


def test_large_flow_rate_equals_greedy_on_gpu():
    cfg = wl.config1(replicas=6, T=1200)
    flow = cfg.with_(groups=(wl.Group(wl.POLICY_FLOW, b_fp=0xFFFF0000, n_replicas=6),))
    greedy = cfg.with_(groups=(wl.Group(wl.POLICY_GREEDY, n_replicas=6),))
    a, b = run_gpu(flow), run_gpu(greedy)
    for k in ("trace", "hist", "complog"):
        assert (a[k] == b[k]).all()
    assert_same(flow, a, orc.run(flow), cfg.T_max, "flow b=65535")


def test_edge_shapes():
    # one replica; zero steps; tiny capacities (Acap blocks, waiting room of one); no outputs at all
    one = degenerate_config(n=1, l=2, o=3, policy="flow", b=1, K=0, c=0, M=11, T=5)
    gpu = run_gpu(one, n_steps=0)
    assert (gpu["counters"] == 0).all()
    tight = wl.config1(replicas=3, T=400).with_(Qcap=1, Acap=2, M=700)
    assert_same(tight, run_gpu(tight), orc.run(tight), 400, "tight")
    ref = orc.run(tight)
    assert ref["counters"][:, orc.CIDX["acap_blocked_steps"]].sum() > 0
    bare = wl.config1(replicas=3, T=300).with_(trace_stride=0, hist_bins=0, complog_cap=0)
    assert_same(bare, run_gpu(bare), orc.run(bare), 300, "bare")
    burst = degenerate_config(n=200, l=1, o=1, policy="greedy", b=0, K=0, c=0, M=100000, T=40, Qcap=1000, Acap=700)
    assert_same(burst, run_gpu(burst), orc.run(burst), 40, "burst")
    strided = wl.config1(replicas=2, T=1000).with_(trace_stride=7)
    assert_same(strided, run_gpu(strided, pieces=[500, 3, 497]), orc.run(strided), 1000, "stride 7")


def test_host_buffer_entry_point():
    from paper_2604_11001_b200 import binding as fb
    cfg = wl.config1(replicas=16, T=500)
    out = fb.fcsim_simulate_host(cfg)
    ref = orc.run(cfg)
    assert_same(cfg, out, ref, 500, "simulate_host")
    assert_summary_close(cfg, out["summary"], ref["counters"], ref["hist"], 500, ref["complog"])


def test_large_active_set_and_lazy_removal_paths():
    # Acap > 1024 (several 32-entry blocks per watching lane), completions piling up between removals,
    # removal forced by storage (active range full of completed entries) and by evictions
    many = degenerate_config(n=40, l=1, o=3, policy="greedy", b=0, K=0, c=0, M=100000, T=120, Qcap=2000, Acap=1500)
    many = many.with_(arrivals=(wl.Arrivals((wl.poisson_table(30.0),)),), decode=(wl.uniform_table(1, 60),),
                      complog_cap=8192)
    assert_same(many, run_gpu(many), orc.run(many), 120, "Acap 1500")
    tight = wl.config1(replicas=6, T=1500).with_(
        Acap=40, Qcap=30, M=12000, arrivals=(wl.Arrivals((wl.poisson_table(1.5),)),),
        groups=(wl.Group(wl.POLICY_FLOW, b_fp=0x30000, n_replicas=6),))
    ref = orc.run(tight)
    assert ref["counters"][:, orc.CIDX["acap_blocked_steps"]].sum() > 0
    assert_same(tight, run_gpu(tight), ref, 1500, "storage-bound")
    churn = wl.config2(replicas=2, T=3000).with_(M=20000, Acap=96)
    assert_same(churn, run_gpu(churn, pieces=[1000, 1, 1999]), orc.run(churn), 3000, "eviction churn")


def test_trace_bulk_copy_variant():
    # opt-in variant: trace records staged in shared memory and stored with 256-byte bulk copies.  Rows of 333
    # records: odd rows start 8 bytes off a 16-byte boundary and must fall back to plain stores.
    cfg = wl.config1(replicas=9, T=333).with_(trace_bulk=1)
    assert_same(cfg, run_gpu(cfg, pieces=[100, 7, 226]), orc.run(cfg), 333, "bulk trace")
    cfg = wl.config2(replicas=2, T=2000).with_(trace_bulk=1)
    assert_same(cfg, run_gpu(cfg), orc.run(cfg), 2000, "bulk trace cfg2")


def test_maximum_sizes():
    # lengths at the 16-bit limit, capacity 2^30, an active ring so large that a CTA holds a single warp,
    # 255 arrivals in a slot, the largest flow rate
    big = wl.SimConfig(
        M=1 << 30, K=0, T_max=300, Qcap=9000, Acap=16000, seed=(1 << 63) + 5, class_law=wl.constant_table(0),
        prompt=(wl.uniform_table(65000, 65535),), decode=(wl.table_from_pmf(1, [0.5] + [0.0] * 65533 + [0.5]),),
        arrivals=(wl.Arrivals((wl.table_from_pmf(0, [0.5] + [0.0] * 254 + [0.5]),)),),
        groups=(wl.Group(wl.POLICY_FLOW, b_fp=0xFFFFFFFF, n_replicas=3),
                wl.Group(wl.POLICY_GREEDY, n_replicas=3, rng_replica_base=0xFFFFFFF0)),
        trace_stride=1, hist_bins=4, hist_shift=30, complog_cap=100000)
    gpu = run_gpu(big)
    assert gpu["launch"]["warps_per_block"] == 1
    ref = orc.run(big)
    assert_same(big, gpu, ref, 300, "maximum sizes")
    assert ref["counters"][:, orc.CIDX["max_U"]].max() > 1 << 28
    assert ref["counters"][:, orc.CIDX["dropped"]].sum() > 0


def test_horizon_limit_and_range_errors():
    from paper_2604_11001_b200 import binding as fb
    cfg = wl.config1(replicas=2, T=50)
    sim = fb.Simulation(cfg)
    sim.run(50)
    with pytest.raises(fb.FcsimError) as e:
        sim.run(1)
    assert e.value.code == -4
    assert sim.steps_done == 50
    sim.close()
    # slots close to the 24-bit horizon limit: arrival times near 2^24 must survive the packing
    late = wl.config1(replicas=2, T=(1 << 24) - 1)
    assert fb.fcsim_query_sizes(late.with_(trace_stride=0, complog_cap=0))["trace"] == 0


@pytest.mark.parametrize("seed", range(250))
def test_random_medium_configs(seed):
    # preset-sized laws, thousands of slots, every policy: lazy removal, in-place eviction, storage-bound
    # squeezes and resumed launches all occur
    cfg = wl.random_medium_config(seed)
    cut = 1 + (seed * 97) % (cfg.T_max - 1)
    ref = orc.run(cfg, threads=4)
    gpu = run_gpu(cfg, pieces=[cut, cfg.T_max - cut])
    assert_same(cfg, gpu, ref, cfg.T_max, cfg.name)
    # logs of 300 entries overflow (histogram percentiles), logs of 20 000 do not (exact percentiles)
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], cfg.T_max, ref["complog"])


def test_handles_with_different_shared_memory_needs_coexist():
    # a handle that needs more than the default 48 KB of shared memory per CTA must keep working after a
    # smaller one has been created (the opt-in limit belongs to the kernel, not to the handle)
    from paper_2604_11001_b200 import binding as fb
    big_cfg = degenerate_config(n=20, l=1, o=3, policy="greedy", b=0, K=0, c=0, M=100000, T=60, Qcap=2000, Acap=5000)
    big_cfg = big_cfg.with_(decode=(wl.uniform_table(1, 40),))
    small_cfg = wl.config1(replicas=4, T=60)
    big = fb.Simulation(big_cfg)
    assert big.launch_info()["smem_per_block"] > 48 * 1024
    small = fb.Simulation(small_cfg)
    small.run(60)
    big.run(60)
    small_c, _ = small.stats()
    big_c, _ = big.stats()
    assert (big_c == orc.run(big_cfg)["counters"]).all()
    assert (small_c == orc.run(small_cfg)["counters"]).all()
    big.close()
    small.close()


def test_evictions_that_keep_the_generated_tokens():
    # every evicting policy on the heavy-tailed lengths of preset 5 and on preset 2's laws, many evictions,
    # resumed launches (rewritten entries cross the save/restore of the rings), kept tokens next to 2^16
    import dataclasses
    base = wl.config5(replicas=1, T=6000)
    groups = tuple(wl.Group(pol, b_fp=0x28000, chunk=256, n_replicas=3, m_admit=base.M - 64,
                            b_class=(1, 1, 1), rng_replica_base=5, preempt_keep=1)
                   for pol in (wl.POLICY_FLOW, wl.POLICY_GREEDY, wl.POLICY_CHUNKED, wl.POLICY_ALPHA,
                               wl.POLICY_CLASSFLOW))
    cfg = base.with_(groups=groups, trace_stride=1, complog_cap=4096)
    ref = orc.run(cfg)
    ev = ref["counters"][:, orc.CIDX["evictions"]].reshape(5, 3).sum(axis=1)
    assert (ev > 50).all(), ev
    assert ref["counters"][:, orc.CIDX["wasted_tokens"]].sum() == 0
    assert_same(cfg, run_gpu(cfg, pieces=[1500, 7, 2493, 2000]), ref, 6000, "keep, preset-5 laws")
    off = cfg.with_(groups=tuple(dataclasses.replace(g, preempt_keep=0) for g in groups))
    assert (orc.run(off)["counters"] != ref["counters"]).any()
    # longest lengths the variant accepts, l_max + o_max = 65536, with two running requests and a capacity that
    # overflows 10 slots before the first one ends: the second is evicted holding 35 525 tokens, l becomes 65 525
    big = degenerate_config(n=1, l=30000, o=35536, policy="greedy", b=0, K=0, c=0, M=131052, T=36000, Acap=2, keep=1)
    big = big.with_(trace_stride=500, complog_cap=16)
    refb = orc.run(big)
    assert refb["counters"][0, orc.CIDX["evictions"]] == 1 and refb["counters"][0, orc.CIDX["completed"]] == 2
    assert refb["counters"][0, orc.CIDX["completed_tokens"]] == 2 * 35536
    assert refb["counters"][0, orc.CIDX["prefill_tokens"]] == 4 * 30000 + 65525
    assert_same(big, run_gpu(big), refb, 36000, "keep, 16-bit edge")


def test_keep_variant_argument_errors():
    from paper_2604_11001_b200 import binding as fb
    too_long = degenerate_config(n=1, l=30001, o=35536, policy="greedy", b=0, K=0, c=0, M=90000, T=10, keep=1)
    with pytest.raises(fb.FcsimError):
        fb.Simulation(too_long)
    mc = degenerate_config(n=1, l=2, o=3, policy=wl.POLICY_MC, b=0, K=0, c=0, M=100, T=10, keep=1)
    with pytest.raises(fb.FcsimError):
        fb.Simulation(mc)
    flag = degenerate_config(n=1, l=2, o=3, policy="greedy", b=0, K=0, c=0, M=100, T=10, keep=2)
    with pytest.raises(fb.FcsimError):
        fb.Simulation(flag)


def test_mc_many_finishers_in_one_slot():
    # worst-case projection with more than 32 requests ending in the same slot (their corrections are collected
    # one per lane and flushed when the lanes run out), with and without a binding capacity
    for M, mode in ((100000, 1), (330, 1), (330, 0)):
        cfg = degenerate_config(n=48, l=1, o=3, policy=wl.POLICY_MC, b=0, K=0, c=0, M=M, T=300, Qcap=600, Acap=400)
        cfg = cfg.with_(decode=(wl.uniform_table(1, 4),), arrivals=(wl.Arrivals((wl.poisson_table(44.0),)),),
                        groups=(wl.Group(wl.POLICY_MC, n_replicas=3, mc_worst_case=mode),), complog_cap=20000)
        ref = orc.run(cfg)
        c = ref["counters"]
        assert (c[:, orc.CIDX["completed"]] > 32 * 150).all()
        if M == 330:
            assert (c[:, orc.CIDX["gate_blocked_steps"]] > 50).all()
        assert_same(cfg, run_gpu(cfg, pieces=[100, 200]), ref, 300, f"MC finishers M={M} worst={mode}")


def test_policies_interleaved_over_groups_on_a_side_stream():
    # every policy's kernel walks a work list made of several non-adjacent groups of unequal size; the call is
    # made on a stream other than the default one, in resumed pieces, and the kernels of the policies run side
    # by side on streams of the handle
    import dataclasses
    import torch
    from paper_2604_11001_b200 import binding as fb
    base = wl.random_medium_config(3, n_replicas=1)
    proto = {g.policy: g for seed in (3, 4, 5, 6) for g in wl.random_medium_config(seed).groups}
    order = [1, 0, 3, 1, 2, 0, 0, 5, 1, 4, 2, 0]
    sizes = [3, 1, 2, 5, 1, 4, 2, 2, 1, 3, 2, 6]
    groups, rid = [], 0
    for pol, n in zip(order, sizes):
        if pol not in proto:
            continue
        groups.append(dataclasses.replace(proto[pol], n_replicas=n, rng_replica_base=rid,
                                          b_class=(2, 1, 1, 1)[:base.n_classes]))
        rid += n
    cfg = base.with_(groups=tuple(groups), T_max=1200, Acap=200, Qcap=40, complog_cap=300)
    assert len({g.policy for g in cfg.groups}) >= 4
    ref = orc.run(cfg, threads=8)
    sim = fb.Simulation(cfg)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for piece in (1, 499, 700):
            sim.run(piece, side)
        counters, summary = sim.stats(side)
    gpu = {"counters": counters, "summary": summary}
    for name in ("trace", "hist", "complog"):
        v = getattr(sim, name)()
        gpu[name] = None if v is None else v.cpu().numpy()
    sim.close()
    assert_same(cfg, gpu, ref, 1200, "interleaved policies")


def test_dense_tables_take_the_guide_fall_back_search():
    # length laws with far more thresholds than a guide has buckets (60 000 equiprobable prompt lengths: about four
    # thresholds per bucket, so every fifth lookup must finish with the search behind the guide record), an arrival
    # count law with mass at both ends, and a class law with a class of probability zero
    prompt = (wl.uniform_table(1, 60000), wl.uniform_table(7, 7), wl.table_from_pmf(3, [0.999] + [1e-3 / 4999] * 4999))
    decode = (wl.uniform_table(1, 300), wl.geometric_table(3.0, 4000), wl.uniform_table(2, 3))
    cfg = wl.SimConfig(
        M=4000000, K=0, T_max=500, Qcap=64, Acap=256, seed=77, class_law=wl.table_from_pmf(0, [0.6, 0.0, 0.4]),
        prompt=prompt, decode=decode,
        arrivals=(wl.Arrivals((wl.table_from_pmf(0, [0.55] + [0.0] * 2 + [0.4] + [0.0] * 26 + [0.05]),)),),
        groups=(wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(2.5), n_replicas=6),
                wl.Group(wl.POLICY_GREEDY, n_replicas=6, rng_replica_base=100)),
        trace_stride=1, hist_bins=32, hist_shift=5, complog_cap=4096)
    ref = orc.run(cfg, threads=4)
    assert ref["counters"][:, orc.CIDX["completed"]].min() > 200
    assert_same(cfg, run_gpu(cfg, pieces=[123, 377]), ref, 500, "dense tables")


def test_index_checked_build_records_no_violation():
    # the same kernels compiled with every shared-memory and output index compared with its bound, over random
    # configurations of all policies and cuts of the presets; run in a process of its own (one build per process)
    import subprocess
    import sys
    runner = os.path.join(os.path.dirname(os.path.abspath(__file__)), "checked_runner.py")
    out = subprocess.run([sys.executable, runner], capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "violations: 0" in out.stdout, out.stdout[-2000:]


def test_two_handles_driven_from_two_threads():
    # handles with different shared-memory needs use the same kernels; each thread creates its handle, runs it in
    # many short calls and reads its statistics while the other does the same
    import threading
    from paper_2604_11001_b200 import binding as fb
    big_cfg = degenerate_config(n=20, l=1, o=3, policy="greedy", b=0, K=0, c=0, M=100000, T=400, Qcap=2000, Acap=5000)
    big_cfg = big_cfg.with_(decode=(wl.uniform_table(1, 40),))
    small_cfg = wl.config1(replicas=8, T=400)
    out, errors = {}, []

    def drive(name, cfg):
        try:
            import torch
            stream = torch.cuda.Stream()
            sim = fb.Simulation(cfg)
            for _ in range(40):
                sim.run(10, stream)
            out[name] = sim.stats(stream)[0]
            sim.close()
        except Exception as e:   # reported by the main thread
            errors.append((name, repr(e)))

    threads = [threading.Thread(target=drive, args=("big", big_cfg)),
               threading.Thread(target=drive, args=("small", small_cfg))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
    assert (out["big"] == orc.run(big_cfg)["counters"]).all()
    assert (out["small"] == orc.run(small_cfg)["counters"]).all()


def test_exact_percentiles_from_the_completion_log():
    # the hand trace whose 7th smallest latency is 6 while its histogram bin ends at 7
    cfg = degenerate_config(n=1, l=2, o=3, policy="flow", b=1, K=0, c=0, M=11, T=12, hist_bins=8).with_(hist_shift=2)
    s = run_gpu(cfg)["summary"][0]
    assert s["p95_latency"] == 6.0 and s["p99_latency"] == 6.0 and s["percentile_source"] == 2
    # groups of unequal size, latencies on both sides of 4096 (two-digit selection), several replicas per group,
    # p95 and p99 in different high digits; one group completes nothing
    base = wl.config2(replicas=1, T=9000)
    groups = (wl.Group(wl.POLICY_FLOW, b_fp=0x6000, n_replicas=37, rng_replica_base=3),
              wl.Group(wl.POLICY_FLOW, b_fp=0, n_replicas=2),
              wl.Group(wl.POLICY_GREEDY, n_replicas=11),
              wl.Group(wl.POLICY_FLOW, b_fp=0x20000, n_replicas=1, rng_replica_base=77))
    cfg = base.with_(groups=groups, Qcap=4096, trace_stride=0, hist_shift=7, complog_cap=8192)
    ref = orc.run(cfg, threads=8)
    want = orc.summarize(cfg, ref["counters"], ref["hist"], 9000, ref["complog"])
    assert want[0]["max_lat"] > 4096 and want[0]["percentile_source"] == 2 and want[1]["percentile_source"] == 0
    assert want[0]["p99_latency"] - want[0]["p95_latency"] > 100
    hist_rule = orc.summarize(cfg, ref["counters"], ref["hist"], 9000)
    assert hist_rule[0]["p95_latency"] != want[0]["p95_latency"]
    gpu = run_gpu(cfg, pieces=[4000, 5000])
    assert_same(cfg, gpu, ref, 9000, "exact percentiles")
    assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], 9000, ref["complog"])
    # a log too small for the run: the histogram rule, and the summary says so
    short = cfg.with_(complog_cap=64)
    refs = orc.run(short, threads=8)
    gpus = run_gpu(short)
    assert gpus["summary"][0]["percentile_source"] == 1
    assert_summary_close(short, gpus["summary"], refs["counters"], refs["hist"], 9000, refs["complog"])


def test_standing_queue_of_200000_over_a_long_run():
    # |P| + |Q| summed over the slots passes 2^32 within what used to be one launch: the per-launch partial sums
    # are 32-bit, so the library must cut the launches short enough (Qcap + 2 Acap per slot at most).  Nothing is
    # ever activated (b = 0), so the slot-exact Little identity reads sum_N = resid_age.
    from paper_2604_11001_b200 import binding as fb
    cfg = degenerate_config(n=255, l=1, o=1, policy="flow", b=0, K=0, c=0, M=1000, T=33000, Qcap=200000, Acap=64,
                            replicas=2)
    cfg = cfg.with_(trace_stride=1000, complog_cap=0, hist_bins=0)
    sim = fb.Simulation(cfg)
    per = sim.launch_info()["max_steps_per_launch"]
    assert per * (200000 + 128) < (1 << 32) - (1 << 30)
    sim.close()
    gpu = run_gpu(cfg)
    c = gpu["counters"]
    I = orc.CIDX
    assert (c[:, I["sum_N"]] > (1 << 32)).all() and (c[:, I["sum_lat"]] == 0).all()
    assert (c[:, I["sum_N"]] == c[:, I["sum_lat"]] + c[:, I["resid_age"]]).all()
    assert (c[:, I["q_final"]] == 200000).all() and (c[:, I["dropped"]] == 255 * 33000 - 200000).all()
    ref = orc.run(cfg, threads=2)
    assert_same(cfg, gpu, ref, 33000, "standing queue")


def test_many_activations_per_slot():
    # six arrivals per slot and a cache that serves about as many: the kernels that activate several queue heads
    # at once are chosen; gate, token budget (with and without), storage bound and flow-control budget all end
    # runs of activations, evictions push requests back in front of the window on the queue
    for K, M, Acap in ((0, 1400, 200), (45, 3000, 200), (0, 1000, 200), (0, 100000, 48)):
        cfg = wl.SimConfig(
            M=M, K=K, T_max=700, Qcap=100, Acap=Acap, seed=91 + K, class_law=wl.table_from_pmf(0, [0.5, 0.5]),
            prompt=(wl.uniform_table(1, 20), wl.uniform_table(5, 9)), decode=(wl.uniform_table(1, 30), wl.uniform_table(2, 12)),
            arrivals=(wl.Arrivals((wl.poisson_table(6.0),)), wl.Arrivals((wl.poisson_table(3.0), wl.poisson_table(9.0)), (1 << 27, 1 << 28))),
            groups=(wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(5.5), n_replicas=5),
                    wl.Group(wl.POLICY_GREEDY, n_replicas=5, arrivals_id=1),
                    wl.Group(wl.POLICY_ALPHA, n_replicas=5, m_admit=int(0.8 * M)),
                    wl.Group(wl.POLICY_GREEDY, n_replicas=4, preempt_keep=1, rng_replica_base=40),
                    wl.Group(wl.POLICY_CLASSFLOW, n_replicas=5, b_class=(3, 4)),
                    wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(40.0), n_replicas=3, arrivals_id=1)),
            trace_stride=1, hist_bins=64, hist_shift=1, complog_cap=6000)
        ref = orc.run(cfg, threads=4)
        c = ref["counters"]
        assert c[:, orc.CIDX["admitted"]].min() > 2 * 700
        if M == 1000:
            assert c[:, orc.CIDX["evictions"]].sum() > 100 and c[:, orc.CIDX["gate_blocked_steps"]].min() > 50
        if K:
            assert c[:, orc.CIDX["budget_blocked_steps"]].sum() > 100
        if Acap == 48:
            assert c[:, orc.CIDX["acap_blocked_steps"]].sum() > 0
        gpu = run_gpu(cfg, pieces=[333, 367])
        assert_same(cfg, gpu, ref, 700, f"many activations K={K} M={M} Acap={Acap}")
        assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], 700, ref["complog"])


def test_arrivals_drawn_when_they_reach_the_queue_head():
    # heavy overload without per-slot outputs: the kernels that let arrivals wait undrawn in a long queue are chosen.
    # Two-state arrivals (quiet / very busy) make the queue drain below the threshold and fill up again, so drawn and
    # undrawn arrivals mix, late arrivals land inside the window on the queue head, evictions push requests back in
    # front of it, bursts of up to 200 arrivals are activated in one slot, and launches are resumed in between.
    base = wl.config5(replicas=1, T=100)
    for i, (Qcap, M, K) in enumerate(((128, 600000, 2048), (200, 70000, 0), (256, 250000, 700))):
        groups = (wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(0.8), n_replicas=4),
                  wl.Group(wl.POLICY_GREEDY, n_replicas=4),
                  wl.Group(wl.POLICY_CHUNKED, chunk=512, n_replicas=3),
                  wl.Group(wl.POLICY_ALPHA, n_replicas=3, m_admit=int(0.9 * M)),
                  wl.Group(wl.POLICY_GREEDY, n_replicas=3, preempt_keep=1, rng_replica_base=50),
                  wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(2.5), n_replicas=3, preempt_keep=1, rng_replica_base=9))
        arr = wl.Arrivals((wl.poisson_table(0.05), wl.poisson_table(9.0)), (1 << 25, 1 << 26))
        cfg = base.with_(M=M, K=K, T_max=5000, Qcap=Qcap, Acap=256, seed=300 + i, arrivals=(arr,), groups=groups,
                         trace_stride=0, complog_cap=0, hist_bins=256, hist_shift=4)
        ref = orc.run(cfg, threads=8)
        c = ref["counters"]
        assert c[:, orc.CIDX["dropped"]].min() > 1000 and (i == 0 or c[:, orc.CIDX["evictions"]].sum() > 100)
        gpu = run_gpu(cfg, pieces=[1777, 1, 3222])
        assert_same(cfg, gpu, ref, 5000, f"undrawn arrivals {i}")
        assert_summary_close(cfg, gpu["summary"], ref["counters"], ref["hist"], 5000, ref["complog"])
    # short requests, a cache that takes hundreds of them, 200 arrivals in the busy slots: many activations per slot
    burst = wl.SimConfig(
        M=1500, K=0, T_max=600, Qcap=900, Acap=1200, seed=44, class_law=wl.constant_table(0),
        prompt=(wl.uniform_table(1, 6),), decode=(wl.uniform_table(1, 5),),
        arrivals=(wl.Arrivals((wl.constant_table(0), wl.constant_table(200)), (1 << 29, 1 << 30)),),
        groups=(wl.Group(wl.POLICY_GREEDY, n_replicas=4), wl.Group(wl.POLICY_FLOW, b_fp=wl.b_to_fp(90.0), n_replicas=4)),
        trace_stride=0, hist_bins=64, hist_shift=0, complog_cap=0)
    ref = orc.run(burst, threads=4)
    assert ref["counters"][:, orc.CIDX["dropped"]].min() > 0 and ref["counters"][:, orc.CIDX["admitted"]].min() > 10000
    assert_same(burst, run_gpu(burst, pieces=[250, 350]), ref, 600, "undrawn arrivals, bursts")
