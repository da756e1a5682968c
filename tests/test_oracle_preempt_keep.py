"""The eviction variant that keeps the generated tokens, (l, o) <- (l + j, o - j), pinned by what it must conserve.

The paper's model refreshes an evicted request (Section 3.3); this variant is an addition, so its pins are
exact consequences of its definition: once the system has drained, every request has delivered exactly its
ORIGINAL output length, and every cache slot-token ever held belonged to a token that was kept, so the total
usage equals the total workload sum of l*o + o(o+1)/2 over the original lengths (the quantity of Prop. 3.2)."""
import numpy as np
import pytest

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl
from pyref import philox_py, sample_py

I = orc.CIDX
M32 = 0xFFFFFFFF


def _draining_config(policy, keep, seed=11, T=2500):
    # arrivals at rate 2 per slot until the modulating chain jumps (probability 1/150 per slot) to a state with no
    # arrivals, from which it never returns: the system then empties
    arr = wl.Arrivals((wl.poisson_table(2.0), wl.constant_table(0)), ((1 << 32) // 150, 0))
    prompt = (wl.uniform_table(1, 6), wl.uniform_table(4, 12))
    decode = (wl.uniform_table(1, 9), wl.geometric_table(6.0, 20))
    grp = wl.Group(policy, b_fp=wl.b_to_fp(5.0), chunk=3, n_replicas=4, m_admit=55, b_class=(3, 2),
                   preempt_keep=keep)
    return wl.SimConfig(M=60, K=0, T_max=T, Qcap=4096, Acap=64, seed=seed, class_law=wl.table_from_pmf(0, [0.6, 0.4]),
                        prompt=prompt, decode=decode, arrivals=(arr,), groups=(grp,), trace_stride=1, hist_bins=0,
                        hist_shift=0, complog_cap=0, name="draining")


def _original_lengths(cfg, replica):
    """(l, o) of every arrival of the run, straight from the generator's definition."""
    key = (cfg.seed & M32, (cfg.seed >> 32) & M32)
    arr = cfg.arrivals[0]
    rid = cfg.groups[0].rng_replica_base + replica
    state, out = 0, []
    for t in range(1, cfg.T_max + 1):
        w = philox_py((t, rid, 0, 0), key)
        if w[2] < arr.switch_thr[state]:
            state ^= 1
        for i in range(sample_py(arr.count[state], w[0])):
            a = philox_py((t, rid, 1, i), key)
            cls = sample_py(cfg.class_law, a[0])
            out.append((sample_py(cfg.prompt[cls], a[1]), sample_py(cfg.decode[cls], a[2])))
    return out


@pytest.mark.parametrize("policy", [wl.POLICY_FLOW, wl.POLICY_GREEDY, wl.POLICY_ALPHA, wl.POLICY_CLASSFLOW])
def test_a_drained_system_has_delivered_every_original_token_and_wasted_nothing(policy):
    cfg = _draining_config(policy, keep=1)
    c = orc.run(cfg)["counters"]
    c0 = orc.run(_draining_config(policy, keep=0))["counters"]
    assert c[:, I["evictions"]].sum() > 10   # the instance does overflow
    for r in range(cfg.n_replicas):
        reqs = _original_lengths(cfg, r)
        assert c[r, I["q_final"]] == 0 and c[r, I["p_final"]] == 0 and c[r, I["dropped"]] == 0
        assert c[r, I["arrived"]] == c[r, I["completed"]] == len(reqs)
        assert c[r, I["completed_tokens"]] == c[r, I["tokens_generated"]] == sum(o for _, o in reqs)
        assert c[r, I["wasted_tokens"]] == 0 and c[r, I["resid_j"]] == 0
        w_total = sum(l * o + o * (o + 1) // 2 for l, o in reqs)
        assert c[r, I["sum_w_completed"]] == w_total == c[r, I["sum_U"]]
        # the paper's own rule on the same arrivals: same workload delivered, the usage also paid for the lost tokens
        # (when it drains too: evict-all with a refresh can repeat the same overflow for ever once arrivals stop)
        if c0[r, I["q_final"]] == 0 and c0[r, I["p_final"]] == 0:
            assert c0[r, I["sum_w_completed"]] == w_total and c0[r, I["completed_tokens"]] == sum(o for _, o in reqs)
            if c0[r, I["wasted_tokens"]] > 0:
                assert c0[r, I["sum_U"]] > w_total and c0[r, I["tokens_generated"]] > c[r, I["tokens_generated"]]
        else:
            assert policy == wl.POLICY_ALPHA
    assert c0[:, I["wasted_tokens"]].sum() > 0


def test_chunked_prefill_loses_only_the_prompt_progress():
    cfg = _draining_config(wl.POLICY_CHUNKED, keep=1)
    c = orc.run(cfg)["counters"]
    assert c[:, I["evictions"]].sum() > 0
    for r in range(cfg.n_replicas):
        reqs = _original_lengths(cfg, r)
        assert c[r, I["completed"]] == len(reqs)
        assert c[r, I["completed_tokens"]] == c[r, I["tokens_generated"]] == sum(o for _, o in reqs)
        w_total = sum(l * o + o * (o + 1) // 2 for l, o in reqs)
        # partially loaded prompts occupy the cache too, so the usage can only exceed the workload
        assert c[r, I["sum_w_completed"]] == w_total <= c[r, I["sum_U"]]


def test_without_evictions_the_variant_changes_nothing():
    a = orc.run(_draining_config(wl.POLICY_GREEDY, keep=1).with_(M=100000, Acap=2048))
    b = orc.run(_draining_config(wl.POLICY_GREEDY, keep=0).with_(M=100000, Acap=2048))
    assert a["counters"][:, I["evictions"]].sum() == 0
    assert (a["counters"] == b["counters"]).all() and (a["trace"] == b["trace"]).all()


def test_the_variant_is_refused_for_the_policy_that_never_evicts():
    cfg = _draining_config(wl.POLICY_MC, keep=1)
    with pytest.raises(Exception):
        orc.run(cfg)
