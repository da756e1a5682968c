"""The checker against an independent pure-Python evaluator on random tiny instances."""
import numpy as np
import pytest

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl
from pyref import brute_force

I = orc.CIDX


@pytest.mark.parametrize("seed", range(30))
def test_brute_force_agreement(seed):
    cfg = wl.random_small_config(1000 + seed, n_replicas=2, T=50)
    out = orc.run(cfg.with_(trace_stride=1, complog_cap=512))
    for r in range(cfg.n_replicas):
        bf = brute_force(cfg, r, cfg.T_max)
        assert out["trace"][r, :, 0].tolist() == bf["U"]
        assert out["trace"][r, :, 1].tolist() == bf["Q"]
        n = int(out["counters"][r, I["n_logged"]])
        assert [tuple(x) for x in out["complog"][r, :n].tolist()] == bf["completions"]
        for k, v in bf["counters"].items():
            assert int(out["counters"][r, I[k]]) == v, (k, r)


def test_random_configs_cover_every_branch():
    tot = np.zeros(orc.N_COUNTERS, dtype=np.int64)
    keep_ev = np.zeros(6, dtype=np.int64)   # evictions under the keep-the-tokens variant, per policy
    for seed in range(30):
        cfg = wl.random_small_config(1000 + seed, n_replicas=2, T=50)
        c = orc.run(cfg)["counters"]
        tot += c.sum(axis=0)
        for g, grp in enumerate(cfg.groups):
            if grp.preempt_keep:
                keep_ev[grp.policy] += c[2 * g:2 * g + 2, I["evictions"]].sum()
                assert c[2 * g:2 * g + 2, I["wasted_tokens"]].sum() == 0
    assert (keep_ev[:5] > 0).all(), keep_ev
    for name in ("dropped", "evictions", "gate_blocked_steps", "budget_blocked_steps", "acap_blocked_steps",
                 "wasted_tokens", "completed", "mmpp_state"):
        assert tot[I[name]] > 0, name
