"""Exact integer identities that every run of the model must satisfy (checker only)."""
import numpy as np
import pytest

from helpers import scaled_presets
from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import workloads as wl

I = orc.CIDX


def check_identities(cfg, out, n_steps):
    c = out["counters"].astype(object)   # Python ints: no overflow in the checks themselves

    def col(n):
        return c[:, I[n]]
    # request conservation: every arrival is dropped, completed, waiting or active
    assert (col("arrived") == col("dropped") + col("completed") + col("q_final") + col("p_final")).all()
    # admission conservation
    assert (col("admitted") == col("completed") + col("evictions") + col("p_final")).all()
    # token conservation
    assert (col("tokens_generated") == col("completed_tokens") + col("wasted_tokens") + col("resid_j")).all()
    # capacity (Section 2.1: U_t <= M for all t)
    assert (col("max_U") <= cfg.M).all()
    # work bound (proof of Prop. 3.2): completed workload <= total KV-time used <= M*T
    assert (col("sum_w_completed") <= col("sum_U")).all()
    assert (col("sum_U") <= cfg.M * n_steps).all()
    # slot-exact Little identity: sum_t N_t = sum of sojourns of the finished + ages of the unfinished
    assert (col("sum_N") == col("sum_lat") + col("resid_age")).all()
    assert (col("steps_done") == n_steps).all()
    if out["trace"] is not None:
        tr = out["trace"]
        assert (tr[:, :, 0] <= cfg.M).all() and (tr[:, :, 0] >= 0).all()
        if cfg.trace_stride == 1:
            assert (tr[:, :, 0].astype(np.int64).sum(axis=1) == out["counters"][:, I["sum_U"]]).all()
            assert (tr[:, :, 0].max(axis=1) == out["counters"][:, I["max_U"]]).all()
            assert (tr[:, :, 1].max(axis=1) == out["counters"][:, I["max_Q"]]).all()
            assert (tr[:, -1, 1] == out["counters"][:, I["q_final"]]).all()
    if out["hist"] is not None:
        assert (out["hist"].astype(np.int64).sum(axis=1) == out["counters"][:, I["completed"]]).all()
    if out["complog"] is not None:
        n = out["counters"][:, I["n_logged"]]
        assert (n == np.minimum(out["counters"][:, I["completed"]], cfg.complog_cap)).all()
        for r in range(c.shape[0]):
            log = out["complog"][r, :n[r]]
            assert (np.diff(log[:, 0]) >= 0).all()
            if n[r] == out["counters"][r, I["completed"]]:
                assert int(log[:, 1].astype(np.int64).sum()) == int(out["counters"][r, I["sum_lat"]])
                if out["hist"] is not None:
                    bins = np.minimum(log[:, 1] >> cfg.hist_shift, cfg.hist_bins - 1)
                    assert (np.bincount(bins, minlength=cfg.hist_bins) == out["hist"][r]).all()


@pytest.mark.parametrize("cfg", scaled_presets(), ids=lambda c: c.name)
def test_identities_on_presets(cfg):
    out = orc.run(cfg, threads=4)
    check_identities(cfg, out, cfg.T_max)
    # the scaled presets exercise what they are meant to exercise
    tot = out["counters"].sum(axis=0)
    assert tot[I["completed"]] > 0 and tot[I["admitted"]] > 0
    if cfg.name.startswith(("cfg1", "cfg2", "cfg5")):
        assert tot[I["evictions"]] > 0 and tot[I["gate_blocked_steps"]] > 0
    if cfg.name.startswith("cfg5"):
        assert out["counters"][:, I["mmpp_state"]].max() <= 1
    assert tot[I["acap_blocked_steps"]] == 0


@pytest.mark.parametrize("seed", range(40))
def test_identities_on_random_tiny_configs(seed):
    cfg = wl.random_small_config(seed, n_replicas=3, T=80)
    out = orc.run(cfg)
    check_identities(cfg, out, cfg.T_max)


@pytest.mark.parametrize("seed", range(6))
def test_identities_on_random_medium_configs(seed):
    cfg = wl.random_medium_config(seed)
    out = orc.run(cfg, threads=4)
    c = out["counters"].astype(object)
    assert (c[:, I["arrived"]] == c[:, I["dropped"]] + c[:, I["completed"]] + c[:, I["q_final"]] + c[:, I["p_final"]]).all()
    assert (c[:, I["sum_N"]] == c[:, I["sum_lat"]] + c[:, I["resid_age"]]).all()
    assert (c[:, I["max_U"]] <= cfg.M).all()


def test_pause_point_extras_are_a_prefix_property():
    # counters of a run stopped after a slots equal a run of a slots: the model is causal
    cfg = wl.config1(replicas=4, T=600)
    a = orc.run(cfg, n_steps=250)
    full = orc.run(cfg, n_steps=600)
    assert (a["trace"] == full["trace"][:, :250]).all()
    check_identities(cfg, a, 250)


def test_sanitized_build_runs_clean():
    # address/UB-sanitised build of the checker on a config that evicts, drops and logs
    import subprocess, sys, os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import ctypes,sys; sys.path.insert(0,%r); sys.path.insert(0,%r)\n"
            "from oracle import fcsim_oracle as orc\n"
            "from paper_2604_11001_b200 import workloads as wl\n"
            "import numpy as np\n"
            "a = orc.run(wl.config1(replicas=2, T=500), sanitize=True)\n"
            "b = orc.run(wl.config1(replicas=2, T=500))\n"
            "assert (a['counters'] == b['counters']).all()\n"
            "for s in range(6):\n"
            "    orc.run(wl.random_small_config(s, 2, 60), sanitize=True)\n"
            "print('ok')\n") % (root, os.path.join(root, "tests"))
    import glob
    asan = glob.glob("/usr/lib/gcc/x86_64-linux-gnu/*/libasan.so")
    if not asan:
        pytest.skip("libasan not installed")
    env = dict(os.environ, LD_PRELOAD=asan[0], ASAN_OPTIONS="detect_leaks=0")
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "ok" in res.stdout, res.stderr[-2000:]
