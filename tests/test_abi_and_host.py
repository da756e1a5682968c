"""CPU-only checks of the boundary: exported symbols, struct layout, host-side validation."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2604_11001_b200 import binding as fb
from paper_2604_11001_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fcsim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fcsim_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = fb.load()
    names = declared_functions()
    assert "fcsim_create" in names and "fcsim_run" in names and "fcsim_stats" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(fb.EXPORTS) == names


def test_counter_block_is_28_int64():
    assert C.sizeof(fb.fcsim_counters) == 28 * 8
    assert C.sizeof(fb.fcsim_summary) == 28 * 8 + 6 * 8 + 8
    assert fb.COUNTER_NAMES[0] == "steps_done" and fb.COUNTER_NAMES[-1] == "mmpp_state"


def test_query_sizes_of_the_presets():
    s = fb.fcsim_query_sizes(wl.config1())
    assert s["counters"] == 64 * 224
    assert s["trace"] == 64 * 2000 * 8
    assert s["hist"] == 64 * 1024 * 4
    assert s["complog"] == 64 * 2048 * 8
    # per replica: 16 header words, the active ring (Acap entries of 8 + 4 bytes), the queue ring (next power of two
    # >= Qcap + Acap entries of 8 bytes)
    assert s["workspace"] == 64 * (64 + 256 * 12 + 512 * 8)
    s5 = fb.fcsim_query_sizes(wl.config5())
    assert s5["trace"] == 0 and s5["complog"] == 0 and s5["hist"] == 262144 * 1024 * 4


def _expect(cfg, code):
    with pytest.raises(fb.FcsimError) as e:
        fb.fcsim_query_sizes(cfg)
    assert e.value.code == code


def test_invalid_configurations_are_refused():
    base = wl.config1(replicas=2, T=100)
    _expect(base.with_(M=0), -1)
    _expect(base.with_(M=100), -1)                      # max l + max o = 128 + 512 > M
    _expect(base.with_(T_max=1 << 24), -1)
    _expect(base.with_(Qcap=0), -1)
    _expect(base.with_(decode=(wl.Table(0, np.array([5, 9], dtype=np.uint32)),)), -1)   # o = 0 possible
    _expect(base.with_(prompt=(wl.Table(1, np.array([9, 5, 7], dtype=np.uint32)),)), -1)  # not monotone
    _expect(base.with_(groups=(wl.Group(3, n_replicas=1),)), -1)
    _expect(base.with_(groups=(wl.Group(wl.POLICY_CHUNKED, chunk=0, n_replicas=1),)), -1)
    _expect(base.with_(groups=(wl.Group(wl.POLICY_FLOW, arrivals_id=1, n_replicas=1),)), -1)
    _expect(base.with_(arrivals=(wl.Arrivals((wl.Table(0, np.arange(1, 301, dtype=np.uint32) * 1000),)),)), -1)
    _expect(base.with_(hist_shift=31), -1)
    _expect(base.with_(Qcap=20000, Acap=20000), -2)      # does not fit the shared memory of one warp
    assert fb.fcsim_strerror(-2).startswith("Qcap")
    assert fb.fcsim_strerror(0) == "ok"


def test_create_without_buffers_is_an_error_not_a_crash():
    # no GPU needed: validation of the buffer table comes before any CUDA call
    cfg = wl.config1(replicas=2, T=100)
    with pytest.raises(fb.FcsimError) as e:
        fb.fcsim_create(cfg, {})
    assert e.value.code == -3
    with pytest.raises(fb.FcsimError) as e:
        fb.fcsim_create(cfg, {"workspace": 16, "counters": 16, "scratch": 8, "trace": 16, "hist": 16, "complog": 16})
    assert e.value.code == -3   # misaligned scratch


def test_null_handles_are_refused():
    lib = fb.load()
    assert lib.fcsim_run(None, 1, None) == -1
    assert lib.fcsim_stats(None, None, None, None) == -1
    assert lib.fcsim_destroy(None) == -1
    assert lib.fcsim_steps_done(None) == -1
