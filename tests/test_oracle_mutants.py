"""Do the checker's pins bite?  One planted mistake at a time.

Each mutant is a copy of oracle/fcsim_oracle.cpp with one small, plausible mistake (a dropped term, an off-by-one,
swapped draws, a wrong order, an ignored limit).  The copy is built in a temporary directory and the checker's own
pin tests (tests/test_oracle_*.py) are run against it in a child process; every mutant must fail at least one
of them.  The mistakes are planted in the CPU checker only.
"""
import os
import shutil
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ORACLE = os.path.join(ROOT, "oracle")
PIN_FILES = ["test_oracle_traces.py", "test_oracle_closed_forms.py", "test_oracle_invariants.py",
             "test_oracle_rng.py", "test_oracle_bruteforce.py", "test_oracle_reductions.py",
             "test_oracle_preempt_keep.py", "test_oracle_stability.py"]

# (name, text in the checker, replacement): the text must occur exactly once
MUTANTS = [
    ("philox key schedule constant", "k0 += 0x9E3779B9u;", "k0 += 0xBB67AE85u;"),
    ("philox mixes the wrong product half", "const uint32_t n0 = hi1 ^ c1 ^ k0,", "const uint32_t n0 = hi0 ^ c1 ^ k0,"),
    ("sampler takes u <= threshold", "std::upper_bound(first, last, u)", "std::lower_bound(first, last, u)"),
    ("arrival state starts at 1", "uint32_t s = 0;  // state of the modulated arrival law", "uint32_t s = 1;"),
    ("arrival state switches with the wrong word", "w[2] < arr.switch_thr[s]", "w[3] < arr.switch_thr[s]"),
    ("count drawn before the switch test",
     "        if (arr.n_states == 2 && w[2] < arr.switch_thr[s]) s ^= 1u;\n"
     "        const int32_t n_t = fcsim_oracle_sample(&arr.count[s], w[0]);",
     "        const int32_t n_t = fcsim_oracle_sample(&arr.count[s], w[0]);\n"
     "        if (arr.n_states == 2 && w[2] < arr.switch_thr[s]) s ^= 1u;"),
    ("budget drawn from the count's word", "(((w[1] >> 16) < (grp.b_fp & 0xffffu)) ? 1 : 0)",
     "(((w[0] >> 16) < (grp.b_fp & 0xffffu)) ? 1 : 0)"),
    ("prompt and decode words swapped",
     "r.l = fcsim_oracle_sample(&cfg.prompt[r.cls], a[1]);\n            r.o = fcsim_oracle_sample(&cfg.decode[r.cls], a[2]);",
     "r.l = fcsim_oracle_sample(&cfg.prompt[r.cls], a[2]);\n            r.o = fcsim_oracle_sample(&cfg.decode[r.cls], a[1]);"),
    ("waiting room holds one more", "if ((int64_t)Q.size() >= (int64_t)cfg.Qcap) {", "if ((int64_t)Q.size() > (int64_t)cfg.Qcap) {"),
    ("arrival stamped one slot early", "r.t_arr = t;", "r.t_arr = t - 1;"),
    ("prospective usage forgets the new tokens", "int64_t G = U_in + Ndec;", "int64_t G = U_in;"),
    ("chunked budget not decode-first", "std::max<int64_t>(0, cfg.K - Ndec)", "(int64_t)cfg.K"),
    ("last chunk brings no token", "if (r.p == r.l) G += 1;  // prefill done: first output token this slot", ""),
    ("one activation too many per slot", "const int64_t cap = classflow ? 0 : (flow ? B_t : INF);",
     "const int64_t cap = classflow ? 0 : (flow ? B_t + 1 : INF);"),
    ("first admission not exempt from the token budget",
     "                if (!(cfg.K == 0 || a == 0 || g <= R)) { C[C_BUDGET_BLOCKED]++; break; }\n                need = (int64_t)h.l + 1;",
     "                if (!(cfg.K == 0 || g <= R)) { C[C_BUDGET_BLOCKED]++; break; }\n                need = (int64_t)h.l + 1;"),
    ("gate refuses an exact fit", "if (G + need > admit_limit) { C[C_GATE_BLOCKED]++; break; }",
     "if (G + need >= admit_limit) { C[C_GATE_BLOCKED]++; break; }"),
    ("gate ignores the first token", "if (G + need > admit_limit) { C[C_GATE_BLOCKED]++; break; }",
     "if (G + need - 1 > admit_limit) { C[C_GATE_BLOCKED]++; break; }"),
    ("oldest evicted instead of newest", "Request r = P.back();\n                P.pop_back();",
     "Request r = P.front();\n                P.erase(P.begin());"),
    ("evicted requests join the tail", "Q.push_front(r);", "Q.push_back(r);"),
    ("eviction goes one request too far", "while (alpha ? !P.empty() : G > M) {", "while (alpha ? !P.empty() : G >= M) {"),
    ("alpha-protection evicts only until it fits", "while (alpha ? !P.empty() : G > M) {", "while (G > M) {"),
    ("alpha-protection limit ignored", "const int64_t admit_limit = alpha ? (int64_t)grp.m_admit : M;",
     "const int64_t admit_limit = M;"),
    ("wasted tokens not counted", "C[C_WASTED_TOKENS] += r.j;", "C[C_WASTED_TOKENS] += 0;"),
    ("eviction releases one token too few", "G -= (int64_t)r.p + r.j + (r.p == r.l ? 1 : 0);", "G -= (int64_t)r.p + r.j;"),
    ("request leaves one token early", "if (r.p == r.l && r.j == r.o) {", "if (r.p == r.l && r.j + 1 >= r.o) {"),
    ("latency without the arrival slot", "const int64_t lat = (int64_t)t - r.t_arr + 1;", "const int64_t lat = (int64_t)t - r.t_arr;"),
    ("workload formula off by o", "C[C_SUM_W_COMPLETED] += (int64_t)r.l * r.o + (int64_t)r.o * (r.o + 1) / 2;",
     "C[C_SUM_W_COMPLETED] += (int64_t)r.l * r.o + (int64_t)r.o * (r.o - 1) / 2;"),
    ("histogram bin without the shift", "hist[std::min<int64_t>(lat >> cfg.hist_shift, cfg.hist_bins - 1)]++;",
     "hist[std::min<int64_t>(lat, cfg.hist_bins - 1)]++;"),
    ("trace records the active count as queue length", "trace[2 * rec + 1] = (int32_t)Q.size();",
     "trace[2 * rec + 1] = (int32_t)P.size();"),
    ("sum_N without the active set", "C[C_SUM_N] += (int64_t)P.size() + (int64_t)Q.size();", "C[C_SUM_N] += (int64_t)Q.size();"),
    ("Algorithm 1 picks the queue head of any class", "while (it != Q.end() && it->cls != k) ++it;", ""),
    ("Algorithm 1 stops at the first refused class", "if (G + need > M) { gate_hit = true; break; }",
     "if (G + need > M) { gate_hit = true; storage_hit = true; break; }"),
    ("MC projection skips the last slot", "if (tau <= last) usage += (int64_t)r.l + r.j + (tau - t + 1);",
     "if (tau < last) usage += (int64_t)r.l + r.j + (tau - t + 1);"),
    ("MC projection forgets this slot's token", "if (tau <= last) usage += (int64_t)r.l + r.j + (tau - t + 1);",
     "if (tau <= last) usage += (int64_t)r.l + r.j + (tau - t);"),
    ("MC projects with the true length in worst-case mode",
     "if (mc && grp.mc_worst_case) r.o_proj = cfg.decode[r.cls].vmin + (int32_t)cfg.decode[r.cls].n - 1;", ""),
    ("kept tokens do not join the prompt", "                    r.l += r.j;\n", ""),
    ("kept tokens are generated again", "                    r.o -= r.j;\n", ""),
    ("kept tokens not delivered", "C[C_COMPLETED_TOKENS] += r.j;", "C[C_COMPLETED_TOKENS] += 0;"),
    ("banked workload of the kept tokens", "C[C_SUM_W_COMPLETED] += (int64_t)r.l * r.j + (int64_t)r.j * (r.j + 1) / 2;",
     "C[C_SUM_W_COMPLETED] += (int64_t)r.l * r.j + (int64_t)r.j * (r.j - 1) / 2;"),
    ("residual age without the current slot", "for (const Request& r : Q) C[C_RESID_AGE] += (int64_t)n_steps - r.t_arr + 1;",
     "for (const Request& r : Q) C[C_RESID_AGE] += (int64_t)n_steps - r.t_arr;"),
]


def _survives(args):
    """Build one mutant and run the pins on it; returns (name, outcome) with outcome 'killed', 'survived' or an error."""
    name, old, new, src = args
    if src.count(old) != 1:
        return name, "text occurs %d times in the checker" % src.count(old)
    tmp = tempfile.mkdtemp(prefix="fcsim_mutant_")
    try:
        pkg = os.path.join(tmp, "oracle")
        os.makedirs(pkg)
        for f in ("__init__.py", "build.py", "fcsim_oracle.py"):
            shutil.copy(os.path.join(ORACLE, f), pkg)
        with open(os.path.join(pkg, "fcsim_oracle.cpp"), "w") as f:
            f.write(src.replace(old, new))
        cc = subprocess.run(["g++", "-std=c++17", "-O1", "-shared", "-fPIC", os.path.join(pkg, "fcsim_oracle.cpp"),
                             "-o", os.path.join(pkg, "libfcsim_oracle.so")], capture_output=True, text=True)
        if cc.returncode != 0:
            return name, "does not compile: " + cc.stderr[-300:]
        env = dict(os.environ, FCSIM_ORACLE_ROOT=tmp)
        run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", "-m",
                              "not gpu and not mutation"] + [os.path.join(ROOT, "tests", f) for f in PIN_FILES],
                             capture_output=True, text=True, env=env, cwd=tmp, timeout=900)
        if run.returncode == 1 or run.returncode < 0:   # a test failed, or the mutant crashed the test process
            return name, "killed"
        if run.returncode == 0:
            return name, "survived"
        return name, "pytest error %d: %s" % (run.returncode, (run.stdout + run.stderr)[-300:])
    finally:
        shutil.rmtree(tmp, ignore_errors=True)


@pytest.mark.mutation
def test_every_planted_mistake_fails_a_pin():
    with open(os.path.join(ORACLE, "fcsim_oracle.cpp")) as f:
        src = f.read()
    with ThreadPoolExecutor(max_workers=max(2, (os.cpu_count() or 2))) as ex:
        results = list(ex.map(_survives, [(n, o, r, src) for n, o, r in MUTANTS]))
    bad = [(n, r) for n, r in results if r != "killed"]
    assert not bad, bad
    assert len(results) >= 40
