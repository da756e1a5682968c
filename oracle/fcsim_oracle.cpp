// TEST INFRASTRUCTURE -- not part of the product path.
//
// Plain, slow, single-threaded CPU simulator of the token-level serving model of
// Section 2.1 driven by the flow-controlled policy of Algorithm 2 (and by the greedy
// prefill-first and chunked-prefill baselines named in the Introduction, and the alpha-protection
// greedy baseline described in Section 4.1; optionally with a preemption that keeps the generated
// tokens, a variant the paper does not have).  It is
// written directly from the paper, one request object at a time, with a std::deque
// waiting queue and a std::vector active set; the KV usage U_t is re-summed from the
// request objects every slot.  It shares no code, header or table with the CUDA
// library.  Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
//
// Every random word comes from Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) keyed by
// the seed, with counter (slot t, replica id, stream, index); tables are integer
// inverse-CDF thresholds passed in by the caller.
//
// Pins (tests/test_oracle_*.py): published Philox known-answer vectors; hand-traced
// instances of the model (tests/golden); request/admission/token conservation; U_t <= M
// (Section 2.1); sum of completed workloads <= sum U_t <= M*T (proof of Prop. 3.2);
// the slot-exact Little identity; the queue recursion Q_t = (Q_{t-1}+n_t-b)^+ (proof of
// Thm. 3.3); the double-sum form of U_t (proof of Thm. 3.6); b -> infinity equals greedy
// (Section 3.3); the stability dichotomy of Prop. 3.5 / Thm. 3.6; an independent
// brute-force evaluator on tiny inputs.
// The MC benchmark's future-memory test (Section 4.1) is evaluated slot by slot; a last-slots-only
// shortcut exists as an opt-in mode and a test compares the two on every admission decision.
// Parity unpinned against the paper (the paper only names them; pinned by hand traces
// and reductions only): the token budget K, GREEDY, CHUNKED and the two-state arrival law.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <deque>
#include <limits>
#include <vector>

extern "C" {

struct orc_table {
    uint32_t n;
    int32_t vmin;
    const uint32_t* cdf;
};
struct orc_arrivals {
    uint32_t n_states;
    orc_table count[2];
    uint32_t switch_thr[2];
};
struct orc_group {
    int32_t policy;  // 0 FLOW, 1 GREEDY, 2 CHUNKED, 3 ALPHA (alpha-protection greedy, Section 4.1),
                     // 4 CLASSFLOW (Algorithm 1: per-class budgets b_k, FIFO within a class),
                     // 5 MC (memory-constrained first-come-first-served benchmark of Section 4.1)
    uint32_t b_fp;
    int32_t chunk;
    int32_t arrivals_id;
    uint32_t rng_replica_base;
    int32_t n_replicas;
    int32_t m_admit;  // ALPHA: a new prompt is admitted only while usage stays <= m_admit = (1-alpha) M
    const int32_t* b_class;  // CLASSFLOW (policy 4, Algorithm 1): activation budget b_k of every class
    int32_t mc_worst_case;   // MC: 0 = output lengths known, 1 = every request is projected with the longest
                             //     output length of its class (the unknown-length adaptation of Section 4.1)
    int32_t preempt_keep;    // what an evicted request loses.  0 = everything (the model of Sections 2.1 and 3.3:
                             //     the request is "refreshed").  1 = only its place in the cache: the j tokens it
                             //     has generated are kept and become part of its prompt, (l, o) <- (l + j, o - j);
                             //     this variant is not in the paper (recompute-style preemption of serving engines)
};
struct orc_config {
    int32_t M, K, T_max, Qcap, Acap;
    uint64_t seed;
    int32_t n_classes;
    orc_table class_law;
    const orc_table* prompt;
    const orc_table* decode;
    int32_t n_arrivals;
    const orc_arrivals* arrivals;
    int32_t n_groups;
    const orc_group* groups;
    int32_t trace_stride, hist_bins, hist_shift, complog_cap;
};
// All arrays are host memory, row r = replica (first_replica + r).  NULL = not wanted.
struct orc_outputs {
    int64_t* counters;   // [n][28]
    int32_t* trace;      // [n][n_steps/stride][2] = {U_t, |Q_t|}
    int32_t* hist;       // [n][hist_bins]
    int32_t* complog;    // [n][complog_cap][2] = {t_done, latency}
    int32_t* arrlog;     // [n][n_steps]  n_t of every slot                    (diagnostic)
    int32_t* arrcls;     // [n][n_steps][n_classes] arrivals of every class     (diagnostic)
    int32_t* admlog;     // [n][admlog_cap][4] = {slot, l, o, t_arr} per admission (diagnostic)
    int64_t admlog_cap;
    int64_t* n_admlog;   // [n]
};

enum {
    C_STEPS_DONE = 0, C_STATUS, C_ARRIVED, C_DROPPED, C_ADMITTED, C_COMPLETED, C_EVICTIONS,
    C_OVERFLOW_STEPS, C_GATE_BLOCKED, C_BUDGET_BLOCKED, C_ACAP_BLOCKED, C_TOKENS_GENERATED,
    C_PREFILL_TOKENS, C_COMPLETED_TOKENS, C_WASTED_TOKENS, C_SUM_LAT, C_MAX_LAT, C_SUM_U, C_MAX_U,
    C_SUM_N, C_MAX_Q, C_SUM_W_COMPLETED, C_N_LOGGED, C_Q_FINAL, C_P_FINAL, C_RESID_AGE, C_RESID_J,
    C_MMPP_STATE, C_COUNT
};

// Philox4x32-10, from its published definition: ten rounds of
//   (hi0,lo0) = 0xD2511F53 * c0,  (hi1,lo1) = 0xCD9E8D57 * c2,
//   (c0,c1,c2,c3) <- (hi1^c1^k0, lo1, hi0^c3^k1, lo0),
// the key bumped by (0x9E3779B9, 0xBB67AE85) between rounds.
void fcsim_oracle_philox(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// vmin + min{k < n-1 : u < cdf[k]}, else vmin+n-1.  std::upper_bound on the first n-1
// thresholds returns exactly that k for a non-decreasing table.
int32_t fcsim_oracle_sample(const orc_table* tab, uint32_t u) {
    const uint32_t* first = tab->cdf;
    const uint32_t* last = tab->cdf + (tab->n - 1);
    return tab->vmin + (int32_t)(std::upper_bound(first, last, u) - first);
}

}  // extern "C"

namespace {

constexpr uint32_t STREAM_STEP = 0;
constexpr uint32_t STREAM_ARR = 1;

struct Request {
    int64_t id;
    int32_t cls, l, o, t_arr;
    int32_t o_proj;  // output length assumed when future memory is projected (MC benchmark)
    int32_t p;  // prompt tokens in the cache
    int32_t j;  // output tokens generated
};

// MC benchmark (Section 4.1): a waiting request is started only if the memory usage of every future slot
// stays within the limit.  The future is the one in which nothing else is started: every running request
// and the candidate h (started in slot t) generate one token per slot until their (projected) last token.
// A request that has generated j tokens before slot t holds l + j + (tau - t + 1) tokens in slot tau >= t,
// up to and including the slot of its last token, t + (o_proj - j) - 1, and nothing afterwards.
// The test walks the future slot by slot until everything has ended and sums the footprints in each slot.
bool fits_future(const std::vector<Request>& P, const Request& h, int32_t t, int64_t M) {
    std::vector<Request> all(P);
    Request c = h;
    c.p = c.l;
    c.j = 0;
    all.push_back(c);
    int64_t horizon = t;  // last slot in which anything is still running
    for (const Request& r : all) horizon = std::max<int64_t>(horizon, (int64_t)t + (r.o_proj - r.j) - 1);
    for (int64_t tau = t; tau <= horizon; ++tau) {
        int64_t usage = 0;
        for (const Request& r : all) {
            const int64_t last = (int64_t)t + (r.o_proj - r.j) - 1;
            if (tau <= last) usage += (int64_t)r.l + r.j + (tau - t + 1);
        }
        if (usage > M) return false;
    }
    return true;
}

// Opt-in shortcut of the same test (mc_mode 1; mc_mode 2 evaluates both and reports a disagreement): between
// two endings the usage only grows, one token per running request and slot, so the maximum over the future is
// reached in some request's last slot and only those slots need to be summed.  A test compares the two on
// every admission decision of a set of random configurations.
bool fits_future_last_slots(const std::vector<Request>& P, const Request& h, int32_t t, int64_t M) {
    std::vector<Request> all(P);
    Request c = h;
    c.p = c.l;
    c.j = 0;
    all.push_back(c);
    for (const Request& e : all) {
        const int64_t tau = (int64_t)t + (e.o_proj - e.j) - 1;  // last slot of e
        int64_t usage = 0;
        for (const Request& r : all) {
            const int64_t r_end = (int64_t)t + (r.o_proj - r.j) - 1;
            if (r_end >= tau) usage += (int64_t)r.l + r.j + (tau - t + 1);
        }
        if (usage > M) return false;
    }
    return true;
}

int64_t kv_usage(const std::vector<Request>& P) {
    int64_t u = 0;
    for (const Request& r : P) u += r.p + r.j;
    return u;
}

int check_table(const orc_table& t, int32_t min_vmin) {
    if (t.n == 0 || t.cdf == nullptr || t.vmin < min_vmin) return -1;
    for (uint32_t k = 1; k + 1 < t.n; ++k)
        if (t.cdf[k] < t.cdf[k - 1]) return -1;
    return 0;
}

int validate(const orc_config& c) {
    if (c.M < 1 || c.K < 0 || c.T_max < 1 || c.Qcap < 1 || c.Acap < 1) return -1;
    if (c.n_classes < 1 || c.n_arrivals < 1 || c.n_groups < 1) return -1;
    if (check_table(c.class_law, 0) || c.class_law.vmin != 0 || (int32_t)c.class_law.n != c.n_classes) return -1;
    int32_t lmax = 0, omax = 0;
    for (int k = 0; k < c.n_classes; ++k) {
        if (check_table(c.prompt[k], 1) || check_table(c.decode[k], 1)) return -1;
        lmax = std::max<int32_t>(lmax, c.prompt[k].vmin + (int32_t)c.prompt[k].n - 1);
        omax = std::max<int32_t>(omax, c.decode[k].vmin + (int32_t)c.decode[k].n - 1);
    }
    if ((int64_t)lmax + omax > c.M) return -1;
    for (int a = 0; a < c.n_arrivals; ++a) {
        if (c.arrivals[a].n_states != 1 && c.arrivals[a].n_states != 2) return -1;
        for (uint32_t s = 0; s < c.arrivals[a].n_states; ++s)
            if (check_table(c.arrivals[a].count[s], 0)) return -1;
    }
    for (int g = 0; g < c.n_groups; ++g) {
        const orc_group& G = c.groups[g];
        if (G.policy < 0 || G.policy > 5 || G.n_replicas < 1) return -1;
        if (G.policy == 5 && (G.mc_worst_case < 0 || G.mc_worst_case > 1)) return -1;
        if (G.preempt_keep < 0 || G.preempt_keep > 1) return -1;
        if (G.preempt_keep && G.policy == 5) return -1;  // the MC benchmark never overflows: nothing to keep
        if (G.policy == 4) {
            if (!G.b_class) return -1;
            for (int k = 0; k < c.n_classes; ++k)
                if (G.b_class[k] < 0 || G.b_class[k] > 65535) return -1;
        }
        if (G.policy == 3 && (G.m_admit < 1 || G.m_admit > c.M)) return -1;
        if (G.arrivals_id < 0 || G.arrivals_id >= c.n_arrivals) return -1;
        if (G.policy == 2 && G.chunk < 1) return -1;
    }
    if (c.trace_stride < 0 || c.hist_bins < 0 || c.hist_shift < 0 || c.hist_shift > 30 || c.complog_cap < 0) return -1;
    return 0;
}

// One replica, slots 1..n_steps.  Returns 0, or a negative code if an invariant of the
// model is violated (that would be a bug in this file, not a property of the inputs).
int run_replica(const orc_config& cfg, const orc_group& grp, uint32_t rng_replica, int32_t n_steps,
                int64_t* C, int32_t* trace, int32_t* hist, int32_t* complog, int32_t* arrlog, int32_t* arrcls,
                int32_t* admlog, int64_t admlog_cap, int64_t* n_admlog_out, int mc_mode, int64_t* n_mc_tests) {
    const uint32_t key[2] = {(uint32_t)(cfg.seed & 0xffffffffu), (uint32_t)(cfg.seed >> 32)};
    const orc_arrivals& arr = cfg.arrivals[grp.arrivals_id];
    const int64_t INF = std::numeric_limits<int64_t>::max() / 4;
    const bool flow = grp.policy == 0, chunked = grp.policy == 2, alpha = grp.policy == 3;
    const bool classflow = grp.policy == 4, mc = grp.policy == 5;
    const int64_t M = cfg.M;
    // alpha-protection greedy (Section 4.1): a new prompt with initial memory l+1 joins only if the usage
    // stays within (1-alpha) M; every other policy admits up to the capacity itself
    const int64_t admit_limit = alpha ? (int64_t)grp.m_admit : M;

    std::deque<Request> Q;
    std::vector<Request> P;
    uint32_t s = 0;  // state of the modulated arrival law
    int64_t next_id = 0, n_admlog = 0;
    bool complog_overflow = false;
    std::memset(C, 0, sizeof(int64_t) * C_COUNT);

    for (int32_t t = 1; t <= n_steps; ++t) {
        // ---- A: this slot's draws; arrivals join the waiting queue (Alg. 2: Q <- Q u A_t)
        uint32_t w[4];
        {
            const uint32_t ctr[4] = {(uint32_t)t, rng_replica, STREAM_STEP, 0u};
            fcsim_oracle_philox(ctr, key, w);
        }
        if (arr.n_states == 2 && w[2] < arr.switch_thr[s]) s ^= 1u;
        const int32_t n_t = fcsim_oracle_sample(&arr.count[s], w[0]);
        const int64_t B_t = (int64_t)(grp.b_fp >> 16) + (((w[1] >> 16) < (grp.b_fp & 0xffffu)) ? 1 : 0);
        if (arrlog) arrlog[t - 1] = n_t;
        for (int32_t i = 0; i < n_t; ++i) {
            uint32_t a[4];
            const uint32_t ctr[4] = {(uint32_t)t, rng_replica, STREAM_ARR, (uint32_t)i};
            fcsim_oracle_philox(ctr, key, a);
            Request r;
            r.cls = fcsim_oracle_sample(&cfg.class_law, a[0]);
            r.l = fcsim_oracle_sample(&cfg.prompt[r.cls], a[1]);
            r.o = fcsim_oracle_sample(&cfg.decode[r.cls], a[2]);
            r.t_arr = t;
            r.p = 0;
            r.j = 0;
            r.o_proj = r.o;
            if (mc && grp.mc_worst_case) r.o_proj = cfg.decode[r.cls].vmin + (int32_t)cfg.decode[r.cls].n - 1;
            if (arrcls) arrcls[(int64_t)(t - 1) * cfg.n_classes + r.cls]++;
            C[C_ARRIVED]++;
            if ((int64_t)Q.size() >= (int64_t)cfg.Qcap) {
                C[C_DROPPED]++;
            } else {
                r.id = next_id++;
                Q.push_back(r);
            }
        }

        // ---- B: usage carried into the slot, and the usage it would reach after one more
        //         token per decoding request (Section 2.1: footprint l_i + j_i(t))
        const int64_t U_in = kv_usage(P);
        int64_t Ndec = 0;
        for (const Request& r : P) Ndec += (r.p == r.l);
        int64_t G = U_in + Ndec;
        int64_t R = (cfg.K == 0) ? INF : (chunked ? std::max<int64_t>(0, cfg.K - Ndec) : cfg.K);

        // ---- C: chunked prefill: partially prefilled requests continue, in activation order
        if (chunked) {
            for (Request& r : P) {
                if (r.p < r.l) {
                    const int64_t g = std::min<int64_t>({(int64_t)grp.chunk, (int64_t)(r.l - r.p), R});
                    r.p += (int32_t)g;
                    if (R != INF) R -= g;
                    G += g;
                    C[C_PREFILL_TOKENS] += g;
                    if (r.p == r.l) G += 1;  // prefill done: first output token this slot
                }
            }
        }

        // ---- D: activation, FIFO, at most B_t requests under flow control (Alg. 2 inner loop)
        int64_t a = 0;
        const int64_t cap = classflow ? 0 : (flow ? B_t : INF);
        if (classflow) {
            // Algorithm 1: for every class k, activate up to b_k waiting requests of that class, first
            // come first served within the class.  A pick that does not fit the cache (or the token
            // budget) ends the loop of its class only; a full active-set storage ends the slot's activation.
            bool gate_hit = false, budget_hit = false, storage_hit = false;
            for (int32_t k = 0; k < cfg.n_classes && !storage_hit; ++k) {
                for (int32_t ak = 0; ak < grp.b_class[k]; ++ak) {
                    auto it = Q.begin();
                    while (it != Q.end() && it->cls != k) ++it;
                    if (it == Q.end()) break;
                    if ((int64_t)P.size() == (int64_t)cfg.Acap) { storage_hit = true; break; }
                    Request h = *it;
                    const int64_t g = h.l, need = (int64_t)h.l + 1;
                    if (!(cfg.K == 0 || a == 0 || g <= R)) { budget_hit = true; break; }
                    if (G + need > M) { gate_hit = true; break; }
                    Q.erase(it);
                    h.p = (int32_t)g;
                    h.j = 0;
                    P.push_back(h);
                    G += need;
                    if (R != INF) R -= std::min(g, R);
                    a++;
                    C[C_ADMITTED]++;
                    C[C_PREFILL_TOKENS] += g;
                    if (admlog && n_admlog < admlog_cap) {
                        int32_t* e = admlog + 4 * n_admlog;
                        e[0] = t; e[1] = h.l; e[2] = h.o; e[3] = h.t_arr;
                    }
                    n_admlog++;
                }
            }
            C[C_GATE_BLOCKED] += gate_hit;
            C[C_BUDGET_BLOCKED] += budget_hit;
            C[C_ACAP_BLOCKED] += storage_hit;
        }
        while (a < cap && !Q.empty()) {
            if ((int64_t)P.size() == (int64_t)cfg.Acap) { C[C_ACAP_BLOCKED]++; break; }
            Request h = Q.front();
            int64_t g, need;
            if (chunked) {
                g = std::min<int64_t>({(int64_t)grp.chunk, (int64_t)h.l, R});
                if (g == 0) { C[C_BUDGET_BLOCKED]++; break; }
                need = g + (g == h.l ? 1 : 0);
            } else {
                g = h.l;
                if (!(cfg.K == 0 || a == 0 || g <= R)) { C[C_BUDGET_BLOCKED]++; break; }
                need = (int64_t)h.l + 1;
            }
            if (G + need > admit_limit) { C[C_GATE_BLOCKED]++; break; }
            if (mc) {
                bool fits;
                if (mc_mode == 1) {
                    fits = fits_future_last_slots(P, h, t, M);
                } else {
                    fits = fits_future(P, h, t, M);
                    if (mc_mode == 2 && fits != fits_future_last_slots(P, h, t, M)) return -20;
                }
                if (n_mc_tests) ++*n_mc_tests;
                if (!fits) { C[C_GATE_BLOCKED]++; break; }
            }
            Q.pop_front();
            h.p = (int32_t)g;
            h.j = 0;
            P.push_back(h);
            G += need;
            if (R != INF) R -= std::min(g, R);
            a++;
            C[C_ADMITTED]++;
            C[C_PREFILL_TOKENS] += g;
            if (admlog && n_admlog < admlog_cap) {
                int32_t* e = admlog + 4 * n_admlog;
                e[0] = t; e[1] = h.l; e[2] = h.o; e[3] = h.t_arr;
            }
            n_admlog++;
        }

        // ---- E: overflow: evict last-in-first-out, refreshed, back to the queue front
        if (G > M) {
            C[C_OVERFLOW_STEPS]++;
            // alpha-protection greedy evicts all active requests on overflow; the others evict
            // last-in-first-out only until the slot fits
            while (alpha ? !P.empty() : G > M) {
                if (P.empty()) return -10;
                Request r = P.back();
                P.pop_back();
                G -= (int64_t)r.p + r.j + (r.p == r.l ? 1 : 0);
                C[C_EVICTIONS]++;
                if (grp.preempt_keep) {
                    // The generated tokens stay with the request as prompt.  They are final, so they count as
                    // delivered now, together with the workload they took: l*j + j(j+1)/2 = sum_{i<=j} (l + i),
                    // which makes the workload of a request the sum over its segments,
                    // w(l, o) = w(l, j) + w(l + j, o - j).
                    C[C_COMPLETED_TOKENS] += r.j;
                    C[C_SUM_W_COMPLETED] += (int64_t)r.l * r.j + (int64_t)r.j * (r.j + 1) / 2;
                    r.l += r.j;
                    r.o -= r.j;
                } else {
                    C[C_WASTED_TOKENS] += r.j;
                }
                r.p = 0;
                r.j = 0;
                Q.push_front(r);
            }
        }

        // ---- F: process: every active request with its prompt in the cache generates one token
        for (Request& r : P) {
            if (r.p == r.l) {
                r.j++;
                C[C_TOKENS_GENERATED]++;
            }
        }
        const int64_t U_t = kv_usage(P);
        if (U_t != G) return -11;
        if (U_t > M) return -12;
        C[C_SUM_U] += U_t;
        C[C_MAX_U] = std::max(C[C_MAX_U], U_t);
        C[C_SUM_N] += (int64_t)P.size() + (int64_t)Q.size();

        // ---- G: completed requests leave and release their cache at the end of the slot
        {
            std::vector<Request> keep;
            keep.reserve(P.size());
            for (const Request& r : P) {
                if (r.p == r.l && r.j == r.o) {
                    const int64_t lat = (int64_t)t - r.t_arr + 1;
                    C[C_COMPLETED]++;
                    C[C_SUM_LAT] += lat;
                    C[C_MAX_LAT] = std::max(C[C_MAX_LAT], lat);
                    C[C_COMPLETED_TOKENS] += r.o;
                    C[C_SUM_W_COMPLETED] += (int64_t)r.l * r.o + (int64_t)r.o * (r.o + 1) / 2;
                    if (hist) hist[std::min<int64_t>(lat >> cfg.hist_shift, cfg.hist_bins - 1)]++;
                    if (complog) {
                        if (C[C_N_LOGGED] < cfg.complog_cap) {
                            complog[2 * C[C_N_LOGGED]] = t;
                            complog[2 * C[C_N_LOGGED] + 1] = (int32_t)lat;
                            C[C_N_LOGGED]++;
                        } else {
                            complog_overflow = true;
                        }
                    }
                } else {
                    keep.push_back(r);
                }
            }
            P.swap(keep);
        }

        // ---- H: record
        if (trace && cfg.trace_stride > 0 && t % cfg.trace_stride == 0) {
            const int64_t rec = t / cfg.trace_stride - 1;
            trace[2 * rec] = (int32_t)U_t;
            trace[2 * rec + 1] = (int32_t)Q.size();
        }
        C[C_MAX_Q] = std::max<int64_t>(C[C_MAX_Q], (int64_t)Q.size());

        if (!classflow) {
            // active set followed by the queue must stay sorted by arrival order
            int64_t prev = -1;
            for (const Request& r : P) { if (r.id <= prev) return -13; prev = r.id; }
            for (const Request& r : Q) { if (r.id <= prev) return -13; prev = r.id; }
        } else {
            // per class: active requests are older than waiting ones, and the queue is in arrival order
            std::vector<int64_t> newest_active(cfg.n_classes, -1), prev(cfg.n_classes, -1);
            for (const Request& r : P) newest_active[r.cls] = std::max(newest_active[r.cls], r.id);
            for (const Request& r : Q) {
                if (r.id <= prev[r.cls] || r.id <= newest_active[r.cls]) return -13;
                prev[r.cls] = r.id;
            }
        }
    }

    C[C_STEPS_DONE] = n_steps;
    C[C_STATUS] = (C[C_ACAP_BLOCKED] > 0 ? 1 : 0) | (complog_overflow ? 2 : 0);
    C[C_Q_FINAL] = (int64_t)Q.size();
    C[C_P_FINAL] = (int64_t)P.size();
    for (const Request& r : Q) C[C_RESID_AGE] += (int64_t)n_steps - r.t_arr + 1;
    for (const Request& r : P) {
        C[C_RESID_AGE] += (int64_t)n_steps - r.t_arr + 1;
        C[C_RESID_J] += r.j;
    }
    C[C_MMPP_STATE] = s;
    if (n_admlog_out) *n_admlog_out = n_admlog;
    return 0;
}

}  // namespace

// mc_mode: how the MC benchmark's future-memory test is evaluated: 0 = slot by slot (the definition),
// 1 = last slots only (shortcut), 2 = both, returning -20 if they ever disagree.  n_mc_tests (may be NULL)
// receives the number of tests made.
extern "C" int fcsim_oracle_run_ex(const orc_config* cfg, int64_t first_replica, int64_t n_replicas,
                                   int32_t n_steps, const orc_outputs* out, int mc_mode, int64_t* n_mc_tests) {
    if (!cfg || !out || !out->counters || mc_mode < 0 || mc_mode > 2) return -1;
    if (n_mc_tests) *n_mc_tests = 0;
    if (validate(*cfg)) return -2;
    if (n_steps < 0 || n_steps > cfg->T_max) return -3;
    int64_t total = 0;
    for (int g = 0; g < cfg->n_groups; ++g) total += cfg->groups[g].n_replicas;
    if (first_replica < 0 || n_replicas < 0 || first_replica + n_replicas > total) return -4;

    const int64_t n_rec = cfg->trace_stride > 0 ? n_steps / cfg->trace_stride : 0;
    int g = 0;
    int64_t g_first = 0;
    for (int64_t k = 0; k < n_replicas; ++k) {
        const int64_t r = first_replica + k;
        while (r >= g_first + cfg->groups[g].n_replicas) {
            g_first += cfg->groups[g].n_replicas;
            ++g;
        }
        const orc_group& grp = cfg->groups[g];
        const uint32_t rng_replica = grp.rng_replica_base + (uint32_t)(r - g_first);
        int32_t* hist = (out->hist && cfg->hist_bins > 0) ? out->hist + k * cfg->hist_bins : nullptr;
        if (hist) std::memset(hist, 0, sizeof(int32_t) * cfg->hist_bins);
        int32_t* complog = (out->complog && cfg->complog_cap > 0) ? out->complog + 2 * k * cfg->complog_cap : nullptr;
        if (complog) std::memset(complog, 0, sizeof(int32_t) * 2 * cfg->complog_cap);
        int rc = run_replica(*cfg, grp, rng_replica, n_steps, out->counters + k * C_COUNT,
                             (out->trace && n_rec > 0) ? out->trace + 2 * k * n_rec : nullptr, hist, complog,
                             out->arrlog ? out->arrlog + k * (int64_t)n_steps : nullptr,
                             out->arrcls ? out->arrcls + k * (int64_t)n_steps * cfg->n_classes : nullptr,
                             out->admlog ? out->admlog + 4 * k * out->admlog_cap : nullptr, out->admlog_cap,
                             out->n_admlog ? out->n_admlog + k : nullptr, mc_mode, n_mc_tests);
        if (rc) return rc;
    }
    return 0;
}

extern "C" int fcsim_oracle_run(const orc_config* cfg, int64_t first_replica, int64_t n_replicas,
                                int32_t n_steps, const orc_outputs* out) {
    return fcsim_oracle_run_ex(cfg, first_replica, n_replicas, n_steps, out, 0, nullptr);
}
