// Host side of fcsim: validation, table upload, launch geometry, resumable runs, statistics.
// The C ABI is declared in include/fcsim.h.
#include "fcsim.h"

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "fcsim_device.cuh"

using namespace fcsim_dev;

static_assert(sizeof(fcsim_counters) == C_COUNT * sizeof(int64_t), "counter block layout");

namespace {

constexpr size_t kSmemBudget = 227 * 1024;   // shared memory one CTA may opt in to
constexpr int kMaxStepsPerLaunch = 32768;    // upper limit of the slots of one launch (see max_steps_per_launch)
constexpr long long kTargetWorkPerLaunch = 1LL << 31;  // replica-steps per launch (bounds launch time)
constexpr uint64_t kGuideMaxRecords = 16384;  // per table: 256 KB of 16-byte records
constexpr int kStatsChunk = 256;             // replicas reduced by one block before it touches the group row
constexpr int kSelChunk = 8;                 // replicas whose completion logs one CTA counts before it moves on

struct Layout {
    int Apad, S;
    uint32_t QC;                                // queue ring in global memory: entries (a power of two)
    size_t gq_off, qwin_off;                    // queue ring in the workspace record; queue window in shared memory
    size_t ws_stride, smem_per_warp, qcnt_off;  // qcnt_off: per-class queue counts (Algorithm 1), 0 = unused
    size_t tstage_off;                          // trace staging buffers, 0 = unused
    size_t state_bytes;                         // ring + state words (+ projection words) saved between launches
    int has_v;
    int min_S;                                  // staging places a slot's arrivals need at most (the largest count)
    int qcnt_classes;                           // classes with a per-class queue count (Algorithm 1 groups), else 0
    int staged_trace;                           // 1 = trace staging buffers (trace_bulk)
    uint32_t prof_mask;                         // MC benchmark: H - 1 when the projection is kept per future slot, else 0
    int warps_per_block;
    int n_rec;
    long long R;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Exact latency percentiles from the completion log: two-digit selection over the latency words (< 2^24 because
// the horizon is): a count per value of the high 12 bits, then, for each of the two percentiles, a count per
// value of the low 12 bits among the latencies whose high bits are the selected ones.
constexpr int kSelBits = 12, kSelBins = 1 << kSelBits;
constexpr int kSelResultWords = 8;  // per group: logged completions, p95, p99 (rest unused)

// The per-group reduction area, in 64-bit words: [G][C_COUNT] counter rows, [G][bins] histogram rows and, with a
// completion log, [G][kSelResultWords] selection results, [G][kSelBins] high-digit counts, [G][2][kSelBins]
// low-digit counts.  Only the first three parts travel to the host.
size_t scratch_words(size_t G, size_t bins, int complog_cap) {
    return G * ((size_t)C_COUNT + bins + (complog_cap > 0 ? (size_t)kSelResultWords + 3 * (size_t)kSelBins : 0));
}
size_t scratch_words_to_host(size_t G, size_t bins, int complog_cap) {
    return G * ((size_t)C_COUNT + bins + (complog_cap > 0 ? (size_t)kSelResultWords : 0));
}

bool table_ok(const fcsim_table& t, int64_t vmin_lo, int64_t vmax_hi) {
    if (t.n == 0 || t.cdf == nullptr) return false;
    if (t.vmin < vmin_lo || (int64_t)t.vmin + (int64_t)t.n - 1 > vmax_hi) return false;
    for (uint32_t k = 1; k + 1 < t.n; ++k)
        if (t.cdf[k] < t.cdf[k - 1]) return false;
    return true;
}

// First and second moment of the law a table realises (value vmin + k has the mass between thresholds k - 1 and k,
// the last value the rest).
void table_moments(const fcsim_table& t, double* m1, double* m2) {
    double prev = 0.0, a = 0.0, b = 0.0;
    for (uint32_t k = 0; k < t.n; ++k) {
        const double cum = k + 1 < t.n ? std::max(prev, (double)t.cdf[k] / 4294967296.0) : 1.0;
        const double v = (double)t.vmin + k;
        a += v * (cum - prev);
        b += v * v * (cum - prev);
        prev = cum;
    }
    *m1 = a;
    if (m2) *m2 = b;
}

// Requests per slot that the cache can serve in the long run: M / E[w], with the per-request workload
// w = l o + o (o + 1) / 2 of Prop. 3.5 (l and o independent within a class).
double capacity_rate(const fcsim_config* c) {
    double ew = 0.0, prev = 0.0;
    for (int k = 0; k < c->n_classes; ++k) {
        const double cum = k + 1 < c->n_classes ? std::max(prev, (double)c->class_law.cdf[k] / 4294967296.0) : 1.0;
        double el, eo, eo2;
        table_moments(c->prompt[k], &el, nullptr);
        table_moments(c->decode[k], &eo, &eo2);
        ew += (cum - prev) * (el * eo + 0.5 * (eo + eo2));
        prev = cum;
    }
    return ew > 0.0 ? (double)c->M / ew : 0.0;
}

// A warp's shared memory for S staging places: saved state, staged arrivals, queue window (64 entries), per-class
// queue counts (Algorithm 1), and the optional trace staging (fcsim_config::trace_bulk = 1: 2 x 32 records of 8
// bytes, each batch leaving with one bulk copy; off by default: measured slower than keeping the records in
// registers, and the extra shared memory costs a CTA).
void set_staging(Layout* L, int S) {
    L->S = S;
    L->qwin_off = L->state_bytes + (size_t)S * 8;
    L->qcnt_off = L->qwin_off + 64 * 8;
    L->smem_per_warp = L->qcnt_off + (L->qcnt_classes ? align_up((size_t)L->qcnt_classes * 4, 16) : 0);
    if (!L->qcnt_classes) L->qcnt_off = 0;
    L->tstage_off = 0;
    if (L->staged_trace) {
        L->tstage_off = L->smem_per_warp;
        L->smem_per_warp += 512;
    }
    int w = kWarpsPerBlock;
    while (w > 1 && (size_t)w * L->smem_per_warp > kSmemBudget) w >>= 1;
    L->warps_per_block = w;
}

// Validates the description and derives the storage layout.  Returns an FCSIM_* code.
int plan(const fcsim_config* c, Layout* L) {
    if (!c) return FCSIM_EINVAL;
    if (c->M < 1 || c->M > (1 << 30) || c->K < 0 || c->T_max < 1 || c->T_max >= (1 << 24)) return FCSIM_EINVAL;
    if (c->Qcap < 1 || c->Acap < 1) return FCSIM_EINVAL;
    if (c->n_classes < 1 || c->n_classes > 256 || !c->prompt || !c->decode) return FCSIM_EINVAL;
    if (c->n_arrivals < 1 || !c->arrivals || c->n_groups < 1 || !c->groups) return FCSIM_EINVAL;
    if (!table_ok(c->class_law, 0, c->n_classes - 1) || c->class_law.vmin != 0 ||
        (int)c->class_law.n != c->n_classes)
        return FCSIM_EINVAL;
    int64_t lmax = 0, omax = 0;
    for (int k = 0; k < c->n_classes; ++k) {
        if (!table_ok(c->prompt[k], 1, 65535) || !table_ok(c->decode[k], 1, 65535)) return FCSIM_EINVAL;
        lmax = std::max<int64_t>(lmax, (int64_t)c->prompt[k].vmin + c->prompt[k].n - 1);
        omax = std::max<int64_t>(omax, (int64_t)c->decode[k].vmin + c->decode[k].n - 1);
    }
    if (lmax + omax > c->M) return FCSIM_EINVAL;  // a single request must fit the cache
    int max_count = 0;
    for (int a = 0; a < c->n_arrivals; ++a) {
        const fcsim_arrivals& A = c->arrivals[a];
        if (A.n_states != 1 && A.n_states != 2) return FCSIM_EINVAL;
        for (uint32_t s = 0; s < A.n_states; ++s) {
            if (!table_ok(A.count[s], 0, 255)) return FCSIM_EINVAL;
            max_count = std::max<int>(max_count, A.count[s].vmin + (int)A.count[s].n - 1);
        }
    }
    long long R = 0;
    bool any_classflow = false, any_mc = false;
    for (int g = 0; g < c->n_groups; ++g) {
        const fcsim_group& G = c->groups[g];
        if (G.policy < 0 || G.policy > 5 || G.n_replicas < 1) return FCSIM_EINVAL;
        if (G.policy == FCSIM_POLICY_MC) {
            if (G.mc_worst_case < 0 || G.mc_worst_case > 1) return FCSIM_EINVAL;
            any_mc = true;
        }
        if (G.policy == FCSIM_POLICY_CLASSFLOW) {
            if (!G.b_class) return FCSIM_EINVAL;
            for (int k = 0; k < c->n_classes; ++k)
                if (G.b_class[k] < 0 || G.b_class[k] > 65535) return FCSIM_EINVAL;
            any_classflow = true;
        }
        if (G.policy == FCSIM_POLICY_ALPHA && (G.m_admit < 1 || G.m_admit > c->M)) return FCSIM_EINVAL;
        if (G.arrivals_id < 0 || G.arrivals_id >= c->n_arrivals) return FCSIM_EINVAL;
        if (G.policy == FCSIM_POLICY_CHUNKED && G.chunk < 1) return FCSIM_EINVAL;
        if (G.preempt_keep < 0 || G.preempt_keep > 1) return FCSIM_EINVAL;
        // kept tokens join the prompt: l + j <= l_max + o_max - 1 must fit the entry's 16-bit prompt field
        if (G.preempt_keep && (G.policy == FCSIM_POLICY_MC || lmax + omax > 65536)) return FCSIM_EINVAL;
        R += G.n_replicas;
    }
    if (R > 0x7fffffffLL) return FCSIM_EINVAL;
    if (c->trace_stride < 0 || c->hist_bins < 0 || c->hist_shift < 0 || c->hist_shift > 30 || c->complog_cap < 0)
        return FCSIM_EINVAL;

    const long long rc = (long long)c->Qcap + c->Acap;  // evictions may push the queue past Qcap
    if (rc > (1 << 20)) return FCSIM_ECAP;
    L->QC = 64;
    while ((long long)L->QC < rc) L->QC <<= 1;
    L->Apad = (int)align_up((size_t)c->Acap, 4);
    L->S = (int)align_up((size_t)std::max(128, max_count), 2);
    // The MC benchmark keeps its projection of the future memory usage with the state: one word per active entry
    // (usage in that request's last slot), or, when that is no larger, one word per future slot (a ring of H slots,
    // H the power of two above the longest output length): a test then walks the candidate's lifetime instead of
    // the active set.
    L->has_v = any_mc ? 1 : 0;
    L->prof_mask = 0;
    size_t proj_words = 0;
    if (any_mc) {
        uint32_t H = 32;
        while ((int64_t)H < omax + 1) H <<= 1;
        if ((int64_t)H <= (int64_t)L->Apad) L->prof_mask = H - 1;
        proj_words = L->prof_mask ? H : (size_t)L->Apad;
    }
    L->state_bytes = (size_t)L->Apad * 8 + (size_t)L->Apad * 4 + proj_words * 4;
    // workspace record of a replica: 16 header words, the saved shared-memory state, the queue ring
    L->gq_off = kHeaderWords * 4 + L->state_bytes;
    L->ws_stride = L->gq_off + (size_t)L->QC * 8;
    if (c->trace_bulk < 0 || c->trace_bulk > 1) return FCSIM_EINVAL;
    L->min_S = (int)align_up((size_t)std::max(32, max_count), 2);
    L->qcnt_classes = any_classflow ? c->n_classes : 0;
    L->staged_trace = (c->trace_stride > 0 && c->trace_bulk == 1) ? 1 : 0;
    set_staging(L, L->S);
    if (L->smem_per_warp > kSmemBudget) return FCSIM_ECAP;
    L->n_rec = c->trace_stride > 0 ? c->T_max / c->trace_stride : 0;
    L->R = R;
    return FCSIM_OK;
}

void sizes_of(const fcsim_config* c, const Layout& L, fcsim_sizes* s) {
    s->workspace = (size_t)L.R * L.ws_stride;
    s->counters = (size_t)L.R * sizeof(fcsim_counters);
    s->trace = (size_t)L.R * (size_t)L.n_rec * 8;
    s->hist = (size_t)L.R * (size_t)c->hist_bins * 4;
    s->complog = (size_t)L.R * (size_t)c->complog_cap * 8;
    s->scratch = scratch_words(c->n_groups, c->hist_bins, c->complog_cap) * 8;
}

// ---- statistics kernels ---------------------------------------------------------------------------
// Group rows in scratch: [n_groups][C_COUNT] int64 counters, then [n_groups][hist_bins] int64 bins.

__device__ __forceinline__ int group_of(const DevGroup* groups, int n_groups, int r) {
    int lo = 0, hi = n_groups - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (groups[mid].first <= r) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ __forceinline__ void combine_into(long long* dst, int field, long long v) {
    if (field == C_MAX_LAT || field == C_MAX_U || field == C_MAX_Q || field == C_STEPS_DONE)
        atomicMax(dst, v);
    else if (field == C_STATUS)
        atomicOr(reinterpret_cast<unsigned long long*>(dst), (unsigned long long)v);
    else
        atomicAdd(reinterpret_cast<unsigned long long*>(dst), (unsigned long long)v);
}

__device__ __forceinline__ long long combine(int field, long long a, long long b) {
    if (field == C_MAX_LAT || field == C_MAX_U || field == C_MAX_Q || field == C_STEPS_DONE) return a > b ? a : b;
    if (field == C_STATUS) return a | b;
    return a + b;
}

// One warp per chunk of replicas; lane k owns counter field k.
__global__ void reduce_counters_kernel(const long long* __restrict__ counters, const DevGroup* __restrict__ groups,
                                       int n_groups, int n_replicas, int chunk, long long* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    const int n_chunks = (n_replicas + chunk - 1) / chunk;
    for (int c = warp; c < n_chunks; c += n_warps) {
        const int r0 = c * chunk, r1 = min(n_replicas, r0 + chunk);
        int g = group_of(groups, n_groups, r0);
        int g_end = groups[g].first + groups[g].n;
        long long acc = 0;
        for (int r = r0; r < r1; ++r) {
            if (r >= g_end) {
                if (lane < C_COUNT) combine_into(out + (size_t)g * C_COUNT + lane, lane, acc);
                acc = 0;
                ++g;
                g_end = groups[g].first + groups[g].n;
            }
            if (lane < C_COUNT) acc = combine(lane, acc, counters[(size_t)r * C_COUNT + lane]);
        }
        if (lane < C_COUNT) combine_into(out + (size_t)g * C_COUNT + lane, lane, acc);
    }
}

// One block per chunk of replicas.  HBM-bound: every histogram word is read once (4 bytes per bin and
// replica), 16 bytes per thread and load when the rows allow it (bins % 4 == 0), several loads in flight.
template <int VEC>
__global__ void reduce_hist_kernel(const int* __restrict__ hist, const DevGroup* __restrict__ groups, int n_groups,
                                   int n_replicas, int bins, int chunk, long long* __restrict__ out) {
    const int n_chunks = (n_replicas + chunk - 1) / chunk;
    for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const int r0 = c * chunk, r1 = min(n_replicas, r0 + chunk);
        for (int b = threadIdx.x * VEC; b < bins; b += blockDim.x * VEC) {
            int g = group_of(groups, n_groups, r0);
            int g_end = groups[g].first + groups[g].n;
            long long acc[4] = {0, 0, 0, 0};
            int r = r0;
            while (r < r1) {
                if (r >= g_end) {
                    for (int v = 0; v < VEC; ++v) {
                        if (acc[v]) atomicAdd(reinterpret_cast<unsigned long long*>(out + (size_t)g * bins + b + v),
                                              (unsigned long long)acc[v]);
                        acc[v] = 0;
                    }
                    ++g;
                    g_end = groups[g].first + groups[g].n;
                }
                const int stop = min(r1, g_end);
                if (VEC == 4) {
                    const int4* row = reinterpret_cast<const int4*>(hist + (size_t)r * bins + b);
                    const size_t pitch = (size_t)bins / 4;
                    int k = 0;
                    for (; r + k + 4 <= stop; k += 4) {  // four independent 16-byte loads in flight
                        const int4 x0 = __ldg(row + (size_t)(k + 0) * pitch), x1 = __ldg(row + (size_t)(k + 1) * pitch);
                        const int4 x2 = __ldg(row + (size_t)(k + 2) * pitch), x3 = __ldg(row + (size_t)(k + 3) * pitch);
                        acc[0] += (long long)x0.x + x1.x + x2.x + x3.x;
                        acc[1] += (long long)x0.y + x1.y + x2.y + x3.y;
                        acc[2] += (long long)x0.z + x1.z + x2.z + x3.z;
                        acc[3] += (long long)x0.w + x1.w + x2.w + x3.w;
                    }
                    for (; r + k < stop; ++k) {
                        const int4 x = __ldg(row + (size_t)k * pitch);
                        acc[0] += x.x; acc[1] += x.y; acc[2] += x.z; acc[3] += x.w;
                    }
                } else {
                    for (int q = r; q < stop; ++q) acc[0] += hist[(size_t)q * bins + b];
                }
                r = stop;
            }
            for (int v = 0; v < VEC; ++v)
                if (acc[v]) atomicAdd(reinterpret_cast<unsigned long long*>(out + (size_t)g * bins + b + v),
                                      (unsigned long long)acc[v]);
        }
    }
}

void launch_reduce_hist(const int* hist, const DevGroup* groups, int G, int R, int bins, int blocks, long long* out,
                        cudaStream_t st) {
    if (bins % 4 == 0)
        reduce_hist_kernel<4><<<blocks, std::min(256, bins / 4), 0, st>>>(hist, groups, G, R, bins, kStatsChunk, out);
    else
        reduce_hist_kernel<1><<<blocks, 256, 0, st>>>(hist, groups, G, R, bins, kStatsChunk, out);
}

// ---- exact percentiles from the completion log ---------------------------------------------------------
// HBM-bound: every logged {slot, latency} pair is read once per pass (8 bytes per completion).
// One CTA walks chunks of replicas; the counts of the current group are kept in shared memory (32-bit: a chunk
// holds far fewer than 2^32 records) and flushed into the group's 64-bit row when the group changes.  Lanes of a
// warp that hit the same bin are combined first (__match_any_sync), because latencies cluster.
// kPass 1: bin = latency >> 12.  kPass 2: sel[g] = {high digit of p95, of p99}; a latency with that high digit
// counts under its low 12 bits in the first, respectively second, table of its group.
template <int kPass>
__global__ void __launch_bounds__(256) latency_digit_kernel(const int2* __restrict__ complog,
                                                            const long long* __restrict__ counters,
                                                            const DevGroup* __restrict__ groups, int n_groups,
                                                            int n_replicas, int cap, int chunk,
                                                            const long long* __restrict__ sel,
                                                            unsigned long long* __restrict__ out) {
    constexpr int kTables = kPass == 1 ? 1 : 2;
    __shared__ unsigned int sh[kTables * kSelBins];
    const int n_chunks = (n_replicas + chunk - 1) / chunk;
    for (int i = threadIdx.x; i < kTables * kSelBins; i += blockDim.x) sh[i] = 0;
    __syncthreads();
    auto flush = [&](int g) {
        __syncthreads();
        for (int i = threadIdx.x; i < kTables * kSelBins; i += blockDim.x) {
            const unsigned int v = sh[i];
            if (v) {
                atomicAdd(out + (size_t)g * kTables * kSelBins + i, (unsigned long long)v);
                sh[i] = 0;
            }
        }
        __syncthreads();
    };
    // Latencies cluster: when all the lanes of a warp that count hit one bin (the rule for the high digit, and for
    // constant lengths) one lane adds their number; otherwise every lane adds one (bins spread, few collisions).
    auto count = [&](unsigned int* table, bool mine, unsigned int bin) {
        const unsigned int voters = __ballot_sync(0xffffffffu, mine);
        if (voters == 0u) return;
        const int leader = __ffs(voters) - 1;
        const unsigned int lead_bin = __shfl_sync(0xffffffffu, bin, leader);
        const bool same = __all_sync(0xffffffffu, !mine || bin == lead_bin);
        if (same) {
            if ((int)(threadIdx.x & 31) == leader) atomicAdd(table + bin, (unsigned)__popc(voters));
        } else if (mine) {
            atomicAdd(table + bin, 1u);
        }
    };
    for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const int r0 = c * chunk, r1 = min(n_replicas, r0 + chunk);
        int g = group_of(groups, n_groups, r0);
        int g_end = groups[g].first + groups[g].n;
        unsigned int hi95 = 0, hi99 = 0;
        if (kPass == 2) { hi95 = (unsigned)sel[(size_t)g * kSelResultWords + 3]; hi99 = (unsigned)sel[(size_t)g * kSelResultWords + 5]; }
        for (int r = r0; r < r1; ++r) {
            if (r >= g_end) {
                flush(g);
                ++g;
                g_end = groups[g].first + groups[g].n;
                if (kPass == 2) { hi95 = (unsigned)sel[(size_t)g * kSelResultWords + 3]; hi99 = (unsigned)sel[(size_t)g * kSelResultWords + 5]; }
            }
            const int n = min((int)counters[(size_t)r * C_COUNT + C_N_LOGGED], cap);
            const int2* __restrict__ row = complog + (size_t)r * cap;
            // every thread of the CTA runs the same number of iterations (warp-wide votes inside)
            for (int base = 0; base < n; base += 4 * (int)blockDim.x) {
                int lat[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {  // four independent loads in flight
                    const int i = base + u * (int)blockDim.x + (int)threadIdx.x;
                    lat[u] = i < n ? __ldg(row + i).y : -1;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool have = lat[u] >= 0;
                    const unsigned int v = (unsigned)lat[u] & 0xffffffu;
                    if (kPass == 1) {
                        count(sh, have, v >> kSelBits);
                    } else {
                        count(sh, have && (v >> kSelBits) == hi95, v & (kSelBins - 1));
                        // both ranks in one high digit (the rule): the first table serves both
                        if (hi99 != hi95) count(sh + kSelBins, have && (v >> kSelBits) == hi99, v & (kSelBins - 1));
                    }
                }
            }
        }
        flush(g);
    }
}

// One CTA of 256 threads per group: the smallest bin whose cumulative count reaches a target rank.
// kPass 1: row = the group's high-digit counts; total = their sum; targets ceil(95 total / 100) and ceil(99 total / 100);
//          res[g] = {total, 0, 0, bin95, rank95 within that bin, bin99, rank99 within that bin, 0}.
// kPass 2: rows = the group's two low-digit tables, targets = the ranks left by pass 1;
//          res[g][1] = p95 and res[g][2] = p99 (high digit << 12 | low digit).
template <int kPass>
__global__ void __launch_bounds__(256) latency_select_kernel(const unsigned long long* __restrict__ tables,
                                                             long long* __restrict__ res) {
    __shared__ unsigned long long part[256];
    __shared__ unsigned long long total_s;
    const int g = blockIdx.x, tid = threadIdx.x;
    constexpr int kPer = kSelBins / 256;
    long long* out = res + (size_t)g * kSelResultWords;
    for (int qi = 0; qi < 2; ++qi) {
        // pass 2 fills the second table only when the two ranks differ in the high digit
        const int tab = (kPass == 1 || out[3] == out[5]) ? 0 : qi;
        const unsigned long long* row = tables + ((size_t)g * (kPass == 1 ? 1 : 2) + tab) * kSelBins;
        unsigned long long mine = 0;
        for (int k = 0; k < kPer; ++k) mine += row[tid * kPer + k];
        part[tid] = mine;
        __syncthreads();
        if (tid == 0) {  // 256 partial sums: a serial scan is short next to the pass over the log
            unsigned long long run = 0;
            for (int k = 0; k < 256; ++k) { const unsigned long long v = part[k]; part[k] = run; run += v; }
            total_s = run;
        }
        __syncthreads();
        const unsigned long long total = total_s;
        unsigned long long target;
        if (kPass == 1) target = ((unsigned long long)(qi == 0 ? 95 : 99) * total + 99) / 100;
        else target = (unsigned long long)out[4 + 2 * qi];
        if (total > 0 && target > 0 && part[tid] < target && part[tid] + mine >= target) {
            unsigned long long cum = part[tid];
            for (int k = 0; k < kPer; ++k) {
                const unsigned long long v = row[tid * kPer + k];
                if (cum + v >= target) {
                    if (kPass == 1) {
                        out[3 + 2 * qi] = tid * kPer + k;
                        out[4 + 2 * qi] = (long long)(target - cum);
                    } else {
                        out[1 + qi] = (out[3 + 2 * qi] << kSelBits) | (long long)(tid * kPer + k);
                    }
                    break;
                }
                cum += v;
            }
        }
        if (kPass == 1 && qi == 0 && tid == 0) out[0] = (long long)total;
        __syncthreads();
    }
}

}  // namespace

// The opt-in shared-memory limit is a property of a kernel, shared by every handle of the process: setting it
// and using it (occupancy query, launch) happen under this lock, so that handles driven from different threads do
// not change it between another handle's two steps.
static std::mutex g_kernel_attr_mutex;

// The step kernel of one policy (6: the MC benchmark with its projection per future slot) for a register
// allocation that lets `ctas` CTAs reside on an SM and for a variant; each policy's kernels are an object of their
// own (fcsim_step_kernels.cu).
static step_kernel_t pick_step_kernel(int policy, int ctas, int rec, bool bulk, bool lazy) {
    switch (policy) {
        case FCSIM_POLICY_FLOW: return step_kernel_of_policy_0(ctas, rec, bulk, lazy);
        case FCSIM_POLICY_GREEDY: return step_kernel_of_policy_1(ctas, rec, bulk, lazy);
        case FCSIM_POLICY_CHUNKED: return step_kernel_of_policy_2(ctas, rec, bulk, lazy);
        case FCSIM_POLICY_ALPHA: return step_kernel_of_policy_3(ctas, rec, bulk, lazy);
        case FCSIM_POLICY_CLASSFLOW: return step_kernel_of_policy_4(ctas, rec, bulk, lazy);
        case FCSIM_POLICY_MC: return step_kernel_of_policy_5(ctas, rec, bulk, lazy);
        case 6: return step_kernel_of_policy_6(ctas, rec, bulk, lazy);
        default: return nullptr;
    }
}

// One launch per policy present in the configuration: its kernel, its groups (a contiguous piece of the
// policy-sorted group array), its launch shape, and the side stream it runs on when there are several.
struct PolicyLaunch {
    int policy = 0;
    step_kernel_t kernel = nullptr;
    int pg_off = 0, pg_cnt = 0;   // its groups in d_pgroups
    int n_work = 0;               // replicas
    bool bulk = false;            // two or more requests arrive, and may be activated, per slot on average
    bool lazy = false;            // at least twice as many requests arrive as the cache can serve: most are dropped
    double busiest = 0.0;         // requests that arrive per slot, the largest over the policy's groups
    int warps_per_block = 0, blocks_per_sm = 0, grid = 0;
    size_t smem_block = 0, tabcache_off = 0;
    cudaStream_t side = nullptr;  // null: the caller's stream
    cudaEvent_t done = nullptr;
};

struct fcsim {
    fcsim_config cfg;                 // scalar fields only; the pointers inside are not kept
    std::vector<fcsim_group> groups;  // host copy
    Layout L;
    fcsim_buffers buf;
    Params params;
    void* d_blob = nullptr;              // one allocation holding everything below up to d_work
    uint32_t* d_pool = nullptr;
    uint4* d_gpool = nullptr;
    int32_t* d_bclass = nullptr;
    std::vector<PolicyLaunch> launches;  // most expensive policy first
    int main_launch = 0;                 // the launch with the most replicas (reported by fcsim_get_launch_info)
    cudaEvent_t fork = nullptr;
    DevGroup* d_pgroups = nullptr;       // the groups sorted by policy (stable), with their work-item offsets
    DevTable* d_tables = nullptr;
    DevArrivals* d_arrivals = nullptr;
    DevGroup* d_groups = nullptr;
    unsigned int* d_work = nullptr;
    int device = 0, sm_count = 0;
    int t_done = 0;
    int last_cuda = 0;
    size_t table_bytes = 0;
};

#define CUDA_TRY(h, call)                                 \
    do {                                                  \
        cudaError_t e__ = (call);                         \
        if (e__ != cudaSuccess) {                         \
            (h)->last_cuda = (int)e__;                    \
            return FCSIM_ECUDA;                           \
        }                                                 \
    } while (0)

// A handle works on the device that was current in fcsim_create; calls made with another device current
// are refused rather than silently launched on the wrong GPU.
static int check_device(fcsim* h) {
    int dev = -1;
    CUDA_TRY(h, cudaGetDevice(&dev));
    return dev == h->device ? FCSIM_OK : FCSIM_EINVAL;
}

extern "C" int fcsim_query_sizes(const fcsim_config* cfg, fcsim_sizes* out) {
    if (!out) return FCSIM_EINVAL;
    Layout L;
    const int rc = plan(cfg, &L);
    if (rc != FCSIM_OK) return rc;
    sizes_of(cfg, L, out);
    return FCSIM_OK;
}

static int upload_tables(fcsim* h, const fcsim_config* c) {
    std::vector<uint32_t> pool;
    std::vector<uint4> gpool;
    // Guide of a table (see guide_bucket in the device code): one record per bucket of the 32-bit range.  The
    // bucket scheme (g, J) is the candidate that leaves the least probability mass to the fall-back search,
    // within kGuideMaxRecords per table; equal buckets (J = 0) suit flat laws, halving buckets (J > 0) suit
    // laws with a long upper tail.
    auto bucket_range = [](uint32_t g, uint32_t J, uint32_t j, uint32_t m, uint32_t* ulo, uint32_t* uhi) {
        // bucket (j, m) holds the v = ~u with clz(v) == j (>= J for j == J) and mantissa m; false if it is empty
        const uint32_t sh = j + (j < J ? 1u : 0u);
        const uint32_t rem = 32u - sh;  // bits of v below the consumed ones
        uint64_t vlo, vhi;
        if (rem >= g) {
            vlo = (uint64_t)m << (rem - g);
            vhi = vlo | ((1ull << (rem - g)) - 1ull);
        } else {
            if (m & ((1u << (g - rem)) - 1u)) return false;
            vlo = vhi = m >> (g - rem);
        }
        if (j < J) { vlo |= 1ull << rem; vhi |= 1ull << rem; }
        *ulo = ~(uint32_t)vhi;
        *uhi = ~(uint32_t)vlo;
        return true;
    };
    auto add = [&](const fcsim_table& t) {
        DevTable d;
        d.off = (uint32_t)pool.size();
        d.n = t.n;
        d.vmin = t.vmin;
        d.guide = 0;
        pool.insert(pool.end(), t.cdf, t.cdf + t.n);
        if (t.n >= 2) {
            const uint32_t* thr_end = t.cdf + (t.n - 1);  // real thresholds: cdf[0 .. n-2]
            auto first_above = [&](uint32_t x) { return (uint32_t)(std::upper_bound(t.cdf, thr_end, x) - t.cdf); };
            double best_mass = 2.0;
            uint32_t best_g = 0, best_J = 0;
            for (uint32_t J = 0; J <= 20; J += 4) {
                for (uint32_t g = 4; g <= 14; ++g) {
                    const uint64_t records = (uint64_t)(J + 1) << g;
                    if (records > kGuideMaxRecords) break;
                    if (J > 0 && g > 10) break;
                    double mass = 0.0;
                    for (uint32_t j = 0; j <= J; ++j)
                        for (uint32_t m = 0; m < (1u << g); ++m) {
                            uint32_t ulo, uhi;
                            if (!bucket_range(g, J, j, m, &ulo, &uhi)) continue;
                            const uint32_t k3 = first_above(ulo) + 2;  // third threshold above the bucket's low end
                            if (k3 < t.n - 1 && t.cdf[k3] <= uhi) mass += (double)uhi - (double)std::max(t.cdf[k3], ulo) + 1.0;
                        }
                    mass /= 4294967296.0;
                    // a larger guide must buy a clearly smaller fall-back mass, and 1e-4 is small enough
                    if (best_mass > 1.5 || (best_mass > 1e-4 && mass < best_mass * 0.7)) { best_mass = mass; best_g = g; best_J = J; }
                    if (mass <= 1e-4) break;
                }
            }
            d.guide = (best_g << 27) | (best_J << 22) | (uint32_t)gpool.size();
            for (uint32_t j = 0; j <= best_J; ++j)
                for (uint32_t m = 0; m < (1u << best_g); ++m) {
                    uint32_t ulo = 0, uhi = 0;
                    uint4 rec = make_uint4(t.n - 1, 0xffffffffu, 0xffffffffu, 0xffffffffu);
                    if (bucket_range(best_g, best_J, j, m, &ulo, &uhi)) {
                        const uint32_t k0 = first_above(ulo);
                        rec.x = k0;
                        if (k0 + 0 < t.n - 1) rec.y = t.cdf[k0];
                        if (k0 + 1 < t.n - 1) rec.z = t.cdf[k0 + 1];
                        if (k0 + 2 < t.n - 1) rec.w = t.cdf[k0 + 2];
                    }
                    gpool.push_back(rec);
                }
        }
        return d;
    };
    std::vector<DevTable> tables;
    tables.push_back(add(c->class_law));
    for (int k = 0; k < c->n_classes; ++k) tables.push_back(add(c->prompt[k]));
    for (int k = 0; k < c->n_classes; ++k) tables.push_back(add(c->decode[k]));
    std::vector<DevArrivals> arrs(c->n_arrivals);
    for (int a = 0; a < c->n_arrivals; ++a) {
        const fcsim_arrivals& A = c->arrivals[a];
        arrs[a].n_states = A.n_states;
        arrs[a].pad = 0;
        arrs[a].count[0] = add(A.count[0]);
        arrs[a].count[1] = A.n_states == 2 ? add(A.count[1]) : arrs[a].count[0];
        arrs[a].thr[0] = A.switch_thr[0];
        arrs[a].thr[1] = A.switch_thr[1];
    }
    std::vector<DevGroup> grps(c->n_groups);
    std::vector<int32_t> bclass(1, 0);
    int first = 0;
    for (int g = 0; g < c->n_groups; ++g) {
        const fcsim_group& G = c->groups[g];
        int32_t boff = 0;
        if (G.policy == FCSIM_POLICY_CLASSFLOW) {
            boff = (int32_t)bclass.size();
            bclass.insert(bclass.end(), G.b_class, G.b_class + c->n_classes);
        }
        grps[g] = DevGroup{G.policy, G.b_fp, G.chunk, G.arrivals_id, G.rng_replica_base, first, G.n_replicas,
                           G.policy == FCSIM_POLICY_ALPHA ? G.m_admit : c->M, boff,
                           G.policy == FCSIM_POLICY_MC ? G.mc_worst_case : 0, G.preempt_keep, first};
        first += G.n_replicas;
    }
    // the same groups sorted by policy (order within a policy kept): one launch per policy walks its piece
    std::vector<DevGroup> pgrps;
    const double cap_rate = capacity_rate(c);
    for (int pol = FCSIM_POLICY_MC; pol >= FCSIM_POLICY_FLOW; --pol) {  // costly policies first
        PolicyLaunch pl;
        pl.policy = pol;
        pl.pg_off = (int)pgrps.size();
        double most = 0.0;  // requests that arrive and may be activated per slot, the largest over the policy's groups
        double busiest = 0.0;  // requests that arrive per slot, the largest over the policy's groups
        for (int g = 0; g < c->n_groups; ++g) {
            if (grps[g].policy != pol) continue;
            DevGroup d = grps[g];
            d.wfirst = pl.n_work;
            pl.n_work += d.n;
            pgrps.push_back(d);
            const fcsim_arrivals& A = c->arrivals[d.arrivals_id];
            double rate = 0.0;
            for (uint32_t st = 0; st < A.n_states; ++st) {
                double m;
                table_moments(A.count[st], &m, nullptr);
                rate = std::max(rate, m);
            }
            busiest = std::max(busiest, rate);
            if (pol == FCSIM_POLICY_FLOW) rate = std::min(rate, (double)d.b_fp / 65536.0);
            most = std::max(most, rate);
        }
        // activations per slot cannot outrun the arrivals, the flow-control rate or what the cache can serve
        pl.bulk = std::min(most, cap_rate) >= 2.0;
        // heavy overload with a waiting room long enough to hide the head: arrivals are drawn when they get there
        pl.lazy = busiest >= 2.0 * cap_rate && c->Qcap >= 128;
        pl.busiest = busiest;
        pl.pg_cnt = (int)pgrps.size() - pl.pg_off;
        if (pl.pg_cnt > 0) h->launches.push_back(pl);
    }
    if (gpool.empty()) gpool.push_back(make_uint4(0, 0, 0, 0));
    if (gpool.size() > (size_t)0x3fffff) return FCSIM_ECAP;  // a guide's first record is a 22-bit index
    // one device allocation and one copy for all the tables (a handle is often created for a short run)
    struct Part { const void* src; size_t bytes; void** dst; };
    const Part parts[] = {
        {gpool.data(), gpool.size() * sizeof(uint4), reinterpret_cast<void**>(&h->d_gpool)},
        {pool.data(), pool.size() * sizeof(uint32_t), reinterpret_cast<void**>(&h->d_pool)},
        {tables.data(), tables.size() * sizeof(DevTable), reinterpret_cast<void**>(&h->d_tables)},
        {arrs.data(), arrs.size() * sizeof(DevArrivals), reinterpret_cast<void**>(&h->d_arrivals)},
        {grps.data(), grps.size() * sizeof(DevGroup), reinterpret_cast<void**>(&h->d_groups)},
        {pgrps.data(), pgrps.size() * sizeof(DevGroup), reinterpret_cast<void**>(&h->d_pgroups)},
        {bclass.data(), bclass.size() * sizeof(int32_t), reinterpret_cast<void**>(&h->d_bclass)},
        {nullptr, 16 * sizeof(unsigned int), reinterpret_cast<void**>(&h->d_work)},  // work counters + debug record: zero
    };
    size_t total = 0;
    for (const Part& q : parts) total += align_up(q.bytes, 256);
    std::vector<unsigned char> blob(total, 0);
    CUDA_TRY(h, cudaMalloc(&h->d_blob, total));
    size_t off = 0;
    for (const Part& q : parts) {
        if (q.src) std::memcpy(blob.data() + off, q.src, q.bytes);
        *q.dst = static_cast<unsigned char*>(h->d_blob) + off;
        off += align_up(q.bytes, 256);
    }
    CUDA_TRY(h, cudaMemcpy(h->d_blob, blob.data(), total, cudaMemcpyHostToDevice));
    h->table_bytes = pool.size() * 4 + tables.size() * sizeof(DevTable) + arrs.size() * sizeof(DevArrivals) +
                     grps.size() * sizeof(DevGroup);
    return FCSIM_OK;
}

static void release(fcsim* h) {
    if (!h) return;
    cudaFree(h->d_blob);  // all the tables
    for (PolicyLaunch& pl : h->launches) {
        if (pl.done) cudaEventDestroy(pl.done);
        if (pl.side) cudaStreamDestroy(pl.side);
    }
    if (h->fork) cudaEventDestroy(h->fork);
    delete h;
}

// trace_window_recs: 0 = the trace buffer holds the whole horizon ([R][T_max / stride] records); otherwise it is a
// window of that many records per replica which the caller of launch_slots moves along the horizon.
static int create_handle(const fcsim_config* cfg, const fcsim_buffers* b, fcsim_t** out, int trace_window_recs) {
    if (!out) return FCSIM_EINVAL;
    *out = nullptr;
    Layout L;
    int rc = plan(cfg, &L);
    if (rc != FCSIM_OK) return rc;
    if (!b) return FCSIM_ESIZE;
    fcsim_sizes sz;
    sizes_of(cfg, L, &sz);
    if (trace_window_recs > 0) sz.trace = (size_t)L.R * (size_t)trace_window_recs * 8;
    if (!b->workspace || !b->counters || !b->scratch) return FCSIM_ESIZE;
    if (sz.trace && !b->trace) return FCSIM_ESIZE;
    if (sz.hist && !b->hist) return FCSIM_ESIZE;
    if (sz.complog && !b->complog) return FCSIM_ESIZE;
    const void* ptrs[6] = {b->workspace, b->counters, b->trace, b->hist, b->complog, b->scratch};
    for (const void* q : ptrs)
        if (q && (reinterpret_cast<uintptr_t>(q) & 15)) return FCSIM_ESIZE;

    fcsim* h = new (std::nothrow) fcsim();
    if (!h) return FCSIM_ENOMEM;
    try {
        h->groups.assign(cfg->groups, cfg->groups + cfg->n_groups);
    } catch (...) {
        delete h;
        return FCSIM_ENOMEM;
    }
    h->cfg = *cfg;
    h->cfg.prompt = h->cfg.decode = nullptr;
    h->cfg.arrivals = nullptr;
    h->cfg.class_law.cdf = nullptr;
    h->cfg.groups = nullptr;
    h->L = L;
    h->buf = *b;

    auto fail = [&](int code) {
        release(h);
        return code;
    };
    cudaError_t e = cudaGetDevice(&h->device);
    if (e != cudaSuccess) return fail(FCSIM_ECUDA);
    // three attribute queries (the whole property structure takes far longer to fill)
    struct { int multiProcessorCount, sharedMemPerMultiprocessor, sharedMemPerBlockOptin; } prop = {0, 0, 0};
    e = cudaDeviceGetAttribute(&prop.multiProcessorCount, cudaDevAttrMultiProcessorCount, h->device);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&prop.sharedMemPerMultiprocessor, cudaDevAttrMaxSharedMemoryPerMultiprocessor, h->device);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&prop.sharedMemPerBlockOptin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device);
    if (e != cudaSuccess) return fail(FCSIM_ECUDA);
    h->sm_count = prop.multiProcessorCount;
    try {
        rc = upload_tables(h, cfg);
    } catch (...) {
        rc = FCSIM_ENOMEM;
    }
    if (rc != FCSIM_OK) return fail(rc);

    // Launch shape, per policy kernel: warps per CTA (1 .. 4) and register allocation (builds for 5, 6, 7 and 8
    // resident CTAs: <= 96, 80, 72, 64 registers) are chosen for the largest number of resident warps per SM, as the
    // occupancy calculator reports it for this device; ties go to the roomier register allocation, then to the
    // larger CTA.  Small slices of shared memory end up register-bound, large ones shared-memory-bound, where
    // smaller CTAs waste less of the SM's 228 KB.  The staging area for generated arrivals is the one part of a
    // warp's slice that the library may size: the shapes are worked out for the roomy one (128 places: a batch of 32
    // slots rarely has to be cut short) and for the smallest one (the largest arrival count of a slot, at least
    // 32), and the small one is taken when it lets more warps reside (Acap = 512: 8 CTAs of 4 warps instead of 7).
    const bool ext = L.qcnt_off || L.has_v;
    // what is recorded per slot is a compile-time property of the kernels of the common policies
    const int rec = (ext || cfg->complog_cap > 0 || L.tstage_off != 0) ? 2 : (L.n_rec > 0 ? 1 : 0);
    const size_t tab_extra = align_up((size_t)(1 + 2 * cfg->n_classes) * sizeof(DevTable), 16);
    const size_t sm_bytes = (size_t)prop.sharedMemPerMultiprocessor;
    auto ctas_by_smem = [&](size_t b) { return sm_bytes / (align_up(b, 1024) + 1024); };
    size_t most_work = 0;
    auto shape = [&](const Layout& L, std::vector<PolicyLaunch>& launches) -> int {
    for (size_t li = 0; li < launches.size(); ++li) {
        PolicyLaunch& pl = launches[li];
        int best_warps = 0;
        for (int w = L.warps_per_block; w >= 1; --w) {
            size_t block = (size_t)w * L.smem_per_warp, tab = 0;
            if (block > (size_t)prop.sharedMemPerBlockOptin) continue;
            // a copy of the table descriptors behind the warps' slices, if it does not cost a resident CTA
            if (cfg->n_classes <= 16 && block + tab_extra <= (size_t)prop.sharedMemPerBlockOptin &&
                ctas_by_smem(block + tab_extra) == ctas_by_smem(block)) {
                tab = block;
                block += tab_extra;
            }
            for (int ctas = 5; ctas <= 8; ++ctas) {
                step_kernel_t k = pick_step_kernel(pl.policy == FCSIM_POLICY_MC && L.prof_mask ? 6 : pl.policy, ctas, rec,
                                                   pl.bulk, pl.lazy);
                if (!k) return FCSIM_EINVAL;
                int occ = 0;
                {
                    std::lock_guard<std::mutex> lock(g_kernel_attr_mutex);
                    e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)block);
                    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k, w * 32, block);
                }
                if (e != cudaSuccess) { h->last_cuda = (int)e; return FCSIM_ECUDA; }
                if (occ * w > best_warps) {
                    best_warps = occ * w;
                    pl.kernel = k;
                    pl.warps_per_block = w;
                    pl.blocks_per_sm = occ;
                    pl.smem_block = block;
                    pl.tabcache_off = tab;
                }
            }
        }
        if (best_warps < 1) return FCSIM_ECAP;
        const long long want = ((long long)pl.n_work + pl.warps_per_block - 1) / pl.warps_per_block;
        pl.grid = (int)std::max<long long>(1, std::min<long long>((long long)h->sm_count * pl.blocks_per_sm, want));
        if ((size_t)pl.n_work > most_work) { most_work = (size_t)pl.n_work; h->main_launch = (int)li; }
    }
    return FCSIM_OK;
    };
    {
        std::vector<PolicyLaunch> roomy = h->launches, tight = h->launches;
        Layout Lt = L;
        set_staging(&Lt, L.min_S);
        rc = shape(L, roomy);
        if (rc == FCSIM_OK && Lt.S < L.S) {
            most_work = 0;
            rc = shape(Lt, tight);
        }
        if (rc != FCSIM_OK) return fail(rc);
        // More resident warps pay when they shorten the run by whole waves of replicas (the warps take replicas from
        // a common queue: with the same number of waves every warp is merely slower), and a small staging area only
        // where a batch of 32 slots rarely overflows it (or is not staged at all: arrivals drawn at the queue head).
        const int m = h->main_launch;
        const long long wr = (long long)roomy[m].blocks_per_sm * roomy[m].warps_per_block * h->sm_count;
        const long long wt = (long long)tight[m].blocks_per_sm * tight[m].warps_per_block * h->sm_count;
        const bool fits = tight[m].lazy || tight[m].busiest * 32.0 <= 2.0 * Lt.S;
        if (Lt.S < L.S && fits && wt > wr && (L.R + wt - 1) / wt < (L.R + wr - 1) / wr) {
            h->launches = tight;
            L = Lt;
            h->L = Lt;
        } else {
            h->launches = roomy;
        }
    }
    // several policies: their launches run side by side (the first on the caller's stream, the others on streams
    // of the handle, forked from and joined to the caller's stream by events), so that no SM idles while the last
    // replicas of one policy finish
    if (h->launches.size() > 1) {
        e = cudaEventCreateWithFlags(&h->fork, cudaEventDisableTiming);
        if (e != cudaSuccess) { h->last_cuda = (int)e; return fail(FCSIM_ECUDA); }
        for (size_t li = 1; li < h->launches.size(); ++li) {
            e = cudaStreamCreateWithFlags(&h->launches[li].side, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->launches[li].done, cudaEventDisableTiming);
            if (e != cudaSuccess) { h->last_cuda = (int)e; return fail(FCSIM_ECUDA); }
        }
    }
    h->L.warps_per_block = h->launches[h->main_launch].warps_per_block;

    // zeroed buffers are the state "before slot 1"
    const struct { void* p; size_t n; } z[] = {{b->workspace, sz.workspace}, {b->counters, sz.counters},
                                               {b->trace, sz.trace},         {b->hist, sz.hist},
                                               {b->complog, sz.complog},     {b->scratch, sz.scratch}};
    for (const auto& it : z) {
        if (it.p && it.n) {
            e = cudaMemset(it.p, 0, it.n);
            if (e != cudaSuccess) { h->last_cuda = (int)e; return fail(FCSIM_ECUDA); }
        }
    }
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { h->last_cuda = (int)e; return fail(FCSIM_ECUDA); }

    Params& p = h->params;
    std::memset(&p, 0, sizeof(p));
    p.M = cfg->M; p.K = cfg->K; p.Qcap = cfg->Qcap; p.Acap = cfg->Acap;
    p.S = L.S; p.Apad = L.Apad;
    p.qmask = L.QC - 1; p.gq_off = (uint32_t)L.gq_off; p.qwin_off = (uint32_t)L.qwin_off;
    p.key0 = (uint32_t)(cfg->seed & 0xffffffffu);
    p.key1 = (uint32_t)(cfg->seed >> 32);
    p.n_classes = cfg->n_classes; p.n_groups = cfg->n_groups; p.n_replicas = (int)L.R;
    p.trace_stride = cfg->trace_stride; p.n_rec = trace_window_recs > 0 ? trace_window_recs : L.n_rec;
    p.rec_base = 0;
    p.hist_bins = cfg->hist_bins; p.hist_shift = cfg->hist_shift; p.complog_cap = cfg->complog_cap;
    p.gpool = h->d_gpool;
    p.bclass = h->d_bclass;
    p.qcnt_off = (uint32_t)L.qcnt_off;
    p.tstage_off = (uint32_t)L.tstage_off;
    p.state_bytes = (uint32_t)L.state_bytes;
    p.has_v = L.has_v;
    p.prof_mask = L.prof_mask;
    p.pool = h->d_pool; p.tables = h->d_tables; p.arrivals = h->d_arrivals;
    p.groups = h->d_pgroups;  // narrowed to the policy's piece at every launch
    p.workspace = static_cast<unsigned char*>(b->workspace);
    p.ws_stride = L.ws_stride;
    p.counters = static_cast<long long*>(b->counters);
    p.trace = L.n_rec > 0 ? static_cast<int2*>(b->trace) : nullptr;
    p.hist = cfg->hist_bins > 0 ? static_cast<int*>(b->hist) : nullptr;
    p.complog = cfg->complog_cap > 0 ? static_cast<int2*>(b->complog) : nullptr;
    p.work_counter = h->d_work;
    p.debug = h->d_work + 8;
    p.smem_per_warp = (uint32_t)L.smem_per_warp;
    *out = h;
    return FCSIM_OK;
}

// Slots of one launch.  Bounded by the work of a launch (its duration) and by the 32-bit partial sums that the
// step kernel keeps per launch and folds into the 64-bit counters at its end.  With n slots per launch:
//   sum of |P| + |Q| per slot          <= (Qcap + 2 Acap) n      (the queue may hold Qcap + Acap after evictions)
//   tokens generated, completions      <= Acap n
//   arrivals                           <= 255 n
//   output lengths of the completions, per lane <= Acap n + M    (tokens made in the launch plus those the
//                                                                 requests running at its start already held)
// so n <= (2^32 - 2^30 - 1) / (Qcap + 2 Acap) keeps all of them exact (M <= 2^30); with Qcap + Acap <= 2^20 that
// is at least 1536 slots.
extern "C" int fcsim_create(const fcsim_config* cfg, const fcsim_buffers* b, fcsim_t** out) {
    return create_handle(cfg, b, out, 0);
}

static int max_steps_per_launch(const fcsim* h) {
    long long s = kTargetWorkPerLaunch / std::max<long long>(1, h->L.R);
    s = std::max<long long>(256, std::min<long long>(s, kMaxStepsPerLaunch));
    const long long per_slot = (long long)h->cfg.Qcap + 2LL * h->cfg.Acap;
    s = std::min<long long>(s, ((1LL << 32) - (1LL << 30) - 1) / per_slot);
    return (int)std::max<long long>(1, s);
}

// One group of concurrent launches (one kernel per policy present) advancing every replica by `now` slots.
static int launch_slots(fcsim* h, int now, cudaStream_t st) {
    CUDA_TRY(h, cudaMemsetAsync(h->d_work, 0, 8 * sizeof(unsigned int), st));  // one work counter per policy
    if (h->launches.size() > 1) CUDA_TRY(h, cudaEventRecord(h->fork, st));
    for (const PolicyLaunch& pl : h->launches) {
        cudaStream_t ls = pl.side ? pl.side : st;
        if (pl.side) CUDA_TRY(h, cudaStreamWaitEvent(pl.side, h->fork, 0));
        Params p = h->params;
        p.t0 = h->t_done;
        p.n_steps = now;
        p.groups = h->d_pgroups + pl.pg_off;
        p.n_groups = pl.pg_cnt;
        p.n_work = pl.n_work;
        p.work_counter = h->d_work + pl.policy;
        p.tabcache_off = (uint32_t)pl.tabcache_off;
        {
            // the limit is a property of the kernel, not of the handle: another handle may have lowered it since
            std::lock_guard<std::mutex> lock(g_kernel_attr_mutex);
            CUDA_TRY(h, cudaFuncSetAttribute(pl.kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_block));
            pl.kernel<<<pl.grid, pl.warps_per_block * 32, pl.smem_block, ls>>>(p);
            CUDA_TRY(h, cudaGetLastError());
        }
        if (pl.side) CUDA_TRY(h, cudaEventRecord(pl.done, pl.side));
    }
    for (const PolicyLaunch& pl : h->launches)
        if (pl.side) CUDA_TRY(h, cudaStreamWaitEvent(st, pl.done, 0));
    h->t_done += now;
    return FCSIM_OK;
}

extern "C" int fcsim_run(fcsim_t* h, int32_t n_steps, void* cuda_stream) {
    if (!h || n_steps < 0) return FCSIM_EINVAL;
    if ((long long)h->t_done + n_steps > h->cfg.T_max) return FCSIM_ERANGE;
    if (int rc = check_device(h)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int per = max_steps_per_launch(h);
    int left = n_steps;
    while (left > 0) {
        const int now = std::min(left, per);
        if (int rc = launch_slots(h, now, st)) return rc;
        left -= now;
    }
    return FCSIM_OK;
}

static double percentile(const long long* hist, int bins, int shift, long long n, int q, long long max_lat) {
    if (n <= 0 || bins <= 0) return 0.0;
    const long long target = (q * n + 99) / 100;
    long long cum = 0;
    int k = 0;
    for (; k < bins; ++k) {
        cum += hist[k];
        if (cum >= target) break;
    }
    if (k >= bins - 1) return (double)max_lat;
    return (double)((((long long)k + 1) << shift) - 1);
}

// The group rows of a statistics call: cleared, reduced on the device into `d_rows` (layout: scratch_words) and
// the part the host needs copied to `host_rows`, all on `st`.  Nothing is allocated here.
static int reduce_groups(fcsim* h, cudaStream_t st, long long* d_rows, long long* host_rows) {
    const int G = (int)h->groups.size();
    const int bins = h->cfg.hist_bins;
    const int R = (int)h->L.R;
    const bool with_log = h->cfg.complog_cap > 0;
    long long* d_cnt = d_rows;
    long long* d_hist = d_cnt + (size_t)G * C_COUNT;
    long long* d_res = d_hist + (size_t)G * bins;
    unsigned long long* d_hi = reinterpret_cast<unsigned long long*>(d_res + (size_t)G * kSelResultWords);
    unsigned long long* d_lo = d_hi + (size_t)G * kSelBins;
    // the area still holds the rows of the previous call: the sums must start from zero
    CUDA_TRY(h, cudaMemsetAsync(d_rows, 0, scratch_words(G, bins, h->cfg.complog_cap) * 8, st));
    const int n_chunks = (R + kStatsChunk - 1) / kStatsChunk;
    {
        const int warps_per_block = 8;
        const int blocks = std::max(1, std::min((n_chunks + warps_per_block - 1) / warps_per_block, h->sm_count * 8));
        reduce_counters_kernel<<<blocks, warps_per_block * 32, 0, st>>>(
            static_cast<const long long*>(h->buf.counters), h->d_groups, G, R, kStatsChunk, d_cnt);
        CUDA_TRY(h, cudaGetLastError());
    }
    if (bins > 0) {
        const int blocks = std::max(1, std::min(n_chunks, h->sm_count * 16));
        launch_reduce_hist(static_cast<const int*>(h->buf.hist), h->d_groups, G, R, bins, blocks, d_hist, st);
        CUDA_TRY(h, cudaGetLastError());
    }
    if (with_log) {
        const int chunk = kSelChunk;
        const int blocks = std::max(1, std::min((R + chunk - 1) / chunk, h->sm_count * 8));
        const int2* log = static_cast<const int2*>(h->buf.complog);
        const long long* cnt = static_cast<const long long*>(h->buf.counters);
        latency_digit_kernel<1><<<blocks, 256, 0, st>>>(log, cnt, h->d_groups, G, R, h->cfg.complog_cap, chunk, d_res, d_hi);
        CUDA_TRY(h, cudaGetLastError());
        latency_select_kernel<1><<<G, 256, 0, st>>>(d_hi, d_res);
        CUDA_TRY(h, cudaGetLastError());
        latency_digit_kernel<2><<<blocks, 256, 0, st>>>(log, cnt, h->d_groups, G, R, h->cfg.complog_cap, chunk, d_res, d_lo);
        CUDA_TRY(h, cudaGetLastError());
        latency_select_kernel<2><<<G, 256, 0, st>>>(d_lo, d_res);
        CUDA_TRY(h, cudaGetLastError());
    }
    CUDA_TRY(h, cudaMemcpyAsync(host_rows, d_rows, scratch_words_to_host(G, bins, h->cfg.complog_cap) * 8,
                                cudaMemcpyDeviceToHost, st));
    return FCSIM_OK;
}

// Per-group summaries from the reduced rows (host arithmetic: one division per figure).
static void fill_summaries(const fcsim* h, const long long* rows, fcsim_summary* per_group_out) {
    const int G = (int)h->groups.size();
    const int bins = h->cfg.hist_bins;
    const double T = (double)h->t_done;
    const long long* res = rows + (size_t)G * ((size_t)C_COUNT + bins);
    for (int g = 0; g < G; ++g) {
        fcsim_summary& s = per_group_out[g];
        std::memcpy(&s.total, rows + (size_t)g * C_COUNT, sizeof(fcsim_counters));
        const double n = (double)h->groups[g].n_replicas;
        const fcsim_counters& c = s.total;
        s.mean_latency = c.completed > 0 ? (double)c.sum_lat / (double)c.completed : 0.0;
        s.mean_utilisation = T > 0 ? (double)c.sum_U / (n * T * (double)h->cfg.M) : 0.0;
        s.request_throughput = T > 0 ? (double)c.completed / (n * T) : 0.0;
        s.token_throughput = T > 0 ? (double)c.tokens_generated / (n * T) : 0.0;
        s.percentile_source = FCSIM_PCT_NONE;
        s.reserved = 0;
        s.p95_latency = s.p99_latency = 0.0;
        const long long* sel = res + (size_t)g * kSelResultWords;
        if (h->cfg.complog_cap > 0 && c.completed > 0 && (c.status & 2) == 0 && sel[0] == c.completed) {
            // every completion of the group is in the log: the order statistics themselves
            s.p95_latency = (double)sel[1];
            s.p99_latency = (double)sel[2];
            s.percentile_source = FCSIM_PCT_EXACT;
        } else if (bins > 0 && c.completed > 0) {
            const long long* gh = rows + (size_t)G * C_COUNT + (size_t)g * bins;
            s.p95_latency = percentile(gh, bins, h->cfg.hist_shift, c.completed, 95, c.max_lat);
            s.p99_latency = percentile(gh, bins, h->cfg.hist_shift, c.completed, 99, c.max_lat);
            s.percentile_source = FCSIM_PCT_HISTOGRAM;
        }
    }
}

extern "C" int fcsim_stats(fcsim_t* h, void* cuda_stream, fcsim_counters* host_out, fcsim_summary* per_group_out) {
    if (!h) return FCSIM_EINVAL;
    if (int rc = check_device(h)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int G = (int)h->groups.size();
    const int R = (int)h->L.R;
    std::vector<long long> host_rows;
    if (per_group_out) {
        try {
            host_rows.resize(scratch_words_to_host(G, h->cfg.hist_bins, h->cfg.complog_cap));
        } catch (...) {
            return FCSIM_ENOMEM;
        }
        if (int rc = reduce_groups(h, st, static_cast<long long*>(h->buf.scratch), host_rows.data())) return rc;
    }
    if (host_out)
        CUDA_TRY(h, cudaMemcpyAsync(host_out, h->buf.counters, (size_t)R * sizeof(fcsim_counters),
                                    cudaMemcpyDeviceToHost, st));
    CUDA_TRY(h, cudaStreamSynchronize(st));
    if (per_group_out) fill_summaries(h, host_rows.data(), per_group_out);
    return FCSIM_OK;
}

// ---- statistics without any allocation --------------------------------------------------------------
// For callers that cannot allocate device memory (a process whose allocator already owns the whole GPU,
// a thread that must avoid the device-wide synchronisation of cudaMalloc/cudaFree).  The per-group rows
// that fcsim_stats keeps in the caller's scratch buffer live here in a fixed array of the device image.
// On the host the array's name is only a stand-in for the symbol, never a device address: its address
// on the current device is queried once per device with cudaGetSymbolAddress and that pointer is what
// the kernels get.
static __device__ __align__(256) long long g_noalloc_scratch[FCSIM_NOALLOC_SCRATCH_WORDS];
static long long g_noalloc_host_rows[FCSIM_NOALLOC_SCRATCH_WORDS];   // host staging for the copy back
constexpr int kNoallocMaxDevices = 64;
static long long* g_noalloc_dev_ptr[kNoallocMaxDevices] = {nullptr};

extern "C" int fcsim_stats_noalloc(fcsim_t* h, void* cuda_stream, fcsim_summary* per_group_out) {
    if (!h || !per_group_out) return FCSIM_EINVAL;
    const int G = (int)h->groups.size();
    const size_t words = scratch_words(G, h->cfg.hist_bins, h->cfg.complog_cap);
    if (words > (size_t)FCSIM_NOALLOC_SCRATCH_WORDS) return FCSIM_ETOOBIG;
    int dev = -1;
    CUDA_TRY(h, cudaGetDevice(&dev));
    if (dev < 0 || dev >= kNoallocMaxDevices || dev != h->device) return FCSIM_EINVAL;
    if (!g_noalloc_dev_ptr[dev]) {   // set-up, once per device, with that device current
        void* sym = nullptr;
        CUDA_TRY(h, cudaGetSymbolAddress(&sym, g_noalloc_scratch));
        g_noalloc_dev_ptr[dev] = static_cast<long long*>(sym);
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (int rc = reduce_groups(h, st, g_noalloc_dev_ptr[dev], g_noalloc_host_rows)) return rc;
    CUDA_TRY(h, cudaStreamSynchronize(st));
    fill_summaries(h, g_noalloc_host_rows, per_group_out);
    return FCSIM_OK;
}

extern "C" int fcsim_destroy(fcsim_t* h) {
    if (!h) return FCSIM_EINVAL;
    release(h);
    return FCSIM_OK;
}

extern "C" int32_t fcsim_steps_done(const fcsim_t* h) { return h ? h->t_done : -1; }

extern "C" int fcsim_get_launch_info(const fcsim_t* h, fcsim_launch_info* out) {
    if (!h || !out) return FCSIM_EINVAL;
    const PolicyLaunch& pl = h->launches[h->main_launch];  // the policy with the most replicas
    out->grid = pl.grid;
    out->block = pl.warps_per_block * 32;
    out->warps_per_block = pl.warps_per_block;
    out->blocks_per_sm = pl.blocks_per_sm;
    out->sm_count = h->sm_count;
    out->smem_per_block = (int32_t)pl.smem_block;
    out->smem_per_warp = (int32_t)h->L.smem_per_warp;
    out->max_steps_per_launch = max_steps_per_launch(h);
    return FCSIM_OK;
}

extern "C" int fcsim_last_cuda_error(const fcsim_t* h) { return h ? h->last_cuda : 0; }

extern "C" const char* fcsim_last_cuda_error_name(const fcsim_t* h) {
    return cudaGetErrorName(static_cast<cudaError_t>(h ? h->last_cuda : 0));
}

extern "C" int fcsim_debug_read(fcsim_t* h, uint32_t out[8]) {
    if (!h || !out) return FCSIM_EINVAL;
    CUDA_TRY(h, cudaMemcpy(out, h->d_work + 8, 8 * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    return FCSIM_OK;
}

extern "C" int fcsim_is_checked_build(void) {
#ifdef FCSIM_CHECKED
    return 1;
#else
    return 0;
#endif
}

extern "C" const char* fcsim_strerror(int code) {
    switch (code) {
        case FCSIM_OK: return "ok";
        case FCSIM_EINVAL: return "invalid argument or configuration";
        case FCSIM_ECAP: return "Qcap/Acap do not fit the shared memory of one warp";
        case FCSIM_ESIZE: return "a required buffer is missing, misaligned or too small";
        case FCSIM_ERANGE: return "steps beyond T_max";
        case FCSIM_ECUDA: return "CUDA runtime error";
        case FCSIM_ENOMEM: return "host allocation failed";
        case FCSIM_ETOOBIG: return "group rows exceed the fixed device scratch of fcsim_stats_noalloc";
        default: return "unknown error";
    }
}

// Whole job with host buffers.  A large trace does not wait for the end of the run: the device holds two
// windows of the horizon (a few thousand records per replica each); while the kernels fill one, the other, already
// full, travels to the caller's rows with one strided copy on a second stream.  The rest of the outputs (counters,
// histograms, completion log) is copied after the last slot.
extern "C" int fcsim_simulate_host(const fcsim_config* cfg, int32_t n_steps, fcsim_counters* host_counters,
                                   void* host_trace, void* host_hist, void* host_complog,
                                   fcsim_summary* per_group_out) {
    fcsim_sizes sz;
    int rc = fcsim_query_sizes(cfg, &sz);
    if (rc != FCSIM_OK) return rc;
    if (n_steps < 0 || n_steps > cfg->T_max) return FCSIM_ERANGE;
    Layout L;
    plan(cfg, &L);
    // Streaming pays when the trace is large and a replica's piece of a window is long enough for the strided
    // copy to run at full speed (16 KB and more; rows of a few KB copy at a fraction of it).
    const long long stride = cfg->trace_stride;
    const long long recs_run = stride > 0 ? n_steps / stride : 0;
    long long win_recs = 0;
    if (host_trace && sz.trace >= ((size_t)256 << 20) && recs_run >= 3 * 2048) {
        win_recs = std::max<long long>(2048, (((long long)64 << 20) / (L.R * 8) + 31) / 32 * 32);
        // a window is filled by whole launches
        const long long per_launch = ((1LL << 31) / std::max<long long>(1, L.R)) / (32 * stride) * 32;
        win_recs = std::min(win_recs, std::max<long long>(0, per_launch));
        if (win_recs < 2048 || win_recs * 3 > recs_run) win_recs = 0;
    }
    fcsim_buffers b;
    std::memset(&b, 0, sizeof(b));
    void** slots[6] = {&b.workspace, &b.counters, &b.trace, &b.hist, &b.complog, &b.scratch};
    size_t bytes[6] = {sz.workspace, sz.counters, sz.trace, sz.hist, sz.complog, sz.scratch};
    if (win_recs > 0) bytes[2] = 2 * (size_t)L.R * (size_t)win_recs * 8;
    cudaStream_t run_st = nullptr, copy_st = nullptr;
    cudaEvent_t filled[2] = {nullptr, nullptr}, sent[2] = {nullptr, nullptr};
    fcsim_t* h = nullptr;
    void* arena = nullptr;  // one device allocation for all the buffers
    auto free_all = [&]() {
        if (h) fcsim_destroy(h);
        cudaFree(arena);
        for (int i = 0; i < 2; ++i) {
            if (filled[i]) cudaEventDestroy(filled[i]);
            if (sent[i]) cudaEventDestroy(sent[i]);
        }
        if (run_st) cudaStreamDestroy(run_st);
        if (copy_st) cudaStreamDestroy(copy_st);
    };
    size_t total = 0;
    for (int i = 0; i < 6; ++i) total += align_up(bytes[i], 256);
    if (cudaMalloc(&arena, std::max<size_t>(total, 256)) != cudaSuccess) return FCSIM_ECUDA;
    {
        size_t off = 0;
        for (int i = 0; i < 6; ++i) {
            if (bytes[i]) *slots[i] = static_cast<unsigned char*>(arena) + off;
            off += align_up(bytes[i], 256);
        }
    }
    rc = create_handle(cfg, &b, &h, (int)win_recs);
    if (rc != FCSIM_OK) { free_all(); return rc; }
    if (win_recs == 0) {
        rc = fcsim_run(h, n_steps, nullptr);
    } else {
        cudaError_t e = cudaStreamCreateWithFlags(&run_st, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&copy_st, cudaStreamNonBlocking);
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&filled[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sent[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) { free_all(); return FCSIM_ECUDA; }
        const size_t win_bytes = (size_t)L.R * (size_t)win_recs * 8;
        const size_t row_bytes = (size_t)L.n_rec * 8;  // the caller's rows hold the whole horizon
        const int per = max_steps_per_launch(h);
        long long rec0 = 0;
        for (int piece = 0; rc == FCSIM_OK && h->t_done < n_steps; ++piece) {
            const int buf = piece & 1;
            const long long slots_now = std::min<long long>(win_recs * stride, (long long)n_steps - h->t_done);
            const long long recs_now = (h->t_done + slots_now) / stride - rec0;
            unsigned char* win = static_cast<unsigned char*>(b.trace) + (size_t)buf * win_bytes;
            if (piece >= 2 && cudaStreamWaitEvent(run_st, sent[buf], 0) != cudaSuccess) { rc = FCSIM_ECUDA; break; }
            h->params.trace = reinterpret_cast<int2*>(win);
            h->params.rec_base = (int32_t)rec0;
            long long left = slots_now;
            while (rc == FCSIM_OK && left > 0) {
                const int now = (int)std::min<long long>(left, per);
                rc = launch_slots(h, now, run_st);
                left -= now;
            }
            if (rc != FCSIM_OK) break;
            e = cudaEventRecord(filled[buf], run_st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(copy_st, filled[buf], 0);
            if (e == cudaSuccess && recs_now > 0)
                e = cudaMemcpy2DAsync(static_cast<unsigned char*>(host_trace) + (size_t)rec0 * 8, row_bytes, win,
                                      (size_t)win_recs * 8, (size_t)recs_now * 8, (size_t)L.R, cudaMemcpyDeviceToHost,
                                      copy_st);
            if (e == cudaSuccess) e = cudaEventRecord(sent[buf], copy_st);
            if (e != cudaSuccess) { h->last_cuda = (int)e; rc = FCSIM_ECUDA; }
            rec0 += recs_now;
        }
        if (rc == FCSIM_OK && cudaStreamSynchronize(run_st) != cudaSuccess) rc = FCSIM_ECUDA;
    }
    if (rc == FCSIM_OK) rc = fcsim_stats(h, run_st, host_counters, per_group_out);
    if (rc == FCSIM_OK) {
        cudaError_t e = cudaSuccess;
        if (win_recs > 0) {
            e = cudaStreamSynchronize(copy_st);
            // records of slots that were not run read as zero, as in a freshly created trace buffer
            if (e == cudaSuccess && recs_run < L.n_rec)
                for (long long r = 0; r < L.R; ++r)
                    std::memset(static_cast<unsigned char*>(host_trace) + ((size_t)r * L.n_rec + (size_t)recs_run) * 8, 0,
                                (size_t)(L.n_rec - recs_run) * 8);
        } else if (host_trace && sz.trace) {
            e = cudaMemcpy(host_trace, b.trace, sz.trace, cudaMemcpyDeviceToHost);
        }
        if (e == cudaSuccess && host_hist && sz.hist) e = cudaMemcpy(host_hist, b.hist, sz.hist, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess && host_complog && sz.complog) {
            // rows are rarely full: with the counters on the host only the longest logged prefix of the rows travels
            long long longest = cfg->complog_cap;
            if (host_counters) {
                longest = 0;
                for (long long r = 0; r < L.R; ++r) longest = std::max<long long>(longest, host_counters[r].n_logged);
            }
            if (longest > 0)
                e = cudaMemcpy2D(host_complog, (size_t)cfg->complog_cap * 8, b.complog, (size_t)cfg->complog_cap * 8,
                                 (size_t)longest * 8, (size_t)L.R, cudaMemcpyDeviceToHost);
        }
        if (e != cudaSuccess) rc = FCSIM_ECUDA;
    }
    free_all();
    return rc;
}
