// Device side of fcsim: one warp advances one replica of the serving model of Section 2.1, slot by slot,
// under Algorithm 2, Algorithm 1, or one of the baselines (greedy, chunked prefill, alpha-protection greedy,
// MC benchmark).
//
// Data layout per replica:
//   ring  [Acap] u64   the active set in activation order, a ring in shared memory while a warp owns the replica
//                      (the same bytes in the caller's workspace between launches);
//                      entry = l | o << 16 | t_arr << 32 | class << 56.
//   state [Acap] u32   one word per active entry (same ring index): for a request whose prompt is in the cache
//                      the slot in which its last token is generated (t_fin = activation slot + o - 1, so its
//                      output count is implied by the slot number and "process all requests" costs nothing);
//                      for a request still prefilling (chunked policy) 0x80000000 | prompt tokens prefilled so
//                      far; 0x40000000 | slot of completion for a request that has completed but whose entry
//                      has not been squeezed out yet (completed entries are removed lazily, many at a time,
//                      and their latency statistics are taken then, one entry per lane).
//   vproj [Acap] i32   only with MC groups, entry form: projected memory usage of the last slot of each active entry.
//   uprof [H]    i32   only with MC groups, profile form (used when H <= Acap, H the power of two above the longest
//                      output length): projected memory usage of the future slots, a ring indexed by slot & (H - 1);
//                      takes the place of vproj.
//   queue [QC]   u64   the FIFO waiting queue, a ring in the replica's record in GLOBAL memory (QC a power of
//                      two >= Qcap + Acap: evictions may push the queue past Qcap).  It is touched at its ends
//                      only: arrivals are appended (plain stores, nobody waits for them), the head is read
//                      through qwin, evicted requests are pushed back on the head (Section 3.3: LIFO eviction
//                      to the queue front keeps "active set, then queue" sorted by arrival).  Keeping the queue
//                      out of shared memory is what lets more warps reside on an SM.
//   qwin  [64]   u64   shared-memory copy of the queue entries with sequence numbers [wseq, wseq + 64), slot =
//                      sequence number & 63; the head is always inside, and the window is topped up from global
//                      memory 32 entries at a time, long before they are needed.
//                      Under Algorithm 1 a pick may leave the middle of the queue (first request of a
//                      class); the entries ahead of it then shift by one place.
//   stage [S]    u64   arrivals generated ahead of time for the next batch of <= 32 slots.
//   qcnt  [classes] u32  only with Algorithm-1 groups: waiting requests per class.
// Only ring, state and vproj are saved between launches (plus 16 scalar words); the queue lives in global memory
// and the rest is rebuilt.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace fcsim_dev {

constexpr int kWarpsPerBlock = 4;
constexpr int kHeaderWords = 16;  // per-replica scalar state kept in the workspace
constexpr uint32_t kNoFin = 0xFFFFFFFFu;
constexpr uint32_t kPrefillBit = 0x80000000u;
constexpr uint32_t kDead = 0x40000000u;  // state word of a completed entry awaiting removal: kDead | slot of completion
                                         // (its latency statistics are taken when it is squeezed out)
__device__ __forceinline__ bool is_dead(uint32_t sw) { return (sw >> 30) == 1u; }  // bit 31 marks a prefilling entry

enum CounterIdx {
    C_STEPS_DONE = 0, C_STATUS, C_ARRIVED, C_DROPPED, C_ADMITTED, C_COMPLETED, C_EVICTIONS,
    C_OVERFLOW_STEPS, C_GATE_BLOCKED, C_BUDGET_BLOCKED, C_ACAP_BLOCKED, C_TOKENS_GENERATED,
    C_PREFILL_TOKENS, C_COMPLETED_TOKENS, C_WASTED_TOKENS, C_SUM_LAT, C_MAX_LAT, C_SUM_U, C_MAX_U,
    C_SUM_N, C_MAX_Q, C_SUM_W_COMPLETED, C_N_LOGGED, C_Q_FINAL, C_P_FINAL, C_RESID_AGE, C_RESID_J,
    C_MMPP_STATE, C_COUNT
};

struct DevTable {
    uint32_t off;  // first threshold in the pool
    uint32_t n;
    int32_t vmin;
    uint32_t guide;  // 0 = none; else bits 27..31: g (mantissa bits), 22..26: J (levels), 0..21: first record in the guide pool
};
struct DevArrivals {
    DevTable count[2];
    uint32_t thr[2];
    uint32_t n_states;
    uint32_t pad;
};
struct DevGroup {
    int32_t policy;
    uint32_t b_fp;
    int32_t chunk;
    int32_t arrivals_id;
    uint32_t rng_base;
    int32_t first;  // index of the group's first replica
    int32_t n;
    int32_t admit_limit;  // usage a new admission may reach: M, or (1-alpha) M for the alpha-protection policy
    int32_t bclass_off;   // Algorithm 1: index of the group's per-class budgets in Params::bclass
    int32_t mc_worst;     // MC benchmark: project with the class's longest output length
    int32_t keep;         // 1 = an evicted request keeps its generated tokens as prompt: (l, o) <- (l + j, o - j)
    int32_t wfirst;       // index of the group's first replica among the work items of its policy's launch
};

struct Params {
    int32_t M, K, Qcap, Acap, S, Apad;  // Apad: padded storage size of the active ring
    uint32_t qmask;               // queue ring size - 1 (a power of two)
    uint32_t gq_off;              // byte offset of the queue ring in a replica's workspace record
    uint32_t key0, key1;
    int32_t n_classes, n_groups, n_replicas;  // n_groups: entries of `groups`
    int32_t n_work;               // replicas this launch advances (those of the groups in `groups`)
    int32_t trace_stride, n_rec, hist_bins, hist_shift, complog_cap;  // n_rec: records a trace row holds
    int32_t rec_base;             // index of the first record the trace rows hold (0 unless the buffer is a window
                                  // on the horizon that the host moves from launch to launch)
    int32_t t0, n_steps;
    const uint32_t* pool;         // all thresholds
    const uint4* gpool;           // guide records {k0, thresholds k0, k0+1, k0+2}, one per bucket of u
    const int32_t* bclass;        // per-class budgets b_k of the Algorithm-1 groups
    uint32_t qcnt_off;            // byte offset of the per-class queue counts in a warp's shared memory (0 = none)
    uint32_t qwin_off;            // byte offset of the queue window in a warp's shared memory
    uint32_t tabcache_off;        // byte offset in the CTA's shared memory of a copy of `tables` (0 = none)
    uint32_t state_bytes;         // ring + state words (+ projection words): what is saved between launches
    int32_t has_v;                // 1 = the MC benchmark's projection words follow the state words
    uint32_t prof_mask;           // MC benchmark: 0 = one projection word per active entry; else H - 1, the words are
                                  // the projected usage of the future slots (ring of H slots)
    uint32_t tstage_off;          // byte offset of the trace staging area (2 x 32 records) in a warp's shared
                                  // memory; 0 = records are kept in registers and stored with plain stores
    const DevTable* tables;       // [0] class law, [1 .. nc] prompt, [1+nc .. 2nc] decode
    const DevArrivals* arrivals;
    const DevGroup* groups;       // the groups of this launch's policy, in replica order
    unsigned char* workspace;     // [R] records of ws_stride bytes
    unsigned long long ws_stride;
    long long* counters;          // [R][C_COUNT]
    int2* trace;
    int* hist;
    int2* complog;
    unsigned int* work_counter;
    unsigned int* debug;          // 8 words: first failed index check (checked build), else untouched
    uint32_t smem_per_warp;
};

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and xors,
// key schedule k += (0x9E3779B9, 0xBB67AE85).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t& o0, uint32_t& o1, uint32_t& o2,
                                              uint32_t& o3) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    o0 = c0; o1 = c1; o2 = c2; o3 = c3;
}

// Inverse-CDF lookup: vmin + (first k < n-1 with thresholds[k] > u, else n-1).
// A table with a guide answers with ONE 16-byte load in all but rare cases.  The 32-bit range of u is cut into
// buckets; the record of a bucket holds k0, the first index whose threshold exceeds the bucket's lowest u, and the
// thresholds k0, k0+1, k0+2 (0xffffffff where there is none), so the answer is k0 plus the number of those that
// are <= u.  Only when all three are (a bucket with more than three thresholds, or the very top of the range)
// does a binary search over the thresholds from k0+3 finish the job.
// Buckets: with v = ~u and j = min(clz(v), J), bucket (j, m) takes the g bits m that follow the leading one of
// v (for j == J: the g bits after J leading zeros).  J = 0 gives 2^g equal buckets; J > 0 halves the bucket
// width with every leading one of u, which keeps the long thin upper tail of a geometric or lognormal law at a
// few thresholds per bucket.  The host picks (g, J) per table.
__device__ __forceinline__ uint32_t guide_bucket(uint32_t guide, uint32_t u) {
    const uint32_t g = guide >> 27, J = (guide >> 22) & 31u;
    const uint32_t v = ~u;
    const uint32_t j = min((uint32_t)__clz((int)v), J);
    const uint32_t sh = j + (j < J ? 1u : 0u);  // bits before the mantissa; <= 31 because J <= 30
    return (guide & 0x3fffffu) + (j << g) + ((v << sh) >> (32u - g));
}
__device__ __forceinline__ int guide_finish(const uint32_t* __restrict__ cdf, uint32_t n, uint4 rec, uint32_t u) {
    uint32_t k = rec.x + (rec.y <= u ? 1u : 0u) + (rec.z <= u ? 1u : 0u) + (rec.w <= u ? 1u : 0u);
    if (rec.w <= u) {
        uint32_t hi = n - 1;
        while (k < hi) {
            const uint32_t mid = (k + hi) >> 1;
            if (__ldg(cdf + mid) > u) hi = mid; else k = mid + 1;
        }
    }
    return (int)min(k, n - 1);
}
__device__ __forceinline__ int sample_table(const uint32_t* __restrict__ pool, const uint4* __restrict__ gpool,
                                            const DevTable tb, uint32_t u) {
    const uint32_t* __restrict__ cdf = pool + tb.off;
    if (tb.guide >> 27) return tb.vmin + guide_finish(cdf, tb.n, __ldg(gpool + guide_bucket(tb.guide, u)), u);
    uint32_t lo = 0, hi = tb.n - 1;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (__ldg(cdf + mid) > u) hi = mid; else lo = mid + 1;
    }
    return tb.vmin + (int)lo;
}

// Bulk asynchronous copy shared -> global of one staged block of trace records (TMA engine, no tensor map).
// Both addresses must be 16-byte aligned and the size a multiple of 16; the caller checks that.
__device__ __forceinline__ void bulk_store_commit(void* gdst, const void* ssrc, uint32_t bytes) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(ssrc);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // staged records visible to the async proxy
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(s), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Wait until at most `pending` of this thread's bulk copies have not finished READING their source.
template <int kPending>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kPending) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Two independent lookups (prompt and decode length of one arrival): both records are requested before either
// is used, so that their round trips to the L2 overlap.
__device__ __forceinline__ void sample_pair(const uint32_t* __restrict__ pool, const uint4* __restrict__ gpool,
                                            const DevTable ta, uint32_t ua, const DevTable tb, uint32_t ub, int& va,
                                            int& vb) {
    if ((ta.guide >> 27) && (tb.guide >> 27)) {
        const uint4 ra = __ldg(gpool + guide_bucket(ta.guide, ua));
        const uint4 rb = __ldg(gpool + guide_bucket(tb.guide, ub));
        va = ta.vmin + guide_finish(pool + ta.off, ta.n, ra, ua);
        vb = tb.vmin + guide_finish(pool + tb.off, tb.n, rb, ub);
    } else {
        va = sample_table(pool, gpool, ta, ua);
        vb = sample_table(pool, gpool, tb, ub);
    }
}

__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}
__device__ __forceinline__ uint32_t lanemask_gt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_gt;" : "=r"(m));
    return m;
}

__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

__device__ __forceinline__ long long warp_sum64(long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// A value computed ONCE: it passes through a register move that the compiler will not repeat.  The lane and
// warp numbers and the warp's offsets in shared memory are cheap to derive from the thread index, so cheap that
// the compiler otherwise derives them again at most of their hundreds of uses instead of keeping them, which
// costs more than a tenth of all executed instructions.  Only integers take this route: a pointer would lose
// its address space on the way.
__device__ __forceinline__ uint32_t once(uint32_t v) { uint32_t r; asm("mov.b32 %0, %1;" : "=r"(r) : "r"(v)); return r; }
__device__ __forceinline__ int once(int v) { int r; asm("mov.b32 %0, %1;" : "=r"(r) : "r"(v)); return r; }

// A value that every lane of the warp holds, handed to the compiler as such: the result of a warp-wide reduction
// is uniform by construction, so conditions and loop bounds computed from it need no reconvergence bookkeeping.
__device__ __forceinline__ uint32_t uni(uint32_t v) { return __reduce_max_sync(0xffffffffu, v); }
__device__ __forceinline__ int uni(int v) { return (int)__reduce_max_sync(0xffffffffu, (uint32_t)v); }
__device__ __forceinline__ uint64_t uni(uint64_t v) {
    return ((uint64_t)__reduce_max_sync(0xffffffffu, (uint32_t)(v >> 32)) << 32) | __reduce_max_sync(0xffffffffu, (uint32_t)v);
}

__device__ __forceinline__ uint64_t pack_entry(int l, int o, int t_arr, int cls) {
    return (uint64_t)(uint32_t)(l | (o << 16)) | ((uint64_t)(uint32_t)(t_arr | (cls << 24)) << 32);
}
__device__ __forceinline__ int entry_l(uint64_t e) { return (int)((uint32_t)e & 0xffffu); }
__device__ __forceinline__ int entry_o(uint64_t e) { return (int)((uint32_t)e >> 16); }
__device__ __forceinline__ int entry_tarr(uint64_t e) { return (int)((uint32_t)(e >> 32) & 0xffffffu); }
__device__ __forceinline__ int entry_cls(uint64_t e) { return (int)(e >> 56); }

// Index-checked build (-DFCSIM_CHECKED): every shared-memory and output index is compared with its
// bound; a bad one is recorded (line, index, bound, replica) in Params::debug and the access goes to a
// dummy location instead, so a logic error shows up as a report, never as a memory fault.
#ifdef FCSIM_CHECKED
template <typename T>
__device__ __forceinline__ T& checked_ref(T* base, long long idx, long long limit, int line, unsigned int* dbg,
                                          unsigned int replica) {
    __shared__ T dummy[kWarpsPerBlock * 32];
    if (idx >= 0 && idx < limit) return base[idx];
    if (atomicCAS(dbg, 0u, (unsigned)line) == 0u) {
        dbg[1] = (unsigned)idx;
        dbg[2] = (unsigned)limit;
        dbg[3] = replica;
    }
    return dummy[threadIdx.x];
}
#define RING(i) checked_ref(ring, (i), Acap, __LINE__, p.debug, r)
#define STATE(i) checked_ref(state, (i), Acap, __LINE__, p.debug, r)
#define STAGE(i) checked_ref(stage, (i), S, __LINE__, p.debug, r)
#define TROW(i) checked_ref(trow + p.rec_base, (long long)(i) - p.rec_base, p.n_rec, __LINE__, p.debug, r)
#define LROW(i) checked_ref(lrow, (i), p.complog_cap, __LINE__, p.debug, r)
#define HROW(i) checked_ref(hrow, (i), p.hist_bins, __LINE__, p.debug, r)
#else
#define RING(i) ring[(i)]
#define STATE(i) state[(i)]
#define STAGE(i) stage[(i)]
#define TROW(i) trow[(i)]
#define LROW(i) lrow[(i)]
#define HROW(i) hrow[(i)]
#endif

// An arrival whose lengths have not been drawn yet waits in the queue as a placeholder: prompt field 0 (a real
// prompt has at least one token), slot of arrival, and, in the output-length field, its rank among the slot's
// arrivals, which together are the counter of its draw.  Only the queue ring in global memory and, for a moment,
// the window hold placeholders; convert_window draws the lengths of those inside the window, one per lane.
__device__ __forceinline__ bool is_placeholder(uint64_t e) { return ((uint32_t)e & 0xffffu) == 0u; }

__device__ __forceinline__ void convert_window(uint64_t* qwin, uint32_t wseq, uint32_t qh, int nQ, uint32_t rid,
                                            uint32_t key0, uint32_t key1, const uint32_t* __restrict__ pool,
                                            const uint4* __restrict__ gpool, const DevTable* tabs, int n_classes) {
    const uint32_t lane = threadIdx.x & 31u;
#pragma unroll 1
    for (uint32_t half = 0; half < 2u; ++half) {
        const uint32_t sq = wseq + 32u * half + lane;
        const bool in = sq - qh < (uint32_t)nQ;
        const uint64_t e = in ? qwin[sq & 63u] : 1ull;
        if (is_placeholder(e)) {
            uint32_t a0, a1, a2, a3;
            philox4x32_10((uint32_t)entry_tarr(e), rid, 1u, (uint32_t)entry_o(e), key0, key1, a0, a1, a2, a3);
            const int cls = sample_table(pool, gpool, tabs[0], a0);
            int l, o;
            sample_pair(pool, gpool, tabs[1 + cls], a1, tabs[1 + n_classes + cls], a2, l, o);
            qwin[sq & 63u] = pack_entry(l, o, entry_tarr(e), cls);
        }
    }
    __syncwarp();
}

// One launch advances the replicas of the groups that share one policy; a configuration with several
// policies is run as several launches that the host issues side by side.
// kPol: the policy, a compile-time constant: the slot loop is one long chain of short warp-uniform decisions,
// and every test of the policy that the compiler resolves shortens it (and frees the registers of the state
// that only other policies keep).
// kRec: what is recorded per slot: 0 = no trace and no completion log, 1 = trace only, 2 = whatever the
// parameters say (decided at run time).
// kExt (= kPol >= 4): the per-class activation of Algorithm 1 (policy 4) and the future-memory test of the MC
// benchmark (policy 5) use extra per-warp state (class counts, projection words).
// kPol 6 is the MC benchmark again, with its projection kept per future slot instead of per active entry
// (the host picks it when the longest output length is short next to the active set's storage).
// kMinCtas: resident CTAs per SM the register allocation must allow (5: <= 96 registers, 6: <= 80, 7: <= 72,
// 8: <= 64).  The host asks the occupancy calculator about all of them.
// kBulk: the whole-prompt first-come-first-served policies (0, 1, 3, 6) first try to activate several queue heads at
// once; the host asks for it when two or more requests arrive (and may be activated) per slot on average.  With
// fewer the extra code only costs.
// kLazy: arrivals that join a long queue wait as placeholders and are drawn when the window on the queue reaches
// them.  The host asks for it when most arrivals are dropped anyway (heavy overload); elsewhere the extra code
// costs more than the draws it saves.
template <int kPol, int kMinCtas, int kRec, bool kBulk, bool kLazy>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, kMinCtas) fcsim_step_kernel(const Params p) {
    constexpr bool kExt = kPol >= 4;
    constexpr bool kMcProfile = kPol == 6;  // MC benchmark, projection per future slot
    // Completed entries tolerated inside the active range before they are squeezed out (they always are when the
    // storage runs out).  The whole-prompt policies touch the range only where a request finishes, so removal
    // as late as possible measured fastest; the policies that walk the range (chunked prefills, Algorithm 1's
    // storage check, the MC projections) want it short.
    constexpr int kCompactAt = (kPol <= 1 || kPol == 3 || kPol == 6) ? 256 : 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // the table descriptors of the length laws are read for every generated arrival: the host reserves room
    // for a copy behind the warps' slices when that does not cost a resident CTA
    const bool tab_shared = p.tabcache_off != 0;
    DevTable* s_tables = reinterpret_cast<DevTable*>(smem_raw + p.tabcache_off);
    if (tab_shared) {
        for (int i = threadIdx.x; i < 1 + 2 * p.n_classes; i += blockDim.x) s_tables[i] = p.tables[i];
    }
    __syncthreads();
    const DevTable* __restrict__ tabs = tab_shared ? s_tables : p.tables;
    const int lane = once((int)(threadIdx.x & 31));
    const int warp = once((int)(threadIdx.x >> 5));
    // the warp's slice of shared memory and the areas in it, each as an offset that is computed once
    const uint32_t my_off = (uint32_t)warp * p.smem_per_warp;
    unsigned char* my = smem_raw + once(my_off);
    uint64_t* ring = reinterpret_cast<uint64_t*>(my);
    uint32_t* state = reinterpret_cast<uint32_t*>(smem_raw + once(my_off + (uint32_t)p.Apad * 8u));
    // MC benchmark: vproj[k] = memory usage projected for the last slot of active entry k (same ring as state)
    int* vproj = reinterpret_cast<int*>(smem_raw + once(my_off + (uint32_t)p.Apad * 12u));
    const int state_bytes = (int)p.state_bytes;  // multiple of 16 (host guarantees)
    uint64_t* stage = reinterpret_cast<uint64_t*>(smem_raw + once(my_off + (uint32_t)state_bytes));
    // waiting requests per class (Algorithm 1 only)
    uint32_t* qcnt = reinterpret_cast<uint32_t*>(smem_raw + once(my_off + p.qcnt_off));
    uint64_t* qwin = reinterpret_cast<uint64_t*>(smem_raw + once(my_off + p.qwin_off));  // window on the queue head (64 entries)

    const int Acap = p.Acap, Qcap = p.Qcap, M = p.M, K = p.K, S = p.S;
    const bool kinf = (K == 0);
    const uint32_t FULL = 0xffffffffu;
    const uint32_t gt_mask = lanemask_gt();
    const uint32_t lt_mask = lanemask_lt();
    int bsh = 5;  // lane c watches the entries [c << bsh, (c+1) << bsh) of the active range
    while ((32 << bsh) < Acap) ++bsh;

    for (;;) {
        // ------------------------------------------------------------------ next replica
        unsigned int wi = 0;  // work item: the wi-th replica of this policy
        if (lane == 0) wi = atomicAdd(p.work_counter, 1u);
        wi = uni(wi);  // lane 0 holds it, the others zero
        if (wi >= (unsigned)p.n_work) break;

        int gi = 0;
        {
            int lo = 0, hi = p.n_groups - 1;
            while (lo < hi) {  // last group whose first work item is <= wi
                const int mid = (lo + hi + 1) >> 1;
                if (p.groups[mid].wfirst <= (int)wi) lo = mid; else hi = mid - 1;
            }
            gi = uni(lo);
        }
        DevGroup grp = p.groups[gi];
        grp.b_fp = uni(grp.b_fp); grp.chunk = uni(grp.chunk); grp.arrivals_id = uni(grp.arrivals_id);
        grp.rng_base = uni(grp.rng_base); grp.first = uni(grp.first); grp.admit_limit = uni(grp.admit_limit);
        grp.bclass_off = uni(grp.bclass_off); grp.mc_worst = uni(grp.mc_worst); grp.keep = uni(grp.keep);
        grp.wfirst = uni(grp.wfirst);
        const unsigned int r = (unsigned)grp.first + (wi - (unsigned)grp.wfirst);  // the replica's index
        const DevArrivals* arrp = p.arrivals + grp.arrivals_id;
        const DevTable cnt0 = arrp->count[0];
        const DevTable cnt1 = arrp->count[1];
        const uint32_t thr0 = arrp->thr[0], thr1 = arrp->thr[1];
        const bool two_state = uni(arrp->n_states) == 2u;
        const uint32_t rid = grp.rng_base + (r - (unsigned)grp.first);
        constexpr int policy = kPol;
        const int chunk = grp.chunk;
        const int admit_limit = grp.admit_limit;

        // ------------------------------------------------------------------ load state
        unsigned char* ws = p.workspace + (size_t)r * p.ws_stride;
        uint32_t* hdr = reinterpret_cast<uint32_t*>(ws);
        const uint32_t hw = (lane < kHeaderWords) ? hdr[lane] : 0u;
        auto hword = [&](int j) { return uni(lane == j ? hw : 0u); };
        uint32_t qh = hword(0);                 // sequence number of the queue head (ring place = qh & qmask)
        int shead = (int)hword(1);              // ring position of the oldest active entry
        int nP = (int)hword(2);                 // entries in the active range, completed ones included
        int nQ = (int)hword(3);
        int U = (int)hword(4);                  // usage carried out of the last slot, completions released
        int Ndec = (int)hword(5);               // active requests whose prompt is fully in the cache
        uint32_t next_fin = ~hword(6);          // stored complemented so that zeroed memory means "none"
        int n_pref = (int)hword(7);             // active requests still prefilling
        int pf_lo = (int)hword(8);              // lower bound on the index of the oldest of those
        uint32_t mstate = hword(9);
        uint32_t status = hword(10);
        int nD = (int)hword(11);                // completed entries still inside the active range
        {
            const uint4* src = reinterpret_cast<const uint4*>(ws + kHeaderWords * 4);
            uint4* dst = reinterpret_cast<uint4*>(my);
            for (int i = lane; i < state_bytes / 16; i += 32) dst[i] = src[i];
        }
        // ---- the queue: ring in global memory, its head seen through the shared-memory window
        uint64_t* __restrict__ gq = reinterpret_cast<uint64_t*>(ws + p.gq_off);
        const uint32_t qmask = p.qmask;
        uint32_t wseq = qh;  // the window holds the entries with sequence numbers [wseq, wseq + 64)
        // With kLazy, arrivals that join a long queue are not drawn at once (most are dropped when the waiting room is
        // full, and the lengths of the others are not needed before they reach the head): they wait as placeholders
        // and are drawn, 32 at a time, when the window reaches them.  Algorithm 1 needs the class at arrival.
        constexpr bool kLazyOk = kLazy && kPol != 4;
        bool q_raw = false;  // the window may hold placeholders: draw them before the head is read
        auto q_ready = [&]() {
            if (kLazyOk && q_raw) {
                convert_window(qwin, wseq, qh, nQ, rid, p.key0, p.key1, p.pool, p.gpool, tabs, p.n_classes);
                q_raw = false;
            }
        };
        auto q_get = [&](uint32_t seq) -> uint64_t {  // seq in [qh, qh + nQ)
            return (seq - wseq < 64u) ? qwin[seq & 63u] : gq[seq & qmask];
        };
        auto q_put = [&](uint32_t seq, uint64_t e) {  // global memory is always written, the window when it covers seq
            gq[seq & qmask] = e;
            if (seq - wseq < 64u) qwin[seq & 63u] = e;
        };
        // (re)load the part of the window from sequence number `from` on (all earlier queue writes of this warp
        // must be behind a __syncwarp)
        auto q_fill = [&](uint32_t from) {
#pragma unroll 1
            for (uint32_t sq = from + (uint32_t)lane; sq - wseq < 64u; sq += 32u)
                if (sq - qh < (uint32_t)nQ) qwin[sq & 63u] = gq[sq & qmask];
            q_raw = true;
            __syncwarp();
        };
        // one entry leaves at the head; when half of the window is used up it moves on by 32 entries
        auto q_pop = [&]() {
            ++qh;
            --nQ;
            if (qh - wseq >= 32u) {
                wseq += 32u;
                __syncwarp();
                q_fill(wseq + 32u);
            }
        };
        // an evicted request becomes the head again (lane 0 writes; callers synchronise the warp afterwards)
        auto q_push_front = [&](uint64_t e) {
            --qh;
            ++nQ;
            if ((int)(qh - wseq) < 0) wseq = qh;  // the window slides down by one; its last entry stays in global memory
            if (lane == 0) q_put(qh, e);
        };
        q_fill(wseq);
        long long* cptr = p.counters + (size_t)r * C_COUNT;
        long long cnt = (lane < C_COUNT) ? cptr[lane] : 0;  // lane k owns counter k
        __syncwarp();

// The value is evaluated by every lane BEFORE the lane test: arguments may contain warp-wide primitives.
#define CADD(idx, v) do { const long long v__ = (long long)(v); if (lane == (idx)) cnt += v__; } while (0)
#define CMAX(idx, v) do { const long long v__ = (long long)(v); if (lane == (idx)) cnt = (cnt > v__) ? cnt : v__; } while (0)
#define CSET(idx, v) do { const long long v__ = (long long)(v); if (lane == (idx)) cnt = v__; } while (0)
#define WA(x) ((x) >= Acap ? (x) - Acap : (x))

        // per-launch partial sums of the quantities touched every slot.  The 32-bit ones cannot wrap because the
        // host bounds the slots of a launch by (2^32 - 2^30) / (Qcap + 2 Acap): sumN grows by at most
        // Qcap + 2 Acap per slot, tokgen by at most Acap, arrived and accepted by at most 255.
        unsigned long long sumU = 0;
        uint32_t sumN = 0, tokgen = 0, arrived = 0, accepted = 0;
        int maxU = 0, maxQ = 0;
        int nTot = nP - nD + nQ;  // requests in the system: changes only when requests arrive or complete
        int n_logged = uni(lane == C_N_LOGGED ? (int)cnt : 0);
        uint64_t q_e = 0;  // the queue head's entry when known, else 0 (saves shared-memory reads in blocked slots)
        // Whole-prompt policies: once the headroom gate has refused the queue head, it keeps refusing it until
        // memory is released (a completion or an eviction): the usage only grows and the head does not change.
        // While the flag is up a slot's activation attempt is just counted as refused.
        bool gate_closed = false;
        bool mc_refused = false;  // MC benchmark: the last future-memory test refused the queue head
        // statistics of completions, private to the lane that saw them; reduced once when the replica is put back
        // (acc_o: the output lengths of a launch's completions add up to at most the tokens generated in the
        // launch, <= Acap per slot, plus the tokens the running requests held at its start, <= M <= 2^30)
        unsigned long long acc_lat = 0, acc_w = 0;
        uint32_t acc_o = 0, completed = 0;
        int acc_maxlat = 0;
        // cmin: lane c holds a lower bound of the smallest finishing slot among its stretch of the active
        // range (exact except after an eviction, which a later rescan repairs)
        uint32_t cmin = kNoFin;

        int t = p.t0;
        const int t_end = p.t0 + p.n_steps;

        // trace: lane k keeps the record of slot k of the current batch of draws; the batch's records are stored
        // together when its last slot is done (one coalesced store per warp and batch)
        const int stride = (kRec == 0) ? 0 : p.trace_stride;
        const bool tracing = (kRec == 1) || (kRec == 2 && stride > 0);
        int tr_u = 0, tr_q = 0;
        // staged variant (stride 1): the batch's records go to shared memory (two buffers of 32) and leave with one
        // bulk copy issued by lane 0 when address and size allow it (multiples of 16 bytes)
        int2* tstage = reinterpret_cast<int2*>(my + p.tstage_off);
        const bool staged = kRec == 2 && p.tstage_off != 0 && tracing && stride == 1;  // the host asks for kRec 2 with it
        int tbuf = 0;
        // trow[rec] is record rec of this replica: rec_base <= rec < rec_base + n_rec
        int2* trow = (kRec != 0 && p.trace) ? p.trace + ((long long)r * p.n_rec - p.rec_base) : nullptr;
        int* hrow = p.hist ? p.hist + (size_t)r * p.hist_bins : nullptr;
        int2* lrow = (kRec == 2 && p.complog) ? p.complog + (size_t)r * p.complog_cap : nullptr;

        // Squeeze the completed entries out of the active range: survivors slide towards the newest end
        // (right-to-left pass) and the oldest end of the ring advances.
        auto compact = [&]() {
            int holes = 0;
            for (int base = (nP - 1) & ~31; base >= 0; base -= 32) {
                const int i = base + lane;
                const bool valid = i < nP;
                uint32_t sw = kDead;
                uint64_t e = 0;
                if (valid) sw = STATE(WA(shead + i));
                const bool dead = valid && is_dead(sw);
                const uint32_t m = __ballot_sync(FULL, dead);
                const int sh = holes + __popc(m & gt_mask);  // completed entries after this one
                const bool mv = valid && !dead && sh > 0;
                int v = 0;
                if (mv || dead) e = RING(WA(shead + i));
                if (dead) {
                    // the statistics of the completions, 32 at a time instead of one lane at a time
                    const int l = entry_l(e), o = entry_o(e);
                    const int lat = (int)(sw & ~kDead) - entry_tarr(e) + 1;
                    acc_lat += (unsigned)lat;
                    acc_o += (unsigned)o;
                    acc_maxlat = max(acc_maxlat, lat);
                    acc_w += (unsigned long long)l * o + (unsigned long long)o * (o + 1) / 2;
                    if (hrow) atomicAdd(&HROW(min(lat >> p.hist_shift, p.hist_bins - 1)), 1);
                }
                if (kPol == 5 && mv) v = vproj[WA(shead + i)];
                __syncwarp();
                if (mv) {
                    RING(WA(shead + i + sh)) = e;
                    STATE(WA(shead + i + sh)) = sw;
                    if (kPol == 5) vproj[WA(shead + i + sh)] = v;
                }
                __syncwarp();
                holes += __popc(m);
            }
            shead = WA(shead + nD);
            nP -= nD;
            pf_lo = max(0, pf_lo - nD);
            nD = 0;
        };
        // block minima of the finishing slots, from scratch
        auto rebuild_minima = [&]() {
            cmin = kNoFin;
            for (int base = 0; base < nP; base += 32) {
                const int i = base + lane;
                const uint32_t sw = (i < nP) ? STATE(WA(shead + i)) : kDead;
                const uint32_t m = __reduce_min_sync(FULL, is_dead(sw) ? kNoFin : sw);
                if (lane == (base >> bsh)) cmin = min(cmin, m);
            }
            next_fin = __reduce_min_sync(FULL, cmin);
        };
        rebuild_minima();
        auto squeeze_now = [&]() {
            compact();
            rebuild_minima();
        };
        if ((kExt && policy == 4)) {  // Algorithm 1 picks per class: count the waiting requests of every class
            for (int c = lane; c < p.n_classes; c += 32) qcnt[c] = 0;
            __syncwarp();
            for (int i = lane; i < nQ; i += 32) atomicAdd(&qcnt[entry_cls(q_get(qh + (uint32_t)i))], 1u);
            __syncwarp();
        }

        while (t < t_end) {
            // -------------------------------------------------------------- batch: draws of up to 32 slots
            int L = min(32, t_end - t);
            __syncwarp();  // the staged arrivals of the previous batch have all been read
            uint32_t w0, w1, w2, w3;
            philox4x32_10((uint32_t)(t + 1 + lane), rid, 0u, 0u, p.key0, p.key1, w0, w1, w2, w3);
            const int Bt = (int)(grp.b_fp >> 16) + (((w1 >> 16) < (grp.b_fp & 0xffffu)) ? 1 : 0);
            int n = sample_table(p.pool, p.gpool, cnt0, w0);
            uint32_t smask = 0;  // bit k = arrival state in slot t+1+k
            if (two_state) {
                const int n1 = sample_table(p.pool, p.gpool, cnt1, w0);
                const uint32_t f0 = __ballot_sync(FULL, w2 < thr0);
                const uint32_t f1 = __ballot_sync(FULL, w2 < thr1);
                if (f0 == f1) {  // same flips from either state: parity of the flips so far
                    const uint32_t upto = f0 & (lt_mask | (1u << lane));
                    const uint32_t mine = (mstate ^ (uint32_t)__popc(upto)) & 1u;
                    smask = __ballot_sync(FULL, mine != 0u);
                } else {
                    uint32_t cur = mstate;
                    for (int k = 0; k < 32; ++k) {
                        cur ^= ((cur ? f1 : f0) >> k) & 1u;
                        smask |= cur << k;
                    }
                }
                if ((smask >> lane) & 1u) n = n1;
            }
            if (lane >= L) n = 0;
            int incl = warp_incl_scan(n, lane);
            // arrivals that join a long queue are not generated now (see below): nothing is staged
            const bool lazy = kLazyOk && nQ >= 96;
            if (!lazy) L = min(L, __popc(__ballot_sync(FULL, incl <= S)));  // staged arrivals must fit; n <= S so L >= 1
            if (lane >= L) n = 0;
            const int excl = incl - n;
            const int N = uni(lane == L - 1 ? incl : 0);
            // generate the N arrivals of these slots, one per lane (stream 1, index = rank within the slot), unless
            // they join a long queue: then those that are accepted are drawn when the window reaches them
#pragma unroll 1
            for (int base = 0; base < (lazy ? 0 : N); base += 32) {
                const int idx = base + lane;
                int lo = 0, hi = L - 1;
#pragma unroll
                for (int it = 0; it < 5; ++it) {  // slot k = first with incl_k > idx
                    const int mid = (lo + hi) >> 1;
                    const int v = __shfl_sync(FULL, incl, mid);
                    if (lo < hi) { if (v > idx) hi = mid; else lo = mid + 1; }
                }
                const int ex_k = __shfl_sync(FULL, excl, lo);
                if (idx < N) {
                    uint32_t a0, a1, a2, a3;
                    philox4x32_10((uint32_t)(t + 1 + lo), rid, 1u, (uint32_t)(idx - ex_k), p.key0, p.key1, a0, a1,
                                  a2, a3);
                    const int cls = sample_table(p.pool, p.gpool, tabs[0], a0);
                    int l, o;
                    sample_pair(p.pool, p.gpool, tabs[1 + cls], a1, tabs[1 + p.n_classes + cls], a2, l, o);
                    STAGE(idx) = pack_entry(l, o, t + 1 + lo, cls);
                }
            }
            __syncwarp();
            // A slot asks for its count only when it has arrivals AND the waiting room has a place: bit k of
            // nzmask says whether slot k has arrivals, lane k holds the count and where its arrivals are staged.
            // Arrivals that find the room full are dropped without being looked at; their number is the
            // difference between the batch's total and the accepted ones.
            const uint32_t nzmask = __ballot_sync(FULL, n > 0);
            const uint32_t btmask = __ballot_sync(FULL, Bt > (int)(grp.b_fp >> 16));  // slots whose B_t is rounded up
            const uint32_t packed = (uint32_t)n | ((uint32_t)excl << 8);
            arrived += N;

            // -------------------------------------------------------------- the slots of the batch
            for (int k = 0; k < L; ++k) {
                ++t;
                const int B_t = (int)(grp.b_fp >> 16) + (int)((btmask >> k) & 1u);

                // ---- arrivals join the queue tail; a full waiting room drops the rest
                if (((nzmask >> k) & 1u) && nQ < Qcap) {
                    const uint32_t info = uni(lane == k ? packed : 0u);
                    const int sp = (int)(info >> 8);  // where the slot's arrivals are staged
                    const int acc = min((int)(info & 0xffu), Qcap - nQ);
                    const uint32_t tail = qh + (uint32_t)nQ;
                    if (lazy) {
#pragma unroll 1
                        for (int i = lane; i < acc; i += 32) q_put(tail + (uint32_t)i, pack_entry(0, i, t, 0));
                        if (tail - wseq < 64u) q_raw = true;  // the queue has shrunk into the window meanwhile
                    } else {
#pragma unroll 1
                        for (int i = lane; i < acc; i += 32) {
                            const uint64_t e = STAGE(sp + i);
                            q_put(tail + (uint32_t)i, e);
                            if ((kExt && policy == 4)) atomicAdd(&qcnt[entry_cls(e)], 1u);
                        }
                    }
                    nQ += acc;
                    nTot += acc;
                    accepted += acc;
                    __syncwarp();
                }

                // ---- usage the slot would reach, token room
                int G = U + Ndec;
                int R = (policy == 2) ? max(0, K - Ndec) : K;

                // ---- chunked policy: continuing prefills first, in activation order
                if (policy == 2 && n_pref > 0) {
                    int first_left = -1;
#pragma unroll 1
                    for (int base = pf_lo & ~31; base < nP; base += 32) {
                        const int i = base + lane;
                        uint32_t sw = 0;
                        uint64_t e = 0;
                        if (i < nP) sw = STATE(WA(shead + i));
                        const bool pf = (sw & kPrefillBit) != 0;
                        if (pf) e = RING(WA(shead + i));
                        const int pcur = (int)(sw & ~kPrefillBit);
                        const int l = entry_l(e);
                        const int d = pf ? min(chunk, l - pcur) : 0;
                        const int dincl = warp_incl_scan(d, lane);
                        int g = d;
                        if (!kinf) g = min(d, max(0, R - (dincl - d)));
                        const bool fin = pf && (pcur + g == l);
                        if (pf && g > 0) {
                            STATE(WA(shead + i)) = fin ? (uint32_t)(t + entry_o(e) - 1) : (kPrefillBit | (uint32_t)(pcur + g));
                        }
                        const int gsum = __reduce_add_sync(FULL, g);
                        const uint32_t finm = __ballot_sync(FULL, fin);
                        const uint32_t leftm = __ballot_sync(FULL, pf && !fin);
                        const int nfin = __popc(finm);
                        if (!kinf) R -= gsum;
                        G += gsum + nfin;
                        CADD(C_PREFILL_TOKENS, gsum);
                        Ndec += nfin;
                        n_pref -= nfin;
                        if (finm) {
                            const uint32_t mine = fin ? (uint32_t)(t + entry_o(e) - 1) : kNoFin;
                            const uint32_t bm = __reduce_min_sync(FULL, mine);
                            if (lane == (base >> bsh)) cmin = min(cmin, bm);
                            next_fin = min(next_fin, bm);
                        }
                        if (first_left < 0 && leftm) first_left = base + (__ffs(leftm) - 1);
                        if (!kinf && R == 0 && first_left >= 0) break;  // nothing more can move this slot
                    }
                    if (first_left >= 0) pf_lo = first_left;
                    __syncwarp();
                }

                // ---- activation (Alg. 2 inner loop): FIFO, at most B_t under flow control
                int a = 0;
                const int cap = (policy == 0) ? B_t : 0x7fffffff;
                if (gate_closed) {
                    if (cap > 0) CADD(C_GATE_BLOCKED, 1);
                } else {
                    do {
                    if constexpr (policy == 4) {
                        // Algorithm 1: for every class k, up to b_k waiting requests of that class, oldest first.
                        // The pick leaves the middle of the queue: the entries ahead of it move one place
                        // towards the tail and the pick takes the freed place next to the active range.
                        bool gate_hit = false, budget_hit = false, storage_hit = false;
                        const int32_t* bk = p.bclass + grp.bclass_off;
                        if (nD > 0 && nP + nQ > Acap) {  // the picks below take the storage bound at face value
                            __syncwarp();
                            squeeze_now();
                        }
                        if (nQ > 0 && nQ <= 32 && p.n_classes <= 8) {
                            // Short queue: all picks of the slot at once (lane = waiting request).  A request is
                            // picked when fewer than b_k requests of its class wait ahead of it; the picks are
                            // activated class by class, in queue order within a class.  Taken only when every pick
                            // passes the gate, the token budget and the storage bound (the usage is largest with all
                            // of them in, so one test covers every prefix); otherwise the loop below decides pick by pick.
                            const bool in = lane < nQ;
                            const uint64_t e = qwin[(qh + (uint32_t)lane) & 63u];
                            const int cls = in ? entry_cls(e) : -1;
                            int rank = 0, before = 0, npick = 0, mytake = 0;
                            bool picked = false;
                            for (int kc = 0; kc < p.n_classes; ++kc) {
                                const uint32_t mk = __ballot_sync(FULL, cls == kc);
                                const int take = min(__popc(mk), __ldg(bk + kc));
                                if (cls == kc) {
                                    rank = __popc(mk & lt_mask);
                                    picked = rank < take;
                                    before = npick;
                                }
                                if (lane == kc) mytake = take;
                                npick += take;
                            }
                            const int l = entry_l(e);
                            const int tot_l = __reduce_add_sync(FULL, picked ? l : 0);
                            if (npick > 0 && nP + npick <= Acap && G + tot_l + npick <= M &&
                                (kinf || npick == 1 || tot_l <= R)) {
                                const int dest = nP + before + rank;  // place in the active range
                                const uint32_t sw = picked ? (uint32_t)(t + entry_o(e) - 1) : kNoFin;
                                const uint32_t pm = __ballot_sync(FULL, picked);
                                // the requests left behind keep their order and close ranks towards the tail
                                const uint32_t stay_seq = qh + (uint32_t)(npick + lane - __popc(pm & lt_mask));
                                __syncwarp();  // every lane holds its entry: the window may be overwritten
                                if (picked) {
                                    RING(WA(shead + dest)) = e;
                                    STATE(WA(shead + dest)) = sw;
                                } else if (in) {
                                    q_put(stay_seq, e);
                                }
                                if (lane < p.n_classes) qcnt[lane] -= (uint32_t)mytake;
                                const int c0 = nP >> bsh;
                                const bool lo_part = (dest >> bsh) == c0;
                                const uint32_t m0 = __reduce_min_sync(FULL, lo_part ? sw : kNoFin);
                                const uint32_t m1 = __reduce_min_sync(FULL, lo_part ? kNoFin : sw);
                                if (lane == c0) cmin = min(cmin, m0);
                                if (lane == c0 + 1) cmin = min(cmin, m1);
                                next_fin = min(next_fin, min(m0, m1));
                                G += tot_l + npick;
                                if (!kinf) R = max(0, R - tot_l);
                                Ndec += npick;
                                nP += npick;
                                a = npick;
                                CADD(C_PREFILL_TOKENS, tot_l);
                                qh += (uint32_t)npick;
                                nQ -= npick;
                                __syncwarp();
                                if (qh - wseq >= 32u) {  // the window moves on as in q_pop
                                    wseq += 32u;
                                    q_fill(wseq + 32u);
                                }
                                q_e = 0;
                                break;
                            }
                        }
                        for (int kc = 0; kc < p.n_classes && !storage_hit; ++kc) {
                            const int b_k = __ldg(bk + kc);
                            for (int ak = 0; ak < b_k && qcnt[kc] > 0; ++ak) {
                                if (nP == Acap) { storage_hit = true; break; }  // completed entries were squeezed out above
                                const uint32_t q0 = qh;
                                int pos = -1;
                                uint64_t e = 0;
                                for (int base = 0; base < nQ && pos < 0; base += 32) {
                                    const int i = base + lane;
                                    const uint64_t c = (i < nQ) ? q_get(q0 + (uint32_t)i) : 0;
                                    const uint32_t m = __ballot_sync(FULL, i < nQ && entry_cls(c) == kc);
                                    if (m) {
                                        const int src = __ffs(m) - 1;
                                        pos = base + src;
                                        e = __shfl_sync(FULL, c, src);
                                    }
                                }
                                if (pos < 0) break;  // cannot happen while the counts are right
                                const int l = entry_l(e);
                                if (!(kinf || a == 0 || l <= R)) { budget_hit = true; break; }
                                if (G + l + 1 > M) { gate_hit = true; break; }
                                for (int base = (pos - 1) & ~31; pos > 0 && base >= 0; base -= 32) {
                                    const int i = base + lane;
                                    const bool mv = i < pos;
                                    uint64_t c = 0;
                                    if (mv) c = q_get(q0 + (uint32_t)i);
                                    __syncwarp();
                                    if (mv) q_put(q0 + (uint32_t)i + 1u, c);
                                    __syncwarp();
                                }
                                const uint32_t sw = (uint32_t)(t + entry_o(e) - 1);
                                if (lane == 0) {
                                    RING(WA(shead + nP)) = e;
                                    STATE(WA(shead + nP)) = sw;
                                    qcnt[kc] -= 1;
                                }
                                next_fin = min(next_fin, sw);
                                if (lane == (nP >> bsh)) cmin = min(cmin, sw);
                                Ndec++;
                                nP++;
                                q_pop();  // the entries ahead of the pick moved up: the freed place is the head's
                                G += l + 1;
                                if (!kinf) R -= min(l, R);
                                a++;
                                CADD(C_PREFILL_TOKENS, l);
                                __syncwarp();
                            }
                        }
                        if (gate_hit) CADD(C_GATE_BLOCKED, 1);
                        if (budget_hit) CADD(C_BUDGET_BLOCKED, 1);
                        if (storage_hit) { CADD(C_ACAP_BLOCKED, 1); status |= 1u; }
                        q_e = 0;
                        break;
                    } else {
                    if constexpr (kBulk && (policy <= 1 || policy == 3 || policy == 6)) {
                        // Several queue heads at once (lane = candidate): the heads that the sequential rule would
                        // admit one after the other are the leading run of candidates whose cumulative need still
                        // passes the gate and whose cumulative prompt tokens still fit the slot's token room (the
                        // slot's first admission is exempt).  The candidate that ends the run is left to the
                        // sequential loop below, which counts the reason.
                        int want = min(min(cap - a, nQ), Acap - nP);
                        if (want >= 2) {
                            want = min(want, 32);
                            q_ready();
                            const bool in = lane < want;
                            const uint64_t e = qwin[(qh + (uint32_t)lane) & 63u];  // the first 32 queue places are in the window
                            const int l = entry_l(e);
                            const int pre = warp_incl_scan(in ? l + 1 : 0, lane);  // tokens the slot's usage grows by
                            const int pre_l = pre - (lane + 1);                    // prompt tokens of candidates 0 .. lane
                            const bool ok = in && G + pre <= admit_limit && (kinf || (a == 0 && lane == 0) || pre_l <= R);
                            const uint32_t okm = __ballot_sync(FULL, ok);
                            int n = (okm == FULL) ? 32 : __ffs((int)~okm) - 1;
                            if constexpr (kMcProfile) {
                                // MC benchmark: the candidates of the run pass the future-memory test one after the
                                // other (each is booked on the projection before the next is tested); the first
                                // refusal ends the run
                                int pass = 0;
#pragma unroll 1
                                for (; pass < n; ++pass) {
                                    const uint64_t ec = __shfl_sync(FULL, e, pass);
                                    const int op_c = grp.mc_worst != 0 ? (tabs[1 + p.n_classes + entry_cls(ec)].vmin +
                                                                          (int)tabs[1 + p.n_classes + entry_cls(ec)].n - 1)
                                                                       : entry_o(ec);
                                    const int a_c = entry_l(ec) - t + 1;
                                    bool over = false;
#pragma unroll 1
                                    for (int base = 0; base < op_c; base += 32) {
                                        const int tau = t + base + lane;
                                        over |= (base + lane < op_c) && (vproj[(uint32_t)tau & p.prof_mask] + a_c + tau > M);
                                    }
                                    if (__any_sync(FULL, over)) break;
#pragma unroll 1
                                    for (int base = 0; base < op_c; base += 32) {
                                        const int tau = t + base + lane;
                                        if (base + lane < op_c) vproj[(uint32_t)tau & p.prof_mask] += a_c + tau;
                                    }
                                }
                                n = pass;
                            }
                            if (n > 0) {
                                const uint32_t sw = (lane < n) ? (uint32_t)(t + entry_o(e) - 1) : kNoFin;
                                if (lane < n) {
                                    RING(WA(shead + nP + lane)) = e;
                                    STATE(WA(shead + nP + lane)) = sw;
                                }
                                // the new entries lie in at most two watched stretches of the active range
                                const int c0 = nP >> bsh;
                                const bool lo_part = ((nP + lane) >> bsh) == c0;
                                const uint32_t m0 = __reduce_min_sync(FULL, lo_part ? sw : kNoFin);
                                const uint32_t m1 = __reduce_min_sync(FULL, lo_part ? kNoFin : sw);
                                if (lane == c0) cmin = min(cmin, m0);
                                if (lane == c0 + 1) cmin = min(cmin, m1);
                                next_fin = min(next_fin, min(m0, m1));
                                const int tot = uni(lane == n - 1 ? pre : 0);
                                G += tot;
                                if (!kinf) R = max(0, R - (tot - n));
                                Ndec += n;
                                nP += n;
                                a += n;
                                CADD(C_PREFILL_TOKENS, tot - n);
                                qh += (uint32_t)n;
                                nQ -= n;
                                q_e = 0;
                                __syncwarp();
                                if (qh - wseq >= 32u) {  // the window moves on as in q_pop
                                    wseq += 32u;
                                    q_fill(wseq + 32u);
                                }
                            }
                        }
                    }
#pragma unroll 1
                    while (a < cap && nQ > 0) {
                        if (nP == Acap) {
                            if (nD > 0) {  // storage, not the model's bound: make room
                                __syncwarp();  // state words written by lane 0 during this slot's activations
                                squeeze_now();
                                continue;
                            }
                            CADD(C_ACAP_BLOCKED, 1); status |= 1u; break;
                        }
                        if (q_e == 0) {
                            q_ready();
                            q_e = uni(qwin[qh & 63u]);  // the head is always inside the window
                        }
                        const int l = entry_l(q_e);
                        int g, need;
                        if (policy == 2) {
                            g = kinf ? min(chunk, l) : min(min(chunk, l), R);
                            if (g == 0) { CADD(C_BUDGET_BLOCKED, 1); break; }
                            need = g + (g == l ? 1 : 0);
                        } else {
                            g = l;
                            if (!(kinf || a == 0 || g <= R)) { CADD(C_BUDGET_BLOCKED, 1); break; }
                            need = l + 1;
                        }
                        if (G + need > admit_limit) {
                            CADD(C_GATE_BLOCKED, 1);
                            gate_closed = (a == 0) && (policy <= 1 || policy == 3);
                            break;
                        }
                        if (kMcProfile) {
                            // MC benchmark (Section 4.1): start the queue head only if the usage of every future
                            // slot stays within M.  uprof[tau & mask] is the usage of slot tau >= t if nothing else
                            // starts; the head would hold l + (tau - t + 1) = a_h + tau in the slots t .. f_h.
                            // Lane = future slot: one read-only pass tests, a second one books the head.
                            const uint64_t eh = q_e;
                            const int op_h = grp.mc_worst != 0 ? (tabs[1 + p.n_classes + entry_cls(eh)].vmin +
                                                                  (int)tabs[1 + p.n_classes + entry_cls(eh)].n - 1)
                                                               : entry_o(eh);
                            const int a_h = l - t + 1;
                            bool over = false;
#pragma unroll 1
                            for (int base = 0; base < op_h; base += 32) {
                                const int tau = t + base + lane;
                                over |= (base + lane < op_h) && (vproj[(uint32_t)tau & p.prof_mask] + a_h + tau > M);
                            }
                            if (__any_sync(FULL, over)) { CADD(C_GATE_BLOCKED, 1); break; }
#pragma unroll 1
                            for (int base = 0; base < op_h; base += 32) {
                                const int tau = t + base + lane;
                                if (base + lane < op_h) vproj[(uint32_t)tau & p.prof_mask] += a_h + tau;
                            }
                        }
                        if (kPol == 5) {
                            // MC benchmark (Section 4.1): start the queue head only if the usage of every future
                            // slot stays within M.  With a_i = l_i - (activation slot) + 1, request i holds a_i + tau
                            // in slot tau up to its last slot f_i; the usage can only peak in some last slot.
                            // vproj[k] holds the usage of slot f_k for the running requests, so the head h
                            // (last slot f_h) fits iff vproj[k] + a_h + f_k <= M for every k with f_k <= f_h and
                            // the usage of slot f_h itself, sum over f_i >= f_h of (a_i + f_h) + a_h + f_h, is <= M.
                            const uint64_t eh = q_e;
                            const bool worst = grp.mc_worst != 0;
                            const int op_h = worst ? (tabs[1 + p.n_classes + entry_cls(eh)].vmin +
                                                      (int)tabs[1 + p.n_classes + entry_cls(eh)].n - 1)
                                                   : entry_o(eh);
                            const int f_h = t + op_h - 1, a_h = l - t + 1;
                            // One pass tests the head and, tentatively, already books it on every earlier last
                            // slot; a refusal takes the booking back in a second pass.  Right after a refusal
                            // the next test is expected to fail too and runs read-only, booking only if it passes.
                            const bool tentative = !mc_refused;
                            bool ok = true;
                            long long S = 0;
#pragma unroll 4
                            for (int base = 0; base < nP; base += 32) {
                                // loads first and unconditionally (lanes past the range read entry 0 and ignore
                                // it), so that the iterations' shared-memory round trips overlap
                                const int i = base + lane;
                                const bool in = i < nP;
                                const int si = WA(shead + (in ? i : 0));
                                const uint32_t swi = STATE(si);
                                const uint64_t ei = RING(WA(shead + (in ? i : 0)));
                                const uint32_t vi = (uint32_t)vproj[si];
                                const bool live = in && !is_dead(swi);
                                uint32_t f_i = swi;
                                if (worst) {
                                    const DevTable d = tabs[1 + p.n_classes + (live ? entry_cls(ei) : 0)];
                                    f_i += (uint32_t)(d.vmin + (int)d.n - 1 - entry_o(ei));
                                }
                                // unsigned arithmetic: ignored lanes may hold anything; for live entries
                                // v <= M + 2 * 65536 < 2^31
                                const int v = (int)(vi + (uint32_t)a_h + f_i);
                                if (live && (int)f_i <= f_h) {
                                    if (v > M) ok = false;
                                    if (tentative) vproj[si] = v;
                                }
                                if (live && (int)f_i >= f_h) S += (int)((uint32_t)(entry_l(ei) + entry_o(ei)) - swi + (uint32_t)f_h);
                            }
                            S = warp_sum64(S) + a_h + f_h;
                            const bool fits = !__any_sync(FULL, !ok) && S <= M;
                            if (fits != tentative) {  // take the booking back, or make the one the read-only test skipped
#pragma unroll 2
                                for (int base = 0; base < nP; base += 32) {
                                    const int i = base + lane;
                                    const uint32_t swi = (i < nP) ? STATE(WA(shead + i)) : kDead;
                                    if (!is_dead(swi)) {
                                        int f_i = (int)swi;
                                        if (worst) {
                                            const uint64_t ei = RING(WA(shead + i));
                                            f_i += tabs[1 + p.n_classes + entry_cls(ei)].vmin +
                                                   (int)tabs[1 + p.n_classes + entry_cls(ei)].n - 1 - entry_o(ei);
                                        }
                                        if (f_i <= f_h) vproj[WA(shead + i)] += fits ? (a_h + f_i) : -(a_h + f_i);
                                    }
                                }
                            }
                            mc_refused = !fits;
                            if (!fits) { CADD(C_GATE_BLOCKED, 1); break; }
                            if (lane == 0) vproj[WA(shead + nP)] = (int)S;
                        }
                        uint32_t sw;
                        if (g == l) {
                            sw = (uint32_t)(t + entry_o(q_e) - 1);
                            next_fin = min(next_fin, sw);
                            if (lane == (nP >> bsh)) cmin = min(cmin, sw);
                            Ndec++;
                        } else {
                            sw = kPrefillBit | (uint32_t)g;
                            if (n_pref == 0) pf_lo = nP;
                            n_pref++;
                        }
                        if (lane == 0) {
                            RING(WA(shead + nP)) = q_e;
                            STATE(WA(shead + nP)) = sw;
                        }
                        __syncwarp();  // the next pick may scan the active range (MC projection) or squeeze it
                        nP++;
                        q_pop();
                        q_e = 0;
                        G += need;
                        if (!kinf) R -= min(g, R);
                        a++;
                        CADD(C_PREFILL_TOKENS, g);
                    }
                    }
                    } while (false);
                    if (a > 0) { CADD(C_ADMITTED, a); __syncwarp(); }
                }

                // ---- overflow: evict the most recently activated until the slot fits (LIFO, Section 3.3);
                //      evicted requests lose all progress (or, in the variant that keeps the generated tokens,
                //      only their place in the cache) and are again the head of the queue
                if (G > M) {
                    maxU = max(maxU, U);  // the last slot's usage, before this slot's evictions lower it
                    gate_closed = false;
                    CADD(C_OVERFLOW_STEPS, 1);
                    int nev = 0, wasted = 0;
                    if (policy == 3) {
                        // alpha-protection greedy (Section 4.1): every active request goes back to the queue.
                        // Completed entries are squeezed out first, so the whole active range is live and is
                        // copied, in order, in front of the queue head.
                        if (nD > 0) {
                            __syncwarp();
                            compact();
                        }
                        long long kept_w = 0;
                        const uint32_t nqh = qh - (uint32_t)nP;
                        wseq = nqh;  // the window restarts at the new head (reloaded below)
                        for (int base = 0; base < nP; base += 32) {
                            const int i = base + lane;
                            if (i < nP) {
                                const uint32_t sw = STATE(WA(shead + i));
                                uint64_t e = RING(WA(shead + i));
                                if (!(sw & kPrefillBit)) {
                                    const int j = t - (int)sw + entry_o(e) - 1;
                                    wasted += j;
                                    if (grp.keep != 0 && j > 0) {
                                        const int l = entry_l(e);
                                        kept_w += (long long)l * j + (long long)j * (j + 1) / 2;
                                        e = pack_entry(l + j, entry_o(e) - j, entry_tarr(e), entry_cls(e));
                                    }
                                }
                                gq[(nqh + (uint32_t)i) & qmask] = e;
                            }
                        }
                        wasted = __reduce_add_sync(FULL, wasted);
                        if (grp.keep != 0) {  // kept tokens are final: delivered now, with the workload they took
                            CADD(C_COMPLETED_TOKENS, wasted);
                            CADD(C_SUM_W_COMPLETED, warp_sum64(kept_w));
                            wasted = 0;
                        }
                        nev = nP;
                        qh = nqh;
                        nQ += nP;
                        nP = 0;
                        __syncwarp();
                        q_fill(wseq);
                        Ndec = 0;
                        n_pref = 0;
                        G = 0;
                        q_e = 0;
                        cmin = kNoFin;
                        next_fin = kNoFin;
                    }
#pragma unroll 1
                    while (policy != 3 && G > M && nP > nD) {
                        int i = nP - 1;
                        uint32_t sw = uni(STATE(WA(shead + i)));
                        if (is_dead(sw)) {
                            // completed entries lie on top of the newest live one: find it (backwards, 32 at a
                            // time), and let it change places with the completed entry at the top (whose record
                            // is still needed for its statistics); it is evicted from the top place below
                            const uint32_t sw_top = sw;
                            int found = -1;
#pragma unroll 1
                            for (int top = nP; found < 0 && top > 0; top -= 32) {
                                const int idx = top - 32 + lane;
                                const uint32_t w = (idx >= 0) ? STATE(WA(shead + idx)) : kDead;
                                const uint32_t m = __ballot_sync(FULL, !is_dead(w));
                                if (m) found = top - 1 - __clz(m);
                            }
                            i = found;
                            sw = uni(STATE(WA(shead + i)));
                            const uint64_t moved = RING(WA(shead + i));
                            const uint64_t top_e = RING(WA(shead + nP - 1));
                            __syncwarp();
                            if (lane == 0) {
                                RING(WA(shead + nP - 1)) = moved;
                                RING(WA(shead + i)) = top_e;
                                STATE(WA(shead + i)) = sw_top;
                            }
                            __syncwarp();
                        }
                        uint64_t e = uni(RING(WA(shead + nP - 1)));
                        if (sw & kPrefillBit) {
                            G -= (int)(sw & ~kPrefillBit);
                            n_pref--;
                        } else {
                            const int j = t - (int)sw + entry_o(e) - 1;  // tokens generated before this slot
                            const int l = entry_l(e);
                            G -= l + j + 1;
                            Ndec--;
                            if (grp.keep == 0) {
                                wasted += j;
                            } else if (j > 0) {
                                // the generated tokens stay with the request as prompt; they are final, so they
                                // are delivered now, with the workload they took: sum_{i<=j} (l + i)
                                CADD(C_COMPLETED_TOKENS, j);
                                CADD(C_SUM_W_COMPLETED, (long long)l * j + (long long)j * (j + 1) / 2);
                                e = pack_entry(l + j, entry_o(e) - j, entry_tarr(e), entry_cls(e));
                            }
                        }
                        q_push_front(e);
                        q_e = e;
                        if ((kExt && policy == 4) && lane == 0) qcnt[entry_cls(e)] += 1;
                        nP--;
                        nev++;
                    }
                    if (pf_lo > nP) pf_lo = nP;
                    CADD(C_EVICTIONS, nev);
                    CADD(C_WASTED_TOKENS, wasted);
                    __syncwarp();
                }

                // ---- process: one token per request whose prompt is in the cache; U_t = G
                tokgen += Ndec;
                U = G;
                sumU += (unsigned)G;
                sumN += nTot;

                // ---- retire the requests that generated their last token in this slot: their statistics
                //      are taken now, their entries are only marked and squeezed out later in bulk
                if ((uint32_t)t == next_fin) {
                    int ndone = 0, sum_lo = 0;
                    int pend_f = 0, pend_a = 0, npend = 0;  // lane q < npend: projected last slot and offset of an early finisher
                    auto mc_release = [&]() {
                        __syncwarp();  // the finishers' state words are marked
#pragma unroll 2
                        for (int vb = 0; vb < nP; vb += 32) {
                            const int vi = vb + lane;
                            const bool in = vi < nP;
                            const int si = WA(shead + (in ? vi : 0));
                            const uint32_t swv = STATE(si);
                            const uint64_t ev = RING(WA(shead + (in ? vi : 0)));
                            const bool live = in && !is_dead(swv);
                            const DevTable dv = tabs[1 + p.n_classes + (live ? entry_cls(ev) : 0)];
                            // a completed entry takes no correction: later than any slot
                            const int f_v = live ? (int)swv + dv.vmin + (int)dv.n - 1 - entry_o(ev) : 0x3fffffff;
                            int delta = 0;
                            for (int q = 0; q < npend; ++q) {
                                const int f_c = __shfl_sync(FULL, pend_f, q), a_c = __shfl_sync(FULL, pend_a, q);
                                if (f_v <= f_c) delta += a_c + f_v;
                            }
                            if (delta != 0) vproj[si] -= delta;
                        }
                        npend = 0;
                    };
                    uint32_t due = __ballot_sync(FULL, cmin == (uint32_t)t);
#pragma unroll 1
                    while (due) {
                        const int c = __ffs(due) - 1;
                        due &= due - 1;
                        uint32_t gmin = kNoFin;  // new minimum of lane c's stretch
                        const int stop = min(nP, (c + 1) << bsh);
#pragma unroll 1
                        for (int base = c << bsh; base < stop; base += 32) {
                            const int i = base + lane;
                            const uint32_t sw = (i < nP) ? STATE(WA(shead + i)) : kDead;
                            const bool done = (sw == (uint32_t)t);
                            const uint32_t m = __ballot_sync(FULL, done);
                            uint64_t e = 0;
                            if (m) {
                                if (done) {
                                    e = RING(WA(shead + i));
                                    sum_lo += entry_l(e) + entry_o(e);
                                    if (lrow) {
                                        const int li = n_logged + ndone + __popc(m & lt_mask);  // activation order
                                        if (li < p.complog_cap) LROW(li) = make_int2(t, t - entry_tarr(e) + 1);
                                    }
                                    // latency, workload and histogram of the completion are taken when the entry
                                    // is squeezed out, many entries at a time
                                    STATE(WA(shead + i)) = kDead | (uint32_t)t;
                                }
                                ndone += __popc(m);
                                if (kMcProfile && grp.mc_worst != 0) {
                                    // worst-case projection: a request that ends before its projected last slot
                                    // f_c = t + (longest output of its class - o) leaves the projected usage of the
                                    // slots t+1 .. f_c, where it was booked with a_c + tau, a_c = l + o - t
                                    uint32_t mm = m;
#pragma unroll 1
                                    while (mm) {
                                        const int src = __ffs(mm) - 1;
                                        mm &= mm - 1;
                                        const uint64_t ec = __shfl_sync(FULL, e, src);
                                        const DevTable dc = tabs[1 + p.n_classes + entry_cls(ec)];
                                        const int extra = dc.vmin + (int)dc.n - 1 - entry_o(ec);  // slots it leaves early
                                        const int a_c = entry_l(ec) + entry_o(ec) - t;
#pragma unroll 1
                                        for (int base = 0; base < extra; base += 32) {
                                            const int tau = t + 1 + base + lane;
                                            if (base + lane < extra) vproj[(uint32_t)tau & p.prof_mask] -= a_c + tau;
                                        }
                                    }
                                }
                                if (kPol == 5 && grp.mc_worst != 0) {
                                    // MC benchmark with worst-case projection: a request that ends before its
                                    // projected last slot f_c leaves the projected usage of every last slot <= f_c.
                                    // The slot's early finishers are collected, one per lane, and taken out of the
                                    // projections in one pass over the active range.
                                    const int cntm = __popc(m);
                                    if (npend + cntm > 32) mc_release();
                                    const int rnk = lane - npend;
                                    const bool take = rnk >= 0 && rnk < cntm;
                                    const int src = take ? (int)__fns(m, 0, rnk + 1) : 0;
                                    const uint64_t ec = __shfl_sync(FULL, e, src);
                                    if (take) {
                                        const DevTable dc = tabs[1 + p.n_classes + entry_cls(ec)];
                                        pend_f = t - entry_o(ec) + dc.vmin + (int)dc.n - 1;
                                        pend_a = entry_l(ec) + entry_o(ec) - t;
                                    }
                                    npend += cntm;
                                }
                            }
                            gmin = min(gmin, __reduce_min_sync(FULL, (done || is_dead(sw)) ? kNoFin : sw));
                        }
                        if (lane == c) cmin = gmin;
                    }
                    if (kPol == 5 && npend > 0) mc_release();
                    next_fin = __reduce_min_sync(FULL, cmin);
                    if (ndone > 0) {
                        // the usage only falls when requests leave or are evicted: its maximum is taken there
                        maxU = max(maxU, G);
                        gate_closed = false;
                        nD += ndone;
                        nTot -= ndone;
                        Ndec -= ndone;
                        completed += ndone;
                        U -= __reduce_add_sync(FULL, sum_lo);
                        if (lrow) {
                            if (n_logged + ndone > p.complog_cap) status |= 2u;
                            n_logged = min(p.complog_cap, n_logged + ndone);
                        }
                        __syncwarp();
                        // completed entries are squeezed out when enough have piled up (and whenever the storage
                        // of the active range runs out, or the whole range is sent back)
                        if (nD >= kCompactAt) squeeze_now();
                    }
                }

                if (kMcProfile) {  // slot t has passed: its place in the ring is slot t + H's, which nothing reaches yet
                    __syncwarp();
                    if (lane == 0) vproj[(uint32_t)t & p.prof_mask] = 0;
                }

                // ---- record
                maxQ = max(maxQ, nQ);
                if (kRec != 0 && lane == k) { tr_u = G; tr_q = nQ; }
            }  // slots of the batch
            if constexpr (kRec != 0) if (tracing) {  // the batch was the slots t - L + 1 .. t; lane k holds slot t - L + 1 + k
                const int ts = t - L + 1 + lane;
                if (staged) {
                    int2* sb = tstage + 32 * tbuf;
                    if (lane < L) sb[lane] = make_int2(tr_u, tr_q);
                    __syncwarp();
                    int2* dst = trow + (t - L);  // stride 1: the record of slot s has index s - 1
                    if ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0 && (L & 1) == 0) {
                        if (lane == 0) {
                            bulk_store_commit(dst, sb, (uint32_t)L * 8u);
                            bulk_wait_read<1>();  // the other buffer (copy issued a batch ago) is free again
                        }
                    } else {
                        if (lane < L) TROW(ts - 1) = make_int2(tr_u, tr_q);
                        if (lane == 0) bulk_wait_read<0>();  // no new copy: the other buffer's must have been read
                    }
                    tbuf ^= 1;
                    __syncwarp();
                } else if (lane < L && (stride == 1 || ts % stride == 0)) {
                    TROW(stride == 1 ? ts - 1 : ts / stride - 1) = make_int2(tr_u, tr_q);
                }
            }
            if (two_state) mstate = (smask >> (L - 1)) & 1u;
        }  // while t < t_end

        // ------------------------------------------------------------------ flush, final extras, spill
        if (staged) {  // the staging buffers are reused by the next replica and the copies must land before the exit
            if (lane == 0) bulk_wait_all();
            __syncwarp();
        }
        if (nD > 0) {  // the completions still inside the active range are accounted for before the replica is put back
            __syncwarp();
            compact();
        }
        long long age = 0, resj = 0;
        __syncwarp();  // the queue entries written during the last slots are read by other lanes below
        for (int i = lane; i < nP; i += 32) {
            const uint64_t e = RING(WA(shead + i));
            const uint32_t sw = STATE(WA(shead + i));
            if (!is_dead(sw)) {
                if (!(sw & kPrefillBit)) resj += t_end - (int)sw + entry_o(e);
                age += t_end - entry_tarr(e) + 1;
            }
        }
        for (int i = lane; i < nQ; i += 32) age += t_end - entry_tarr(gq[(qh + (uint32_t)i) & qmask]) + 1;
        age = warp_sum64(age);
        resj = warp_sum64(resj);
        CADD(C_SUM_U, sumU);
        CADD(C_SUM_N, sumN);
        CADD(C_TOKENS_GENERATED, tokgen);
        CADD(C_ARRIVED, arrived);
        CADD(C_DROPPED, arrived - accepted);
        CADD(C_COMPLETED, completed);
        CADD(C_SUM_LAT, warp_sum64((long long)acc_lat));
        CADD(C_SUM_W_COMPLETED, warp_sum64((long long)acc_w));
        CADD(C_COMPLETED_TOKENS, warp_sum64((long long)acc_o));
        CMAX(C_MAX_LAT, __reduce_max_sync(FULL, acc_maxlat));
        CMAX(C_MAX_U, max(maxU, U));  // U: the usage of the last slot if nothing left in it
        CMAX(C_MAX_Q, maxQ);
        CSET(C_STEPS_DONE, t_end);
        CSET(C_STATUS, status);
        CSET(C_N_LOGGED, n_logged);
        CSET(C_Q_FINAL, nQ);
        CSET(C_P_FINAL, nP - nD);
        CSET(C_RESID_AGE, age);
        CSET(C_RESID_J, resj);
        CSET(C_MMPP_STATE, mstate);
        if (lane < C_COUNT) cptr[lane] = cnt;

        uint32_t out = 0;
        switch (lane) {
            case 0: out = qh; break;
            case 1: out = (uint32_t)shead; break;
            case 2: out = (uint32_t)nP; break;
            case 3: out = (uint32_t)nQ; break;
            case 4: out = (uint32_t)U; break;
            case 5: out = (uint32_t)Ndec; break;
            case 6: out = ~next_fin; break;
            case 7: out = (uint32_t)n_pref; break;
            case 8: out = (uint32_t)pf_lo; break;
            case 9: out = mstate; break;
            case 10: out = status; break;
            case 11: out = (uint32_t)nD; break;
            default: break;
        }
        if (lane < kHeaderWords) hdr[lane] = out;
        __syncwarp();  // every lane's last writes to the rings are visible before they are copied out
        {
            uint4* dst = reinterpret_cast<uint4*>(ws + kHeaderWords * 4);
            const uint4* src = reinterpret_cast<const uint4*>(my);
            for (int i = lane; i < state_bytes / 16; i += 32) dst[i] = src[i];
        }
        __syncwarp();
#undef CADD
#undef CMAX
#undef CSET
#undef WA
    }
}

// What the host launches: one function per policy's object (fcsim_step_kernels.cu) returns the kernel for a
// register allocation (CTAs per SM) and a variant (what is recorded, several heads at once, lazy arrivals).
typedef void (*step_kernel_t)(const Params);
step_kernel_t step_kernel_of_policy_0(int ctas, int rec, bool bulk, bool lazy);
step_kernel_t step_kernel_of_policy_1(int ctas, int rec, bool bulk, bool lazy);
step_kernel_t step_kernel_of_policy_2(int ctas, int rec, bool bulk, bool lazy);
step_kernel_t step_kernel_of_policy_3(int ctas, int rec, bool bulk, bool lazy);
step_kernel_t step_kernel_of_policy_4(int ctas, int rec, bool bulk, bool lazy);
step_kernel_t step_kernel_of_policy_5(int ctas, int rec, bool bulk, bool lazy);
step_kernel_t step_kernel_of_policy_6(int ctas, int rec, bool bulk, bool lazy);

}  // namespace fcsim_dev
