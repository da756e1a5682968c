"""Pure-Python cross-checks for the CPU checker (test-only).

* ``philox_py``: Philox4x32-10 written from its published definition with Python integers.
* ``sample_py``: the inverse-CDF rule as a literal linear scan.
* ``brute_force``: an event-free, bookkeeping-free evaluator of the model for tiny inputs: every
  request is a record with a status; the queue order is *derived* (waiting requests sorted by arrival
  id), the active order is derived (sorted by activation sequence number), and every quantity is
  recomputed from the records each slot.  It deliberately shares no structure with the C++ checker.
"""
from __future__ import annotations

M32 = 0xFFFFFFFF


def philox_py(ctr, key):
    c = [int(x) & M32 for x in ctr]
    k0, k1 = int(key[0]) & M32, int(key[1]) & M32
    for r in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k0) & M32, p1 & M32, ((p0 >> 32) ^ c[3] ^ k1) & M32, p0 & M32]
        k0 = (k0 + 0x9E3779B9) & M32
        k1 = (k1 + 0xBB67AE85) & M32
    return tuple(c)


def sample_py(tab, u):
    cdf = [int(x) for x in tab.cdf]
    for k in range(len(cdf) - 1):
        if u < cdf[k]:
            return tab.vmin + k
    return tab.vmin + len(cdf) - 1


def brute_force(cfg, replica, n_steps):
    """Returns dict(U=[..], Q=[..], completions=[(t, lat)..], counters={...}) for one replica."""
    # locate the group
    first = 0
    for g in cfg.groups:
        if replica < first + g.n_replicas:
            grp, rid = g, g.rng_replica_base + (replica - first)
            break
        first += g.n_replicas
    key = (cfg.seed & M32, (cfg.seed >> 32) & M32)
    arr = cfg.arrivals[grp.arrivals_id]
    keep = bool(getattr(grp, "preempt_keep", 0))
    reqs = []           # dicts: id, l, o, t_arr, status in {'wait','active','done'}, act_seq, p, j
    act_seq = 0
    state = 0
    U_tr, Q_tr, comps = [], [], []
    cnt = dict(arrived=0, dropped=0, admitted=0, completed=0, evictions=0, overflow_steps=0,
               gate_blocked_steps=0, budget_blocked_steps=0, acap_blocked_steps=0, tokens_generated=0,
               prefill_tokens=0, completed_tokens=0, wasted_tokens=0, sum_lat=0, max_lat=0, sum_U=0,
               max_U=0, sum_N=0, max_Q=0, sum_w_completed=0)

    def waiting():
        return sorted((r for r in reqs if r["status"] == "wait"), key=lambda r: r["id"])

    def active():
        return sorted((r for r in reqs if r["status"] == "active"), key=lambda r: r["act_seq"])

    def prospective():
        # usage at the end of this slot if nothing else changes: p + j + one new token if prefilled
        return sum(r["p"] + r["j"] + (1 if r["p"] == r["l"] else 0) for r in active())

    for t in range(1, n_steps + 1):
        w = philox_py((t, rid, 0, 0), key)
        if arr.n_states == 2 and w[2] < arr.switch_thr[state]:
            state ^= 1
        n_t = sample_py(arr.count[state], w[0])
        B_t = (grp.b_fp >> 16) + (1 if (w[1] >> 16) < (grp.b_fp & 0xFFFF) else 0)
        for i in range(n_t):
            a = philox_py((t, rid, 1, i), key)
            cls = sample_py(cfg.class_law, a[0])
            l = sample_py(cfg.prompt[cls], a[1])
            o = sample_py(cfg.decode[cls], a[2])
            cnt["arrived"] += 1
            if len(waiting()) >= cfg.Qcap:
                cnt["dropped"] += 1
            else:
                o_proj = o
                if grp.policy == 5 and grp.mc_worst_case:
                    o_proj = cfg.decode[cls].vmin + len(cfg.decode[cls].cdf) - 1
                reqs.append(dict(id=len(reqs), cls=cls, l=l, o=o, o_proj=o_proj, t_arr=t, status="wait",
                                 act_seq=None, p=0, j=0, l0=l, o0=o, kept=0))
        n_dec_start = sum(1 for r in active() if r["p"] == r["l"])
        room = None if cfg.K == 0 else (max(0, cfg.K - n_dec_start) if grp.policy == 2 else cfg.K)
        if grp.policy == 2:
            for r in active():
                if r["p"] < r["l"]:
                    g = min(grp.chunk, r["l"] - r["p"]) if room is None else min(grp.chunk, r["l"] - r["p"], room)
                    r["p"] += g
                    if room is not None:
                        room -= g
                    cnt["prefill_tokens"] += g
        admitted_now = 0
        if grp.policy == 4:
            # Algorithm 1: per class k up to b_k picks, oldest waiting request of that class first
            hits = set()
            stop = False
            for k in range(len(cfg.prompt)):
                if stop:
                    break
                for _ in range(grp.b_class[k]):
                    cand = [r for r in waiting() if r["cls"] == k]
                    if not cand:
                        break
                    if len(active()) == cfg.Acap:
                        hits.add("acap_blocked_steps")
                        stop = True
                        break
                    h = cand[0]
                    if not (room is None or admitted_now == 0 or h["l"] <= room):
                        hits.add("budget_blocked_steps")
                        break
                    if prospective() + h["l"] + 1 > cfg.M:
                        hits.add("gate_blocked_steps")
                        break
                    h["status"], h["p"], h["j"], h["act_seq"] = "active", h["l"], 0, act_seq
                    act_seq += 1
                    if room is not None:
                        room -= min(h["l"], room)
                    admitted_now += 1
                    cnt["admitted"] += 1
                    cnt["prefill_tokens"] += h["l"]
            for name in hits:
                cnt[name] += 1
        while grp.policy != 4:
            if grp.policy == 0 and admitted_now >= B_t:
                break
            wq = waiting()
            if not wq:
                break
            if len(active()) == cfg.Acap:
                cnt["acap_blocked_steps"] += 1
                break
            h = wq[0]
            if grp.policy == 2:
                g = min(grp.chunk, h["l"]) if room is None else min(grp.chunk, h["l"], room)
                if g == 0:
                    cnt["budget_blocked_steps"] += 1
                    break
                need = g + (1 if g == h["l"] else 0)
            else:
                g = h["l"]
                if not (room is None or admitted_now == 0 or g <= room):
                    cnt["budget_blocked_steps"] += 1
                    break
                need = g + 1
            if grp.policy == 5:
                # MC benchmark: run the system forward with no further arrivals or activations and look at
                # the usage of every slot until everything has (by projection) finished
                proj = [dict(l=r["l"], j=r["j"], left=r["o_proj"] - r["j"]) for r in active()]
                proj.append(dict(l=h["l"], j=0, left=h["o_proj"]))
                ok = True
                while proj and ok:
                    for q in proj:
                        q["j"] += 1
                        q["left"] -= 1
                    ok = sum(q["l"] + q["j"] for q in proj) <= cfg.M
                    proj = [q for q in proj if q["left"] > 0]
                if not ok:
                    cnt["gate_blocked_steps"] += 1
                    break
            limit = grp.m_admit if grp.policy == 3 else cfg.M   # alpha-protection: keep usage <= (1-alpha) M
            if prospective() + need > limit:
                cnt["gate_blocked_steps"] += 1
                break
            h["status"], h["p"], h["j"], h["act_seq"] = "active", g, 0, act_seq
            act_seq += 1
            if room is not None:
                room -= min(g, room)
            admitted_now += 1
            cnt["admitted"] += 1
            cnt["prefill_tokens"] += g
        if prospective() > cfg.M:
            cnt["overflow_steps"] += 1
            while (active() if grp.policy == 3 else prospective() > cfg.M):   # alpha-protection evicts all
                r = active()[-1]
                cnt["evictions"] += 1
                if keep:
                    # the generated tokens stay with the request: it comes back with them in its prompt
                    r["kept"] += r["j"]
                    r["l"], r["o"] = r["l0"] + r["kept"], r["o0"] - r["kept"]
                else:
                    cnt["wasted_tokens"] += r["j"]
                r["status"], r["p"], r["j"], r["act_seq"] = "wait", 0, 0, None
        for r in active():
            if r["p"] == r["l"]:
                r["j"] += 1
                cnt["tokens_generated"] += 1
        U = sum(r["p"] + r["j"] for r in active())
        assert U <= cfg.M
        cnt["sum_U"] += U
        cnt["max_U"] = max(cnt["max_U"], U)
        cnt["sum_N"] += len(active()) + len(waiting())
        for r in active():
            if r["p"] == r["l"] and r["j"] == r["o"]:
                lat = t - r["t_arr"] + 1
                r["status"] = "done"
                comps.append((t, lat))
                cnt["completed"] += 1
                cnt["sum_lat"] += lat
                cnt["max_lat"] = max(cnt["max_lat"], lat)
                if not keep:
                    cnt["completed_tokens"] += r["o"]
                    cnt["sum_w_completed"] += sum(r["l"] + jj for jj in range(1, r["o"] + 1))
        U_tr.append(U)
        Q_tr.append(len(waiting()))
        cnt["max_Q"] = max(cnt["max_Q"], len(waiting()))
    if keep:
        # tokens that can no longer be lost, request by request, in terms of the ORIGINAL lengths: all o0 of a
        # finished request, the kept ones of the others; and the cache-slots those tokens occupied when made
        for r in reqs:
            n_final = r["o0"] if r["status"] == "done" else r["kept"]
            cnt["completed_tokens"] += n_final
            cnt["sum_w_completed"] += sum(r["l0"] + i for i in range(1, n_final + 1))
    cnt["q_final"] = len(waiting())
    cnt["p_final"] = len(active())
    cnt["resid_age"] = sum(n_steps - r["t_arr"] + 1 for r in reqs if r["status"] in ("wait", "active"))
    cnt["resid_j"] = sum(r["j"] for r in active())
    cnt["mmpp_state"] = state
    return dict(U=U_tr, Q=Q_tr, completions=comps, counters=cnt)
