"""Plain oracle of the host-side policies around the serving step: the request handler's decision list and
offloading rule (paper Section 3.2, Eq. 1), the event-driven simulator with lookup-table compute latencies
(Section 5.2) that evaluates the placement objective (Eq. 2), and the state-aware placement (Algorithms 1, 2).

TEST INFRASTRUCTURE ONLY: shares no code with the C++ library, which implements the same rules in
csrc/policy.cu; tests compare the two on seeded instances and pin this file against hand-worked cases.
Everything is written in the paper's order and notation.  Where the paper leaves a choice open, the reading
is stated at the place it is taken.

Cluster model.  Servers n = 0 .. N-1 with gpus[n] identical GPUs; a GPU has compute capacity 1 (the MPS
share a_l of a service is a fraction of it) and `vram` GB.  Server N is the hypothetical server epsilon of
Algorithm 1, stage 3: it owns no GPU of its own and places an instance on free GPUs of any real servers.
A service l has: a (compute share), b (VRAM GB), n_gpus (GPUs one instance spans; 1 for the "<1 GPU"
categories), cat (0 latency-, 1 frequency-sensitive), bs (batch size), slo_ms (latency SLO of a request or
frame), fps and frames (frequency-sensitive: a request is `frames` frames arriving 1/fps apart), and
c_ms[k], the profiled compute time of a batch of up to 2^k requests (the c_ln lookup table).
A request is (t_ms, service, server, u[0..4]): arrival time, service, the server it reaches first, and the
pre-drawn uniform numbers its offloading decisions consume (one per offload, so both implementations and
every evaluation of the objective see the same choices).

"parity unpinned": none.  Pins: tests/test_policy.py (Eq. 1 by hand, the decision list case by case, a
two-server simulation worked by hand, Algorithm 2's tie set and its two loop conditions, the 120-frame
goodput example of Section 3.3).
"""
from __future__ import annotations

import heapq
import math
from typing import Dict, List, Optional, Sequence, Tuple

MAX_OFFLOAD = 5          # Section 4.1 "Maximum offloading count", Table 4
LOCAL, OFFLOAD, TIMEOUT, OFFLOAD_EXCEED, INSUFFICIENT = 0, 1, 2, 3, 4


# ------------------------------------------------------------------------------------ Eq. 1
def offload_probabilities(p_hat: Sequence[float], p_act: Sequence[float], queued_ms: Sequence[float],
                          t_sync_ms: Sequence[float], slo_ms: float) -> List[float]:
    """Eq. 1.  Candidate m has idle goodput p~_m = p^_m - p_m (theoretical minus actual goodput over the window
    [-2 t_m, -t_m]); it is excluded when the expected computation time of its queued requests exceeds
    t_m + SLO_r.  The request is offloaded to m with probability p~_m / sum of p~ over the candidates.
    Reading: a negative idle goodput counts as 0; if no candidate has idle goodput the list is all zeros."""
    idle = []
    for m in range(len(p_hat)):
        ok = queued_ms[m] <= t_sync_ms[m] + slo_ms
        idle.append(max(0.0, p_hat[m] - p_act[m]) if ok else 0.0)
    s = sum(idle)
    return [v / s for v in idle] if s > 0 else [0.0] * len(idle)


def pick(prob: Sequence[float], u: float) -> int:
    """Index chosen by a uniform number u in [0, 1): the first m with u < prob[0] + .. + prob[m]; -1 if all zero."""
    acc = 0.0
    last = -1
    for m, p in enumerate(prob):
        if p <= 0:
            continue
        acc += p
        last = m
        if u < acc:
            return m
    return last


# ------------------------------------------------------------------------------------ compute-time lookup
def compute_ms(c_ms: Sequence[float], batch: int) -> float:
    """c_ln lookup: the profiled time of the smallest power-of-two batch that holds `batch` requests."""
    k = 0
    while (1 << k) < batch and k + 1 < len(c_ms):
        k += 1
    return c_ms[k]


# ------------------------------------------------------------------------------------ placement bookkeeping
def try_place(cluster: Dict, services: Sequence[Dict], used: List[List[List[float]]], l: int, n: int) -> Optional[List[Tuple[int, int]]]:
    """Resources for one instance of service l on server n (n == N: the hypothetical server).  First fit: GPUs
    are scanned in (server, gpu) order and the first n_gpus with a and b free are taken; all on server n for a
    real server, on any servers for epsilon.  Returns the (server, gpu) list and books the resources, or None."""
    N = len(cluster["gpus"])
    s = services[l]
    servers = range(N) if n == N else [n]
    got = []
    for sv in servers:
        for gidx in range(cluster["gpus"][sv]):
            cu, vu = used[sv][gidx]
            if cu + s["a"] <= 1.0 + 1e-12 and vu + s["b"] <= cluster["vram"] + 1e-12:
                got.append((sv, gidx))
                if len(got) == s["n_gpus"]:
                    for (x, y) in got:
                        used[x][y][0] += s["a"]
                        used[x][y][1] += s["b"]
                    return got
    return None


def feasible(cluster: Dict, services: Sequence[Dict], placements: Sequence[Tuple[int, int]]) -> bool:
    used = [[[0.0, 0.0] for _ in range(g)] for g in cluster["gpus"]]
    return all(try_place(cluster, services, used, l, n) is not None for (l, n) in placements)


# ------------------------------------------------------------------------------------ simulator (Section 5.2)
class _Instance:
    def __init__(self, l, n):
        self.l, self.n = l, n
        self.queue: List[int] = []       # work item ids, oldest first
        self.busy_until = 0.0
        self.running = False
        self.done_times: List[float] = []   # completion times of served items (for the actual goodput p)


def simulate(cluster: Dict, services: Sequence[Dict], requests: Sequence[Dict], placements: Sequence[Tuple[int, int]],
             max_offload: int = MAX_OFFLOAD) -> Dict:
    """Replays `requests` against `placements` under the request-handling strategy of Section 3.2 and returns
    phi (Eq. 2: satisfied requests; a frequency-sensitive request of F frames counts F x achieved / required fps,
    at most F) and the handler's answer counts.

    Event-driven: the only events are arrivals (of a request, a frame, or an offloaded item at its new server)
    and batch completions; compute latency comes from the lookup table, transmission is a fixed
    cluster["offload_ms"] per hop.  Events at equal times are served in the order they were scheduled.

    A placed instance is a single queue: when it is idle and its queue is not empty it drops the items whose
    deadline has passed (timeout), takes the oldest bs of the rest as one batch and is busy for c(batch).
    Handling of an item reaching server n at time `now` (Section 3.2, in the paper's order):
      1. deadline passed -> timeout;
      2. a local instance (on n, then on the hypothetical server) is sufficient when the item would finish in
         time there: busy time left + c(bs) per full batch already queued + c(batch it joins) <= time to the
         deadline; the one finishing earliest takes it;
      3. otherwise, offload count == max_offload -> offloading exceed;
      4. otherwise Eq. 1 over the servers not yet on the item's path that hold an instance of its service
         (p^: sum of bs / c(bs) of those instances; p: their completions in [now - 2t, now - t] / t, t =
         cluster["sync_ms"]; queued computation time: the smallest over the server's instances); the item moves
         to the picked server and its offload count grows; no candidate with idle goodput -> resource
         insufficiency."""
    N = len(cluster["gpus"])
    t_sync = cluster["sync_ms"]
    used = [[[0.0, 0.0] for _ in range(g)] for g in cluster["gpus"]]
    insts: List[_Instance] = []
    for (l, n) in placements:
        if try_place(cluster, services, used, l, n) is not None:
            insts.append(_Instance(l, n))
    by_server: Dict[Tuple[int, int], List[int]] = {}
    for i, it in enumerate(insts):
        by_server.setdefault((it.n, it.l), []).append(i)

    # work items: one per latency-sensitive request, one per frame of a frequency-sensitive request
    items = []       # dict(req, l, arrive, deadline, count, path)
    events: List[Tuple[float, int, int, int, int]] = []     # (time, seq, kind 0 arrival / 1 completion, a, b)
    seq = 0
    for r, rq in enumerate(requests):
        s = services[rq["service"]]
        nf = s["frames"] if s["cat"] == 1 else 1
        for f in range(nf):
            t = rq["t_ms"] + (1000.0 * f / s["fps"] if s["cat"] == 1 else 0.0)
            items.append({"req": r, "l": rq["service"], "arrive": t, "deadline": t + s["slo_ms"], "count": 0,
                          "path": [rq["server"]], "done": None})
            heapq.heappush(events, (t, seq, 0, len(items) - 1, rq["server"]))
            seq += 1
    answers = {"served": 0, "timeout": 0, "offload_exceed": 0, "insufficient": 0, "late": 0, "offloads": 0}

    def queued_ms(i: int, now: float, extra: int) -> float:
        """Time until an item joining instance i now (as the extra-th newcomer) would finish."""
        it = insts[i]
        s = services[it.l]
        left = max(0.0, it.busy_until - now) if it.running else 0.0
        q = len(it.queue) + extra
        full, rest = divmod(q, s["bs"])
        return left + full * compute_ms(s["c_ms"], s["bs"]) + (compute_ms(s["c_ms"], rest) if rest else 0.0)

    def start(i: int, now: float):
        nonlocal seq
        it = insts[i]
        s = services[it.l]
        live = []
        for w in it.queue:
            if items[w]["deadline"] < now:
                answers["timeout"] += 1
            else:
                live.append(w)
        batch, it.queue = live[:s["bs"]], live[s["bs"]:]
        if not batch:
            it.running = False
            return
        it.running = True
        it.busy_until = now + compute_ms(s["c_ms"], len(batch))
        it.batch = batch
        heapq.heappush(events, (it.busy_until, seq, 1, i, 0))
        seq += 1

    while events:
        now, _, kind, a, b = heapq.heappop(events)
        if kind == 1:
            it = insts[a]
            for w in it.batch:
                items[w]["done"] = now
                it.done_times.append(now)
                if now <= items[w]["deadline"]:
                    answers["served"] += 1
                else:
                    answers["late"] += 1
            it.running = False
            if it.queue:
                start(a, now)
            continue
        w, n = a, b
        item = items[w]
        l = item["l"]
        s = services[l]
        if item["deadline"] < now:                                           # 1. timed out
            answers["timeout"] += 1
            continue
        best, best_t = -1, math.inf                                          # 2. local, then the hypothetical server
        for srv in (n, N):
            for i in by_server.get((srv, l), []):
                t_fin = queued_ms(i, now, 1)
                if now + t_fin <= item["deadline"] and t_fin < best_t:
                    best, best_t = i, t_fin
            if best >= 0:
                break
        if best >= 0:
            insts[best].queue.append(w)
            if not insts[best].running:
                start(best, now)
            continue
        if item["count"] >= max_offload:                                     # 3. offloading exceed
            answers["offload_exceed"] += 1
            continue
        cand = [m for m in range(N) if m not in item["path"] and by_server.get((m, l))]
        p_hat, p_act, q_ms = [], [], []                                      # 4. Eq. 1
        for m in cand:
            ids = by_server[(m, l)]
            p_hat.append(sum(s["bs"] / compute_ms(s["c_ms"], s["bs"]) * 1000.0 for _ in ids))
            done = sum(1 for i in ids for d in insts[i].done_times if now - 2 * t_sync <= d <= now - t_sync)
            p_act.append(done / t_sync * 1000.0 if t_sync > 0 else 0.0)
            q_ms.append(min(queued_ms(i, now, 0) for i in ids))
        prob = offload_probabilities(p_hat, p_act, q_ms, [t_sync] * len(cand), s["slo_ms"])
        k = pick(prob, requests[item["req"]]["u"][item["count"]])
        if k < 0:
            answers["insufficient"] += 1
            continue
        item["count"] += 1
        item["path"].append(cand[k])
        answers["offloads"] += 1
        heapq.heappush(events, (now + cluster["offload_ms"], seq, 0, w, cand[k]))
        seq += 1

    # Eq. 2
    phi = 0.0
    per_req: Dict[int, List[Dict]] = {}
    for item in items:
        per_req.setdefault(item["req"], []).append(item)
    for r, its in per_req.items():
        s = services[requests[r]["service"]]
        if s["cat"] == 0:
            phi += 1.0 if (its[0]["done"] is not None and its[0]["done"] <= its[0]["deadline"]) else 0.0
        else:
            done = [it["done"] for it in its if it["done"] is not None and it["done"] <= it["deadline"]]
            if done:
                span_ms = max(done) - its[0]["arrive"]
                achieved = len(done) / (span_ms / 1000.0) if span_ms > 0 else float("inf")
                phi += fs_credit(len(its), s["fps"], min(achieved, s["fps"] * len(done) / len(its)))
    answers["phi"] = phi
    answers["instances"] = len(insts)
    return answers


def fs_credit(frames: float, required_fps: float, achieved_fps: float) -> float:
    """Section 3.3: frames x achieved / required, never above the frame count (120 frames, 60 fps required,
    30 achieved -> 60)."""
    return frames * min(1.0, achieved_fps / required_fps)


# ------------------------------------------------------------------------------------ Algorithm 2 (SPF)
def spf(phi, X: Sequence[Tuple[int, int]], theta0: Sequence[Tuple[int, int]], is_set: bool, stage1: bool,
        feasible_fn) -> List[Tuple[int, int]]:
    """Submodular placement for full models.  phi(list of placements) -> objective; X a set of placements
    (every element may be placed again and again) or a priority list (each entry at most once).
    Each round evaluates phi(theta_{k-1} + delta) for every candidate delta that still fits, keeps the tie set
    of the best ones and adds one of it (reading: "arbitrary" = the first in X's order).  The loop goes on while
    the objective does not decrease in stage 1, and only while it strictly grows in the other stages; the
    result is theta_{k-1} of the round that ended the loop."""
    thetas = [list(theta0)]
    phis = [phi(thetas[0])]
    k = 0
    while True:
        k += 1
        tie: List[Tuple[int, int]] = []
        tie_val = None
        prev = thetas[k - 1]
        if is_set:
            cands = list(X)
        else:                                   # a list: the entries not used yet (multiset difference)
            left = list(prev)
            cands = []
            for d in X:
                if d in left:
                    left.remove(d)
                else:
                    cands.append(d)
        for d in cands:
            if not feasible_fn(prev + [d]):
                continue
            v = phi(prev + [d])
            if tie_val is None or v > tie_val:
                tie, tie_val = [d], v
            elif v == tie_val:
                tie.append(d)
        if not tie:
            break
        thetas.append(prev + [tie[0]])
        phis.append(tie_val)
        go_on = phis[k] >= phis[k - 1] if stage1 else phis[k] > phis[k - 1]
        if not go_on:
            break
    return thetas[k - 1]


# ------------------------------------------------------------------------------------ Algorithm 1 (SSSP)
def sssp(cluster: Dict, services: Sequence[Dict], requests: Sequence[Dict], priority: Sequence[Tuple[int, int]],
         max_offload: int = MAX_OFFLOAD) -> List[Tuple[int, int]]:
    """State-aware service placement: S1 the priority list, S2 every (service, real server) as a set, S3 every
    (service, hypothetical server); each stage continues from the placement list of the one before."""
    N, L = len(cluster["gpus"]), len(services)
    phi = lambda th: simulate(cluster, services, requests, th, max_offload)["phi"]
    feas = lambda th: feasible(cluster, services, th)
    th1 = spf(phi, list(priority), [], False, True, feas)
    X = [(l, n) for l in range(L) for n in range(N)]
    th2 = spf(phi, X, th1, True, False, feas)
    Xe = [(l, N) for l in range(L)]
    return spf(phi, Xe, th2, True, False, feas)
