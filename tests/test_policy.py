"""Host policies: the offloading rule (Eq. 1), the handler's decision list, the event-driven simulator and the
placement algorithms.  The oracle (oracle/policy_oracle.py) is pinned by hand-worked cases; the C++ library
is compared with it on seeded random instances.  No GPU."""
import math

import numpy as np
import pytest

from oracle import policy_oracle as P


@pytest.fixture(scope="module")
def E():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara
    return epara


def svc(cat=0, bs=4, slo=100.0, c=10.0, a=0.5, b=4.0, n_gpus=1, fps=0.0, frames=0, c_ms=None):
    return {"a": a, "b": b, "n_gpus": n_gpus, "cat": cat, "bs": bs, "slo_ms": slo, "fps": fps, "frames": frames,
            "c_ms": list(c_ms) if c_ms is not None else [c] * 10}


def req(t, l, n, u=0.5):
    return {"t_ms": float(t), "service": l, "server": n, "u": [u] * 5}


CL2 = {"gpus": [1, 1], "vram": 16.0, "sync_ms": 50.0, "offload_ms": 2.0}


# ------------------------------------------------------------------------------------ Eq. 1
def test_eq1_by_hand_and_exclusion(E):
    # idle goodputs 30, 10, 0 (negative counts as 0), the fourth excluded: queued 130 > t + SLO = 20 + 100
    args = ([50.0, 40.0, 20.0, 90.0], [20.0, 30.0, 25.0, 10.0], [10.0, 120.0, 0.0, 130.0], [20.0] * 4, 100.0)
    exp = [0.75, 0.25, 0.0, 0.0]
    assert P.offload_probabilities(*args) == exp
    assert E.epara_offload_probabilities(*args) == exp
    assert P.offload_probabilities([5.0], [9.0], [0.0], [1.0], 10.0) == [0.0]          # nobody has idle goodput
    assert P.pick(exp, 0.74) == 0 and P.pick(exp, 0.75) == 1 and P.pick(exp, 0.999) == 1 and P.pick([0.0, 0.0], 0.3) == -1


# ------------------------------------------------------------------------------------ decision list
def test_handler_decision_list_case_by_case(E):
    s = [svc(bs=1, slo=25.0, c=10.0)]
    for sim in (P.simulate, E.epara_simulate):
        # local: one instance on server 0, requests 30 ms apart are each served alone in time
        r = sim(CL2, s, [req(0, 0, 0), req(30, 0, 0)], [(0, 0)])
        assert (r["served"], r["phi"], r["offloads"]) == (2, 2.0, 0)
        # three at once on one instance with batch 1: the third would finish at 30 > 25: not sufficient locally,
        # no other server holds the service -> resource insufficiency
        r = sim(CL2, s, [req(0, 0, 0), req(0, 0, 0), req(0, 0, 0)], [(0, 0)])
        assert (r["served"], r["insufficient"], r["phi"]) == (2, 1, 2.0)
        # the same with an instance on server 1: offloaded (2 ms hop), served there at 12 <= 25
        r = sim(CL2, s, [req(0, 0, 0), req(0, 0, 0), req(0, 0, 0)], [(0, 0), (0, 1)])
        assert (r["served"], r["offloads"], r["insufficient"], r["phi"]) == (3, 1, 0, 3.0)
        # maximum offloading count 0: the same request answers offloading exceed instead
        r = sim(CL2, s, [req(0, 0, 0), req(0, 0, 0), req(0, 0, 0)], [(0, 0), (0, 1)], 0)
        assert (r["served"], r["offload_exceed"]) == (2, 1)
        # a request whose service is placed nowhere: resource insufficiency; nothing placed at all: the same
        assert sim(CL2, s, [req(0, 0, 1)], [])["insufficient"] == 1
        # timeout: the hop takes 2 ms, the SLO of this service is 1 ms, so the offloaded item arrives expired
        tight = [svc(bs=1, slo=1.0, c=0.5)]
        r = sim(CL2, tight, [req(0, 0, 0)], [(0, 1)])
        assert (r["offloads"], r["timeout"], r["phi"]) == (1, 1, 0.0)


def test_offloaded_items_never_revisit_a_server(E):
    """Three servers, the service only on server 2, too slow to be of use there (c = 50 > SLO 20): the item goes
    0 -> 2 (the only candidate), cannot be served, and has no candidate left: one offload, then insufficiency."""
    cl = {"gpus": [1, 1, 1], "vram": 16.0, "sync_ms": 5.0, "offload_ms": 1.0}
    s = [svc(bs=1, slo=20.0, c=50.0)]
    for sim in (P.simulate, E.epara_simulate):
        r = sim(cl, s, [req(0, 0, 0)], [(0, 2)])
        assert (r["offloads"], r["insufficient"], r["served"]) == (1, 1, 0)


def test_two_server_trace_worked_by_hand(E):
    """Batch 2, c(1) = 8 ms, c(2) = 10 ms, SLO 30.  Server 0: arrivals at 0, 1, 2, 3.
    t=0: starts alone (done 8).  t=1: queue 1 -> 7 left + c(1) = 15 <= 29: joins.  t=2: queue 2 -> 6 + c(2) = 16: joins.
    t=3: queue 3 -> 5 + c(2) + c(1) = 23 <= 27: joins.  t=8: batch {1, 2} until 18.  t=18: batch {3} until 26 <= 33.
    All four served, none offloaded."""
    s = [svc(bs=2, slo=30.0, c_ms=[8.0] + [10.0] * 9)]
    for sim in (P.simulate, E.epara_simulate):
        r = sim(CL2, s, [req(t, 0, 0) for t in (0, 1, 2, 3)], [(0, 0), (0, 1)])
        assert (r["served"], r["offloads"], r["late"], r["timeout"], r["phi"]) == (4, 0, 0, 0, 4.0)
        # a fifth arrival at t=4 would need 4 + c(2) + c(2) = 24 <= 26: still local; a sixth at t=5: 3 + 10 + 10 + 8 = 31 > 25: offloaded
        r = sim(CL2, s, [req(t, 0, 0) for t in (0, 1, 2, 3, 4, 5)], [(0, 0), (0, 1)])
        assert (r["served"], r["offloads"]) == (6, 1)


def test_frequency_goodput_example_of_section_3_3(E):
    """120 frames, required 50 fps, one instance that manages 25 fps (40 ms per frame, batch 1), generous frame SLO:
    every frame is served, the achieved rate is half the requirement, the request counts 120 x 25 / 50 = 60.
    (The paper's numbers are 60 fps required and 30 achieved; 50 / 25 keeps the arithmetic exact in binary.)"""
    s = [svc(cat=1, bs=1, slo=1e6, c=40.0, fps=50.0, frames=120)]
    assert P.fs_credit(120, 60, 30) == 60
    for sim in (P.simulate, E.epara_simulate):
        r = sim(CL2, s, [req(0, 0, 0)], [(0, 0)])
        assert r["served"] == 120 and abs(r["phi"] - 60.0) < 1e-9


# ------------------------------------------------------------------------------------ Algorithm 2
def test_spf_tie_set_first_member_and_loop_conditions():
    always = lambda th: True
    # objective: number of DISTINCT services placed -> the first round ties between all candidates
    phi = lambda th: float(len({l for l, _ in th}))
    X = [(1, 0), (0, 0), (1, 1)]
    # stage 2 rule (strict growth): places (1,0) [first of the tie set], then (0,0), then stops: the third round's best
    # addition leaves phi at 2, and the result is the list before that round's addition
    assert P.spf(phi, X, [], True, False, always) == [(1, 0), (0, 0)]
    # stage 1 rule (phi may stay equal) on a priority LIST: every entry is placed once, even without gain
    assert P.spf(phi, X, [], False, True, always) == [(1, 0), (0, 0), (1, 1)]
    # a list entry already in theta_0 is not placed again; feasibility filters candidates
    assert P.spf(phi, X, [(1, 0)], False, True, always) == [(1, 0), (0, 0), (1, 1)]
    assert P.spf(phi, X, [], True, False, lambda th: all(n == 0 for _, n in th)) == [(1, 0), (0, 0)]
    # stage 1 stops when an addition would LOWER the objective
    worse = lambda th: -float(len(th))
    assert P.spf(worse, X, [], False, True, always) == []


def _random_instance(rng, n_servers, n_services, n_requests, horizon_ms):
    cluster = {"gpus": [int(g) for g in rng.integers(1, 3, n_servers)], "vram": 16.0, "sync_ms": 20.0, "offload_ms": 1.5}
    services = []
    for l in range(n_services):
        cat = int(rng.integers(0, 2))
        base = float(rng.choice([2.0, 5.0, 9.0]))
        c_ms = [base * (1 + 0.25 * k) for k in range(10)]
        services.append(svc(cat=cat, bs=int(rng.choice([1, 2, 4])), slo=float(rng.choice([1.0, 15.0, 40.0, 120.0])), a=float(rng.choice([0.25, 0.5, 1.0])),
                            b=float(rng.choice([2.0, 6.0, 12.0])), n_gpus=int(rng.choice([1, 1, 2])), fps=float(rng.choice([20.0, 50.0])),
                            frames=int(rng.integers(3, 9)), c_ms=c_ms))
    requests = [{"t_ms": float(rng.uniform(0, horizon_ms)), "service": int(rng.integers(0, n_services)),
                 "server": int(rng.integers(0, n_servers)), "u": [float(x) for x in rng.random(5)]} for _ in range(n_requests)]
    requests.sort(key=lambda r: r["t_ms"])
    return cluster, services, requests


def test_library_simulator_equals_the_oracle_on_random_instances(E):
    rng = np.random.default_rng(0)
    keys = ["served", "timeout", "offload_exceed", "insufficient", "late", "offloads", "instances"]
    saw = {k: 0 for k in keys}
    for trial in range(60):
        N, L = int(rng.integers(1, 5)), int(rng.integers(1, 4))
        cluster, services, requests = _random_instance(rng, N, L, int(rng.integers(5, 60)), 200.0)
        placements = [(int(rng.integers(0, L)), int(rng.integers(0, N + 1))) for _ in range(int(rng.integers(0, 7)))]
        mo = int(rng.integers(0, 6))
        a, b = P.simulate(cluster, services, requests, placements, mo), E.epara_simulate(cluster, services, requests, placements, mo)
        for k in keys:
            assert a[k] == b[k], (trial, k, a, b)
            saw[k] += a[k]
        assert abs(a["phi"] - b["phi"]) <= 1e-9 * max(1.0, abs(a["phi"])), (trial, a, b)
    # every answer of the handler occurred somewhere (late: an item queued on an estimate that later arrivals,
    # batched with it, made too optimistic)
    assert all(saw[k] > 0 for k in keys), saw


def test_library_placement_equals_the_oracle_and_improves_goodput(E):
    rng = np.random.default_rng(1)
    for trial in range(6):
        N, L = int(rng.integers(2, 4)), int(rng.integers(2, 4))
        cluster, services, requests = _random_instance(rng, N, L, 30, 150.0)
        priority = [(int(rng.integers(0, L)), int(rng.integers(0, N)))]
        a = P.sssp(cluster, services, requests, priority)
        b = E.epara_place_sssp(cluster, services, requests, priority)
        assert a == b, (trial, a, b)
        assert P.feasible(cluster, services, a)
        phi = P.simulate(cluster, services, requests, a)["phi"]
        assert phi >= P.simulate(cluster, services, requests, [])["phi"]
        # greedy optimality of the last round: no single further placement on a real server strictly improves
        for l in range(L):
            for n in range(N + 1):
                if P.feasible(cluster, services, a + [(l, n)]):
                    more = P.simulate(cluster, services, requests, a + [(l, n)])["phi"]
                    if n == N:          # the last stage ended because nothing on the hypothetical server improves
                        assert more <= phi + 1e-12


def test_multi_gpu_service_goes_to_one_server_or_to_the_hypothetical_one(E):
    """A service spanning 2 GPUs fits server 1 (two GPUs) but not server 0 (one); with server 1 full it can only be
    placed on the hypothetical server, across servers (stage 3 of Algorithm 1)."""
    cl = {"gpus": [1, 2, 1], "vram": 16.0, "sync_ms": 10.0, "offload_ms": 1.0}
    s = [svc(a=1.0, b=10.0, n_gpus=2, bs=1, slo=50.0, c=5.0)]
    assert not P.feasible(cl, s, [(0, 0)]) and P.feasible(cl, s, [(0, 1)])
    assert not P.feasible(cl, s, [(0, 1), (0, 1)]) and P.feasible(cl, s, [(0, 1), (0, 3)])      # GPUs of servers 0 and 2
    reqs = [req(t, 0, n) for t in range(0, 40, 2) for n in (0, 2)]
    th = P.sssp(cl, s, reqs, [])
    assert th == E.epara_place_sssp(cl, s, reqs, []) and th[0] == (0, 1) and (0, 3) in th


# ------------------------------------------------------------------------------------ profiler -> simulator
def test_profile_table_drives_the_simulator(E):
    """The allocator's sweep on a synthetic timing model (step time 2 ms + 0.5 ms per request, halved per request
    beyond 64): BS sweep under a 20 ms SLO, then the replication sweep at that BS; the table's compute times
    are what the simulator and the placement use."""
    from paper_2511_00603_b200 import profiler
    calls = []

    def measure(name, bs, mt):
        calls.append((name, bs, mt))
        if bs * mt > 2048:
            return None                                          # does not fit: recorded as null, never chosen
        return (2.0 + 0.5 * min(bs, 64) + 0.25 * max(bs - 64, 0)) * (1 + 0.6 * (mt - 1))
    table = profiler.sweep(["svc"], measure, latency_slo_ms={"svc": 20.0})
    t = table["services"]["svc"]
    assert [c[1] for c in calls[:10]] == [1 << k for k in range(10)] and all(c[2] == 1 for c in calls[:10])   # BS first
    assert t["best_bs"] == 32            # 32 -> 18 ms (in the SLO), 64 -> 34 ms (not)
    assert [c[2] for c in calls[10:]] == [2, 4, 8, 16] and all(c[1] == 32 for c in calls[10:])               # then MT at that BS
    assert t["best_mt"] == 1             # every replica adds 60 % to an 18 ms step: none stays inside 20 ms
    assert t["c_ln_ms"]["32"] == 18.0 / 32 and profiler.compute_ms(table, "svc", 20) == 18.0
    s = profiler.service_from_table(table, "svc", cat=0, slo_ms=20.0, a=0.5, b=4.0)
    assert s["bs"] == 32 and s["c_ms"][:6] == [2.5, 3.0, 4.0, 6.0, 10.0, 18.0]
    reqs = [req(0.1 * i, 0, 0) for i in range(64)]
    a, b = P.simulate(CL2, [s], reqs, [(0, 0)]), E.epara_simulate(CL2, [s], reqs, [(0, 0)])
    assert a["served"] == b["served"] and a["phi"] == b["phi"] and a["served"] > 0
    # without an SLO the largest throughput wins, and replicas that do fit are weighed by requests per second
    free = profiler.sweep(["svc"], measure)["services"]["svc"]
    assert free["best_bs"] == 512 and free["best_mt"] in (1, 2, 4) and free["mt_step_ms"]["8"] is None
