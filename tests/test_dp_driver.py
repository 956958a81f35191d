"""The replica driver on CPU threads: frames of several streams dealt over fake replicas that finish in a
scrambled order must come back per stream in frame order, each served exactly once by the replica the
round-robin rule names; sticky streams stay on one replica; Eq. 4 comes from the library."""
import random
import threading
import time

import pytest

from paper_2511_00603_b200 import dp


class FakeReplica:
    """Stands in for one GPU's context: serves a batch after a random delay, remembers who called it."""

    def __init__(self, index, seed, fail_on=None):
        self.index, self.rng, self.fail_on = index, random.Random(seed), fail_on
        self.thread_ids, self.served, self.batches = set(), [], []

    def __call__(self, batch):
        self.thread_ids.add(threading.get_ident())
        time.sleep(self.rng.random() * 0.004)
        self.batches.append(len(batch))
        out = []
        for stream, frame, payload in batch:
            if self.fail_on == (stream, frame):
                raise RuntimeError("replica failed")
            self.served.append((stream, frame))
            out.append((self.index, payload * 2 + 1))
        return out


@pytest.mark.parametrize("n_replicas", [1, 2, 3])
def test_frames_come_back_in_order_and_are_dealt_round_robin(n_replicas):
    reps = [FakeReplica(k, seed=k) for k in range(n_replicas)]
    drv = dp.ReplicaDriver(reps, max_batch=4)
    n_streams, n_frames = 5, 40
    rng = random.Random(9)
    for f in range(n_frames):
        order = list(range(n_streams))
        rng.shuffle(order)
        for s in order:
            k = drv.submit(s, f, payload=1000 * s + f, sticky=(s >= 3))
            assert k == dp.replica_of(s, f, n_replicas, s >= 3)
        if f % 7 == 0:
            time.sleep(0.002)
    got = drv.drain()
    drv.close()
    assert len(got) == n_streams * n_frames
    per_stream = {s: [] for s in range(n_streams)}
    for s, f, (replica, value) in got:
        per_stream[s].append(f)
        assert value == (1000 * s + f) * 2 + 1
        assert replica == dp.replica_of(s, f, n_replicas, s >= 3)
    for s in range(n_streams):
        assert per_stream[s] == list(range(n_frames)), f"stream {s} out of order"
    for r in reps:
        assert len(r.thread_ids) <= 1                      # one host thread per replica
        assert len(r.served) == len(set(r.served))         # nothing served twice
        assert max(r.batches, default=0) <= 4
    for s in (3, 4):                                       # sticky streams live on one replica
        assert len({k for k, r in enumerate(reps) if any(st == s for st, _ in r.served)}) == 1


def test_a_failing_replica_is_reported_and_the_others_keep_serving():
    reps = [FakeReplica(0, seed=1), FakeReplica(1, seed=2, fail_on=(0, 3))]
    drv = dp.ReplicaDriver(reps, max_batch=1)
    for f in range(6):
        drv.submit(0, f, payload=f)
    with pytest.raises(RuntimeError):
        drv.drain(timeout=10)
    drv.close()
    assert (0, 4) in reps[0].served and (0, 2) in reps[0].served       # replica 0 went on


def test_ordered_delivery_releases_only_consecutive_frames():
    od = dp.OrderedDelivery()
    assert od.put(7, 1, "b") == []
    assert od.put(7, 2, "c") == []
    assert od.put(8, 0, "x") == [(8, 0, "x")]
    assert od.put(7, 0, "a") == [(7, 0, "a"), (7, 1, "b"), (7, 2, "c")]
    with pytest.raises(ValueError):
        od.put(7, 1, "again")


def test_group_count_is_the_librarys_eq4():
    from oracle import epara_oracle as O
    for req, grp in [(97, 49), (98, 49), (99, 49), (60, 60), (1, 100), (120.5, 30)]:
        assert dp.dp_group_count(req, grp) == O.dp_group_count(req, grp)
    with pytest.raises(ValueError):
        dp.dp_group_count(10, 0)
