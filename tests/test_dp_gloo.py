"""Two-rank CPU (gloo) test of the replica path: disjoint, complete sharding of requests, sticky
decoder sequences, Eq. 4, max-over-ranks throughput aggregation, and delivery in frame order of results
that two replica processes produce at different speeds."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2511_00603_b200 import dp
    reqs = [{"id": i, "stream": i % 5, "frame": i // 5, "sticky": (i % 5) >= 3} for i in range(100)]
    mine = dp.shard_requests(reqs, rank, world)
    ids = torch.zeros(100, dtype=torch.int64)
    for r in mine:
        ids[r["id"]] = 1
    dist.all_reduce(ids)                      # every request is served exactly once
    sticky_ok = all(dp.replica_of(r["stream"], r["frame"], world, True) == rank for r in mine if r["sticky"])
    # rank 0 takes 10 ms for its share, rank 1 takes 25 ms: the job ran at (n0 + n1) / 25 ms
    thr = dp.whole_job_throughput(len(mine), 10.0 if rank == 0 else 25.0)
    # ordered delivery across processes: every rank "serves" its frames (rank 1 reports them in reverse, as a
    # slower replica would), rank 0 merges the reports through the reorder buffer
    done = [(r["stream"], r["frame"], r["id"] * 3) for r in mine]
    if rank == 1:
        done.reverse()
    reports = [None] * world
    dist.all_gather_object(reports, done)
    ordered_ok = True
    if rank == 0:
        od = dp.OrderedDelivery()
        released = []
        for i in range(max(len(x) for x in reports)):
            for rep in reports:
                if i < len(rep):
                    released += od.put(*rep[i])
        per = {}
        for s, f, val in released:
            per.setdefault(s, []).append(f)
            ordered_ok = ordered_ok and val == (f * 5 + s) * 3
        ordered_ok = ordered_ok and len(released) == 100 and all(per[s] == list(range(20)) for s in range(5))
    out.put((rank, len(mine), bool((ids == 1).all()), sticky_ok and ordered_ok, thr))
    dist.destroy_process_group()


def test_two_replicas_share_the_requests_and_report_job_throughput():
    from paper_2511_00603_b200 import dp
    assert dp.dp_group_count(97, 49) == 2 and dp.dp_group_count(99, 49) == 3
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in ps:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, n0, all0, st0, t0), (r1, n1, all1, st1, t1) = res
    assert n0 + n1 == 100 and all0 and all1 and st0 and st1
    assert abs(t0 - 100 / 0.025) < 1e-6 and abs(t1 - t0) < 1e-9
    # frames of a non-sticky stream alternate between the replicas
    assert [dp.replica_of(0, f, 2, False) for f in range(4)] == [0, 1, 0, 1]
    assert len({dp.replica_of(3, f, 2, True) for f in range(9)}) == 1
