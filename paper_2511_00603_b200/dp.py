"""Request-level data parallelism across GPUs (the paper's DP operator, Section 3.1; motivation in Section 2.3):
the full model set is replicated, the frames of a task are dealt round-robin over the replicas, and nothing is
exchanged between them.  How many replicas a frame-rate requirement needs is Eq. 4, taken from the library
(epara_dp_group_count).

ReplicaDriver is the runtime side: one worker thread per replica (on GPUs: one epara context per GPU, each driven
by its own host thread), frames dealt by replica_of, results handed back per stream in frame order whatever order
the replicas finish in.  A decoder sequence is sticky: all its steps go to the replica that holds its KV pages.
whole_job_throughput is the max-over-ranks aggregation the benchmark uses when replicas are separate processes."""
from __future__ import annotations

import queue
import threading
from typing import Any, Callable, Dict, List, Optional, Sequence, Tuple


def dp_group_count(required_fps: float, group_fps: float) -> int:
    """Eq. 4: ceil(frame-rate requirement / frame rate of one DP group), computed by the library."""
    from . import epara as E
    n = E.epara_dp_group_count(required_fps, group_fps)
    if n < 0:
        raise ValueError("frame rates must be positive")
    return n


def replica_of(stream_id: int, frame_index: int, n_replicas: int, sticky: bool) -> int:
    """Frames of a stream go round-robin over the replicas (alternating assignment); a decoder
    sequence is sticky -- all its steps go where its KV pages live."""
    return (stream_id % n_replicas) if sticky else ((stream_id + frame_index) % n_replicas)


def shard_requests(requests: Sequence[dict], rank: int, world: int) -> List[dict]:
    """The requests this rank serves.  Each request has 'stream', 'frame' and 'sticky'."""
    return [r for r in requests if replica_of(r["stream"], r["frame"], world, r["sticky"]) == rank]


def whole_job_throughput(local_units: int, local_ms: float, device="cpu") -> float:
    """Units processed by all ranks divided by the slowest rank's time (units/s).  Without an
    initialised process group this is the local figure."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return local_units / (local_ms / 1e3)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    n = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(n.item()) / (float(t.item()) / 1e3)


class OrderedDelivery:
    """Per-stream reorder buffer: results may arrive in any order; pop_ready() releases, for every stream, the
    longest run of consecutive frames starting at the next one owed."""

    def __init__(self):
        self.next: Dict[int, int] = {}
        self.held: Dict[int, Dict[int, Any]] = {}
        self.lock = threading.Lock()

    def put(self, stream: int, frame: int, result: Any) -> List[Tuple[int, int, Any]]:
        out = []
        with self.lock:
            h = self.held.setdefault(stream, {})
            if frame < self.next.get(stream, 0) or frame in h:
                raise ValueError(f"frame {frame} of stream {stream} delivered twice")
            h[frame] = result
            n = self.next.get(stream, 0)
            while n in h:
                out.append((stream, n, h.pop(n)))
                n += 1
            self.next[stream] = n
        return out


class ReplicaDriver:
    """Deals frames over replicas and returns results in frame order.

    backends: one callable per replica, run_batch(list of (stream, frame, payload)) -> list of results in the same
    order; it is only ever called from that replica's own thread (one epara context, one host thread).  Each worker
    takes whatever has queued up for its replica (at most max_batch frames) as one batch: one serving step."""

    def __init__(self, backends: Sequence[Callable[[List[Tuple[int, int, Any]]], List[Any]]], max_batch: int = 256,
                 on_result: Optional[Callable[[int, int, Any], None]] = None):
        self.n = len(backends)
        self.backends = list(backends)
        self.max_batch = max_batch
        self.inbox: List[queue.Queue] = [queue.Queue() for _ in range(self.n)]
        self.order = OrderedDelivery()
        self.delivered: List[Tuple[int, int, Any]] = []
        self.on_result = on_result
        self.out_lock = threading.Lock()
        self.errors: List[BaseException] = []
        self.pending = 0
        self.idle = threading.Condition()
        self.threads = [threading.Thread(target=self._work, args=(k,), daemon=True) for k in range(self.n)]
        for t in self.threads:
            t.start()

    def submit(self, stream: int, frame: int, payload: Any, sticky: bool = False) -> int:
        """Queues one frame; returns the replica it was dealt to."""
        k = replica_of(stream, frame, self.n, sticky)
        with self.idle:
            self.pending += 1
        self.inbox[k].put((stream, frame, payload))
        return k

    def _work(self, k: int):
        while True:
            item = self.inbox[k].get()
            if item is None:
                return
            batch = [item]
            while len(batch) < self.max_batch:
                try:
                    nxt = self.inbox[k].get_nowait()
                except queue.Empty:
                    break
                if nxt is None:
                    self.inbox[k].put(None)
                    break
                batch.append(nxt)
            try:
                results = self.backends[k](batch)
                for (stream, frame, _), res in zip(batch, results):
                    for rel in self.order.put(stream, frame, res):
                        with self.out_lock:
                            self.delivered.append(rel)
                            if self.on_result:
                                self.on_result(*rel)
            except BaseException as e:        # a replica that fails is reported by drain(), the others keep serving
                self.errors.append(e)
            with self.idle:
                self.pending -= len(batch)
                self.idle.notify_all()

    def drain(self, timeout: float = 60.0) -> List[Tuple[int, int, Any]]:
        """Waits until every submitted frame has been served; returns (stream, frame, result) in delivery order."""
        with self.idle:
            if not self.idle.wait_for(lambda: self.pending == 0, timeout=timeout):
                raise TimeoutError("replicas did not finish")
        if self.errors:
            raise self.errors[0]
        with self.out_lock:
            return list(self.delivered)

    def close(self):
        for q in self.inbox:
            q.put(None)
        for t in self.threads:
            t.join(timeout=10)


class EparaReplica:
    """A replica backend on one GPU: its own epara context (Server) with the models placed on it; run_batch turns a
    batch of frames into one serving step.  payload: dict with 'model' (index into this replica's models), 'category'
    and the keyword arguments of Server.submit (x / token, kv_len, table)."""

    def __init__(self, device: int, build_models: Callable[[Any], List[int]], workspace_bytes: int = 1 << 30, **cfg):
        import torch
        from . import server
        self.torch = torch
        self.device = device
        with torch.cuda.device(device):
            self.srv = server.Server(device=device, workspace_bytes=workspace_bytes, **cfg)
            self.models = build_models(self.srv)
        self.stream = None

    def __call__(self, batch):
        torch = self.torch
        from . import epara as E
        with torch.cuda.device(self.device):
            if self.stream is None:
                self.stream = torch.cuda.Stream(self.device)       # each replica thread launches on a stream of its own
            with torch.cuda.stream(self.stream):
                tickets = []
                for _, _, pl in batch:
                    kw = {k: v for k, v in pl.items() if k not in ("model", "category")}
                    tickets.append(self.srv.submit(self.models[pl["model"]], pl["category"], **kw))
                left = list(range(len(batch)))
                results: List[Any] = [None] * len(batch)
                while left:
                    self.srv.step()
                    self.stream.synchronize()
                    still = []
                    for i in left:
                        s, logits, am = self.srv.collect(tickets[i])
                        if s == E.PENDING:
                            still.append(i)      # beyond this step's caps: runs in the next one
                        else:
                            results[i] = (s, logits, am)
                    left = still
                return results

    def close(self):
        self.srv.close()
