"""Request-level data parallelism across GPUs (the paper's DP operator, Section 3.1): the full
model set is replicated, requests are dealt round-robin over the replicas, and nothing is
exchanged between them.  Only bookkeeping lives here: which replica serves which request, how
many replicas a frame-rate requirement needs (Eq. 4), and the max-over-ranks timing used to report
whole-job throughput."""
from __future__ import annotations

import math
from typing import List, Sequence

import torch
import torch.distributed as dist


def dp_group_count(required_fps: float, group_fps: float) -> int:
    """Eq. 4: ceil(frame-rate requirement / frame rate of one DP group)."""
    return int(math.ceil(required_fps / group_fps))


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
    if not (dist.is_available() and dist.is_initialized()):
        return local_units / (local_ms / 1e3)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    n = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(n.item()) / (float(t.item()) / 1e3)
