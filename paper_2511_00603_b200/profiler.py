"""Offline profiler for the allocator (paper Section 4.1, "Adaptive Deployment").

The paper's allocator profiles every service offline: first the batch size BS over 2^0 .. 2^9, then, with the
memory partition fixed, the replication degree of co-resident slices MT over 2^0 .. 2^4; the measured compute
time per service is the c_ln that the placement scheduler (Section 3.3) and the simulator (Section 5.2) look up.
Here a "slice" is a co-resident instance of the service inside one serving step: MT = k places k instances
(shared weights, own activations and KV cache) and runs them in the same grouped launches.

sweep() drives any `measure(service, bs, mt) -> milliseconds per step or None` callable, so the selection logic
is testable without a GPU; GpuMeasure is the callable that times real steps through the C-ABI library.
The table it returns (and writes as JSON) is

  {"services": {name: {"bs": [...], "mt": [...],
                       "step_ms": {"<bs>": ms, ...}                  # MT = 1
                       "c_ln_ms": {"<bs>": ms per request, ...},     # = step_ms / bs
                       "mt_step_ms": {"<mt>": ms, ...},              # at the chosen BS
                       "best_bs": b, "best_mt": k, "requests_per_s": r}}}
"""
from __future__ import annotations

import json
from typing import Callable, Dict, List, Optional, Sequence

BS_RANGE = [1 << i for i in range(10)]      # 2^0 .. 2^9
MT_RANGE = [1 << i for i in range(5)]       # 2^0 .. 2^4


def choose_bs(step_ms: Dict[int, float], latency_slo_ms: Optional[float]) -> int:
    """The batch size with the highest throughput bs / step_ms among those whose step meets the latency SLO
    (all of them when there is none); ties go to the smaller batch, and if none meets the SLO the smallest
    measured batch is returned."""
    ok = [b for b in sorted(step_ms) if step_ms[b] is not None and (latency_slo_ms is None or step_ms[b] <= latency_slo_ms)]
    if not ok:
        measured = [b for b in sorted(step_ms) if step_ms[b] is not None]
        return measured[0] if measured else 1
    best = ok[0]
    for b in ok[1:]:
        if b / step_ms[b] > best / step_ms[best] * (1 + 1e-9):
            best = b
    return best


def choose_mt(mt_step_ms: Dict[int, float], bs: int, latency_slo_ms: Optional[float]) -> int:
    """The replication degree with the highest throughput mt * bs / step_ms under the same SLO rule."""
    ok = [k for k in sorted(mt_step_ms) if mt_step_ms[k] is not None and (latency_slo_ms is None or mt_step_ms[k] <= latency_slo_ms)]
    if not ok:
        return 1
    best = ok[0]
    for k in ok[1:]:
        if k * bs / mt_step_ms[k] > best * bs / mt_step_ms[best] * (1 + 1e-9):
            best = k
    return best


def sweep(services: Sequence[str], measure: Callable[[str, int, int], Optional[float]],
          latency_slo_ms: Optional[Dict[str, Optional[float]]] = None, bs_range: Sequence[int] = BS_RANGE,
          mt_range: Sequence[int] = MT_RANGE) -> Dict:
    """BS sweep at MT = 1, then MT sweep at the chosen BS (the order of Section 4.1).  measure() returns None for a
    point that cannot run (out of memory, beyond the model's limits); such points are recorded as null and never chosen."""
    out: Dict = {"services": {}}
    for name in services:
        slo = (latency_slo_ms or {}).get(name)
        step_ms = {b: measure(name, b, 1) for b in bs_range}
        bs = choose_bs(step_ms, slo)
        mt_ms = {k: (step_ms[bs] if k == 1 else measure(name, bs, k)) for k in mt_range}
        mt = choose_mt(mt_ms, bs, slo)
        rps = mt * bs / mt_ms[mt] * 1e3 if mt_ms.get(mt) else None
        out["services"][name] = {
            "bs": list(bs_range), "mt": list(mt_range),
            "step_ms": {str(b): step_ms[b] for b in bs_range},
            "c_ln_ms": {str(b): (step_ms[b] / b if step_ms[b] is not None else None) for b in bs_range},
            "mt_step_ms": {str(k): mt_ms[k] for k in mt_range},
            "best_bs": bs, "best_mt": mt, "latency_slo_ms": slo, "requests_per_s": rps}
    return out


def write_table(table: Dict, path: str) -> None:
    with open(path, "w") as f:
        json.dump(table, f, indent=1, sort_keys=True)


def compute_ms(table: Dict, service: str, batch: int) -> float:
    """c_ln lookup for the simulator: step time of `batch` requests of the service, taken from the smallest
    profiled batch size that holds them (the step runs padded to nothing, but the table is in powers of two)."""
    t = table["services"][service]["step_ms"]
    sizes = sorted(int(b) for b in t if t[b] is not None)
    for b in sizes:
        if b >= batch:
            return float(t[str(b)])
    return float(t[str(sizes[-1])]) * batch / sizes[-1]


def service_from_table(table: Dict, name: str, cat: int, slo_ms: float, a: float, b: float, n_gpus: int = 1, fps: float = 0.0,
                       frames: int = 0) -> Dict:
    """A service description for epara_simulate / epara_place_sssp whose compute times are the profiled ones:
    c_ms[k] = step time at batch 2^k (points the sweep could not run take the last measured time scaled by the
    batch), batch size = the profile's choice."""
    t = table["services"][name]
    c_ms = [compute_ms(table, name, 1 << k) for k in range(10)]
    return {"a": a, "b": b, "n_gpus": n_gpus, "cat": cat, "bs": int(t["best_bs"]), "slo_ms": slo_ms, "fps": fps,
            "frames": frames, "c_ms": c_ms}


class GpuMeasure:
    """measure(service, bs, mt) on the real kernels: places `mt` instances of the service for batch `bs` on one GPU,
    runs `steps` saturated steps after `warmup`, L2 flushed before each, and returns the median device time of a step.
    services: name -> synth model (tensors on the device).  Decoder instances get their own KV cache with lengths
    ~U[kv_lo, kv_hi].  A point whose memory need exceeds what the device has free returns None."""

    def __init__(self, services: Dict[str, Dict], device: int = 0, steps: int = 5, warmup: int = 2, kv_lo: int = 128,
                 kv_hi: int = 1024, slack_bytes: int = 4 << 30):
        import torch
        from . import epara as E, server, workloads as W
        self.torch, self.E, self.server, self.W = torch, E, server, W
        self.services, self.device, self.steps, self.warmup = services, device, steps, warmup
        self.kv_lo, self.kv_hi, self.slack = kv_lo, kv_hi, slack_bytes
        from . import synth
        for p in services.values():
            if p["kind"] == "decoder" and "packed_layers" not in p:
                p["packed_layers"] = [synth.pack_decoder_layer(L) for L in p["layers"]]
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=torch.device("cuda", device))

    def _need_bytes(self, p: Dict, bs: int, mt: int) -> int:
        cfg = self.E.Config(self.device, 256, 1 << 40, 0, 0, 0, self.E.GEMM_TCGEN05, 0, 0)
        desc, _keep = self.E.make_model_desc(p, kv_pool=self._fake_pool(p), max_kv_len=self.kv_hi, max_batch=bs)
        ws = self.E.lib.epara_model_workspace_bytes(self.E.C.byref(cfg), self.E.C.byref(desc))
        kv = 0
        if p["kind"] == "decoder":
            kv = bs * (self.kv_hi + 32) * 2 * p["n_kv_heads"] * p["head_dim"] * 2 * p["n_layers"]
        inputs = bs * 3 * p["img"] * p["img"] * 2 if p["kind"] == "vit" else 0
        return mt * (ws + kv + inputs) + (64 << 20)

    def _fake_pool(self, p: Dict):
        if p["kind"] != "decoder":
            return None
        return self.torch.empty((p["n_layers"], 1, 2, p["n_kv_heads"], 16, p["head_dim"]), dtype=self.torch.bfloat16,
                                device=self.torch.device("cuda", self.device))

    def __call__(self, name: str, bs: int, mt: int) -> Optional[float]:
        torch, E, W = self.torch, self.E, self.W
        p = self.services[name]
        dev = torch.device("cuda", self.device)
        need = self._need_bytes(p, bs, mt)
        free, _total = torch.cuda.mem_get_info(dev)
        if need + self.slack > free:
            return None
        srv = self.server.Server(device=self.device, workspace_bytes=need, cap_fs=bs)
        try:
            insts = [W.Instance(srv, p, E.CAT_FS, bs, seed=7000 + 17 * k, kv_lo=self.kv_lo, kv_hi=self.kv_hi, max_batch=bs)
                     for k in range(mt)]
            stream = torch.cuda.current_stream(dev)
            times: List[float] = []
            for i in range(self.warmup + self.steps):
                self.flush.zero_()
                for inst in insts:
                    inst.submit_all(srv.ctx)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                info = srv.ctx.epara_step(stream.cuda_stream, 0)
                e1.record(stream)
                torch.cuda.synchronize()
                assert info.admitted[1] == bs * mt
                for inst in insts:
                    for t in inst.tickets:
                        st, _ = srv.ctx.epara_collect(t)
                        assert st == E.OK
                if i >= self.warmup:
                    times.append(e0.elapsed_time(e1))
            return sorted(times)[len(times) // 2]
        finally:
            srv.close()
            del srv
            torch.cuda.empty_cache()
