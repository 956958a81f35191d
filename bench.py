"""Benchmark of the categorized serving step.

  python bench.py --gpus N --steps K --warmup W            this library on N GPUs (N > 1: under torchrun)
  python bench.py --impl reference ...                      the CPU oracle on the host cores

A step is one epara_step over one full batch of every co-resident instance of the mixed
workload (3 MLP-A, 3 ViT-S/16, 2 1B decoders; per family one latency-sensitive instance with
batch 4 and frequency-sensitive ones with batch 256): every kernel kind of the path runs in
every step.  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (read + write) per tensor-core GEMM launch of the mixed step, from one ncu pass over the GEMM
# launches of a step (65 tile-pair launches: 7.72 GB read + 3.69 GB written; 12 fused MLP-block launches:
# 2.90 GB read + 1.18 GB written; the 65 weight-streaming launches moved 2.08 GB).  Not measured by this run:
# the profile it comes from is named beside it in the JSON line.  Set to None when the GEMM kernels change.
GEMM_TC_TRAFFIC_PER_LAUNCH_MIXED = 15488294144 / 77
GEMM_TRAFFIC_SOURCE = "profiles/gemm_kernels_mixed_step_dram_traffic.md (one ncu pass, dram__bytes_read.sum + dram__bytes_write.sum)"

E2E_BUFS = 4          # device input buffers per instance in the end-to-end loop
PROFILE_EVERY = 5     # one step in five of the timed region carries per-launch events

METRIC = "mixed-category requests/s"
UNIT = "requests/s"
WORKLOAD = ("mixed co-resident step (configs[3], saturated): 3x MLP-A, 3x ViT-S/16, 2x 1B decoder; per family "
            "instance 0 latency-sensitive batch 4, others frequency-sensitive batch 256; decoder KV ~U[128,4096]")
WORKLOAD_STRESS = ("stress step (configs[4]): 8B-shaped decoder (d 4096, 32 layers, 32/8 heads, FFN 14336) decoding batch "
                   "256 with KV ~U[512,{kv_hi}], co-resident with 16x ViT-B/16 at batch 32, all frequency-sensitive")


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs: through NVML from a
    thread of this process every 20 ms (the timed region is a fraction of a second, too short for a freshly
    started nvidia-smi to deliver a sample), with nvidia-smi as the fallback.  Read-only queries."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []
        self.nvml = self.handle = None
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.stop_flag = threading.Event()

    def _nvml_open(self):
        import pynvml
        pynvml.nvmlInit()
        handle = None
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
        self.nvml, self.handle = pynvml, handle
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        m = pynvml
        self.masks = [(getattr(m, "nvmlClocksThrottleReasonHwSlowdown", 0x8), "hw_slowdown"),
                      (getattr(m, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40), "hw_thermal_slowdown"),
                      (getattr(m, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20), "sw_thermal_slowdown"),
                      (getattr(m, "nvmlClocksThrottleReasonSwPowerCap", 0x4), "sw_power_cap")]

    def _nvml_loop(self):
        m, h = self.nvml, self.handle
        while not self.stop_flag.is_set():
            try:
                self.samples.append(float(m.nvmlDeviceGetClockInfo(h, m.NVML_CLOCK_SM)))
                r = int(m.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for mask, name in self.masks:
                    if r & mask:
                        self.reasons.add(name)
            except Exception:
                pass
            self.stop_flag.wait(0.02)

    def start(self):
        try:
            self._nvml_open()
            self.th = threading.Thread(target=self._nvml_loop, daemon=True)
            self.th.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.nvml is not None:
            self.stop_flag.set()
            self.th.join(timeout=2)
            sm = sorted(self.samples)
            return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": self.max_mhz,
                    "reasons": sorted(self.reasons), "samples": len(sm), "source": "nvml"}
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], None, set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for n, v in zip(self.NAMES, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "source": "nvidia-smi"}


# ------------------------------------------------------------------------------ CPU oracle leg
class OracleSampler:
    """Times the oracle, as it stands, on bounded samples of the mixed step.  Only the configuration numbers and
    the seeded generators are imported: nothing here loads the CUDA library.  The models (MLP-A, ViT-S/16, 1B
    decoder) are generated once.  The step's decoder requests have the KV lengths of the benchmark's own
    seeded draw (4 + 256 requests, ~U[128, 4096]); decoder samples walk through them in the order shortest,
    longest, then evenly spaced ranks, so that a run of 8 or more samples spans the whole range."""

    def __init__(self, seed: int = 3):
        from paper_2511_00603_b200 import configs, synth
        self.synth, self.configs, self.seed = synth, configs, seed
        self.cores = os.cpu_count() or 1
        self.mlp = synth.bits_view(synth.make_mlp(configs.MLP_A, seed=seed))
        self.vit = synth.bits_view(synth.make_vit(seed=seed + 2, **configs.VIT_S))
        self.dec = synth.bits_view(synth.make_decoder(seed=seed + 4, **configs.DEC_1B))
        lens = []
        for k, n in ((6, configs.MIXED_LS_BATCH), (7, configs.MIXED_FS_BATCH)):      # the two decoder instances of the step
            lens += list(synth.make_decode_batch(n, configs.MIXED_KV_LO, configs.MIXED_KV_HI, configs.DEC_1B["vocab"],
                                                 seed * 1000 + k)[1])
        self.lens = sorted(int(v) for v in lens)
        n = len(self.lens)
        ranks = [0, n - 1] + [round((j + 0.5) * n / 6) for j in range(6)]
        self.len_cycle = [self.lens[min(n - 1, r)] for r in ranks]
        self.n_mlp = self.n_vit = self.n_dec = 0

    def time_mlp(self, n: int) -> float:
        from oracle import epara_oracle as O
        x = self.synth.make_mlp_inputs(n, self.configs.MLP_A[0], seed=self.seed + 1000 + self.n_mlp)
        self.n_mlp += n
        xb = [self.synth.to_bits(x[i]) for i in range(n)]
        t0 = time.perf_counter()
        for i in range(n):
            O.mlp_forward(xb[i], self.mlp["W"], self.mlp["b"])
        return time.perf_counter() - t0

    def time_vit(self, n: int) -> float:
        from oracle import epara_oracle as O
        imgs = self.synth.make_images(n, seed=self.seed + 2000 + self.n_vit)
        self.n_vit += n
        ib = [self.synth.to_bits(imgs[i]) for i in range(n)]
        t0 = time.perf_counter()
        for i in range(n):
            O.vit_forward(ib[i], self.vit)
        return time.perf_counter() - t0

    def time_decoder(self, n: int):
        """n decoder requests at the next n lengths of the cycle; returns (seconds, the lengths)."""
        from oracle import epara_oracle as O
        cfg = self.configs.DEC_1B
        total, used = 0.0, []
        for _ in range(n):
            L = self.len_cycle[self.n_dec % len(self.len_cycle)]
            toks, lens, tables, npages = self.synth.make_decode_batch(1, L, L, cfg["vocab"], seed=self.seed + 3000 + self.n_dec)
            pool = self.synth.to_bits(self.synth.make_kv_pool(cfg["n_layers"], npages, cfg["n_kv_heads"], cfg["head_dim"],
                                                              seed=self.seed + 4000 + self.n_dec))
            self.n_dec += 1
            t0 = time.perf_counter()
            O.decoder_step(int(toks[0]), L, tables[0], lambda l, pg: pool[l, pg], self.dec)
            total += time.perf_counter() - t0
            used.append(L)
        return total, used


def oracle_rps(t, counts):
    step_s = sum(counts[k] * t[k] for k in counts)
    return sum(counts.values()) / step_s, step_s


def run_reference(args):
    """The oracle on the host cores.  Each step times a bounded sample of the mixed step -- 32 MLP-A requests,
    1 ViT-S/16 image, 1 decoder request -- and the step's time is the per-family seconds per request times the
    family's request count; the decoder samples walk over the step's own KV lengths (shortest and longest
    first)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    smp = OracleSampler()
    counts = smp.configs.mixed_counts()
    acc = {"mlp": [0.0, 0], "vit": [0.0, 0], "decoder": [0.0, 0]}
    dec_lens = []
    for i in range(args.warmup + args.steps):
        t_m, t_v = smp.time_mlp(32), smp.time_vit(1)
        t_d, used = smp.time_decoder(1)
        if i >= args.warmup:
            for k, t, n in (("mlp", t_m, 32), ("vit", t_v, 1), ("decoder", t_d, 1)):
                acc[k][0] += t
                acc[k][1] += n
            dec_lens += used
    per_req = {k: acc[k][0] / max(acc[k][1], 1) for k in acc}
    rps, step_s = oracle_rps(per_req, counts)
    sample = (f"timed over {args.steps} steps: {acc['mlp'][1]} MLP-A requests, {acc['vit'][1]} ViT-S/16 images, "
              f"{acc['decoder'][1]} 1B-decoder requests at KV lengths {dec_lens} (taken from the step's own lengths: shortest, "
              f"longest, then evenly spaced ranks); a step's time = seconds per request of each family x the family's "
              f"count in the {sum(counts.values())}-request mixed step ({counts}): extrapolated, the full step was never run")
    line = {"impl": "reference", "metric": METRIC, "value": rps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD},
            "cpu_baseline": {"value": rps, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": sample,
                             "seconds_per_request": per_req},
            "e2e": {"value": rps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def cpu_baseline_leg():
    """The oracle timed beside the GPU run: every MLP-A request of a step (516), 16 ViT-S/16 images and 8 decoder
    requests (the step's shortest and longest KV length and six evenly spaced ranks)."""
    smp = OracleSampler()
    counts = smp.configs.mixed_counts()
    t_m = smp.time_mlp(counts["mlp"])
    t_v = smp.time_vit(16)
    t_d, used = smp.time_decoder(8)
    per_req = {"mlp": t_m / counts["mlp"], "vit": t_v / 16, "decoder": t_d / 8}
    rps, step_s = oracle_rps(per_req, counts)
    return {"value": rps, "unit": UNIT, "cores": smp.cores, "kind": "oracle",
            "sample": (f"timed: all {counts['mlp']} MLP-A requests of a step ({t_m:.2f} s), 16 of its {counts['vit']} ViT-S/16 "
                       f"images ({t_v:.2f} s), 8 of its {counts['decoder']} decoder requests at KV lengths {used} ({t_d:.2f} s); "
                       f"ViT and decoder families extrapolated by their counts to the {sum(counts.values())}-request step "
                       f"({step_s:.0f} s)"),
            "seconds_per_request": per_req}


# ------------------------------------------------------------------------------ GPU leg
def poisson_phase(srv, insts, E, W, torch, horizon_s=1.0, warm_s=0.1, seed=3):
    """Closed-loop replay of seeded Poisson arrivals (virtual clock advanced by measured step time)."""
    import ctypes as C
    import numpy as np
    from paper_2511_00603_b200 import synth
    fam_idx = {"mlp": 0, "vit": 0, "decoder": 0}
    arr = []
    for k, inst in enumerate(insts):
        rate = W.MIXED_RATES[inst.kind][fam_idx[inst.kind]]
        fam_idx[inst.kind] += 1
        arr.append((rate, synth.poisson_arrivals(rate, horizon_s + warm_s, seed * 10 + k)))
    ptr = [0] * len(insts)
    nsub = [0] * len(insts)
    live = {}          # ticket -> (inst index, arrival, deadline)
    ls_step_ms, ls_lat_ms, done_ls, done_fs, late_ls, dropped = [], [], 0, [0] * len(insts), 0, 0
    now = 0
    horizon_ns = int((horizon_s + warm_s) * 1e9)
    warm_ns = int(warm_s * 1e9)
    stream = torch.cuda.current_stream(srv.device)
    inp = E.Inputs()
    steps = 0
    while now < horizon_ns:
        any_q = bool(live)
        for k, inst in enumerate(insts):
            a = arr[k][1]
            while ptr[k] < len(a) and a[ptr[k]] <= now:
                t_arr = int(a[ptr[k]])
                dl = t_arr + W.LS_DEADLINE_NS if inst.category == E.CAT_LS else 0
                inst.fill(inp, nsub[k] % inst.n_req, nsub[k] % inst.n_req, deadline_ns=dl, arrival_ns=t_arr, stream=k)
                tk = srv.ctx.epara_submit(inst.mid, inst.category, inp)
                live[tk] = (k, t_arr, dl)
                ptr[k] += 1
                nsub[k] += 1
                any_q = True
        if not any_q:
            nxt = min((arr[k][1][ptr[k]] for k in range(len(insts)) if ptr[k] < len(arr[k][1])), default=horizon_ns)
            now = max(now + 1, int(nxt))
            continue
        t0 = time.perf_counter()
        info = srv.ctx.epara_step(stream.cuda_stream, now)
        stream.synchronize()
        dt_ns = int((time.perf_counter() - t0) * 1e9)
        steps += 1
        end = now + dt_ns
        had_ls = info.admitted[0] > 0
        for tk in list(live.keys()):
            s, _ = srv.ctx.epara_collect(tk)
            if s == E.PENDING:
                continue
            k, t_arr, dl = live.pop(tk)
            if t_arr < warm_ns:
                continue
            if s == E.E_TIMEOUT:
                dropped += 1
            elif insts[k].category == E.CAT_LS:
                ls_lat_ms.append((end - t_arr) / 1e6)
                if end <= dl:
                    done_ls += 1
                else:
                    late_ls += 1
            else:
                done_fs[k] += 1
        if had_ls and now >= warm_ns:
            ls_step_ms.append(dt_ns / 1e6)
        now = end
    span = horizon_s
    fs_credit = 0.0
    for k, inst in enumerate(insts):
        if inst.category == E.CAT_FS:
            achieved = done_fs[k] / span
            fs_credit += done_fs[k] * min(1.0, achieved / arr[k][0])     # frames x achieved / required rate
    q = lambda v, p: (sorted(v)[min(len(v) - 1, int(p * len(v)))] if v else None)
    return {"horizon_s": horizon_s, "steps": steps, "goodput_rps": (done_ls + fs_credit) / span,
            "ls_in_deadline": done_ls, "ls_late": late_ls, "dropped": dropped,
            "ls_step_ms_p50": q(ls_step_ms, 0.5), "ls_step_ms_p99": q(ls_step_ms, 0.99),
            "ls_latency_ms_p50": q(ls_lat_ms, 0.5), "ls_latency_ms_p99": q(ls_lat_ms, 0.99)}


def run_gpu(args):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2511_00603_b200 import build
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    from paper_2511_00603_b200 import epara as E, server, workloads as W
    peaks = read_peaks()
    dev = torch.device("cuda", local)
    stress = args.workload == "stress"
    workload, clamp = WORKLOAD, None
    if stress:
        # size the KV cache to what the device has: lower the upper length bound in steps of 512 until the
        # whole configuration (plus 6 GB of slack for the framework's context and temporaries) fits
        free, total = torch.cuda.mem_get_info(dev)
        kv_hi = W.STRESS_KV_HI
        while kv_hi > 1024 and W.stress_bytes(kv_hi)["total"] + (6 << 30) > free:
            kv_hi -= 512
        need = W.stress_bytes(kv_hi)
        if kv_hi != W.STRESS_KV_HI:
            clamp = {"kv_hi": kv_hi, "free_bytes": free, "needed_bytes_at_8192": W.stress_bytes(W.STRESS_KV_HI)["total"]}
        srv = server.Server(device=local, workspace_bytes=int(need["workspace"]))
        insts = W.build_stress(srv, seed=4, kv_hi=kv_hi)
        workload = WORKLOAD_STRESS.format(kv_hi=kv_hi)
    else:
        srv = server.Server(device=local, workspace_bytes=3 << 30)
        insts = W.build_mixed(srv, seed=3, kv_hi=args.kv_hi)
    n_req = sum(i.n_req for i in insts)
    stream = torch.cuda.current_stream(dev)

    outstanding = []

    def one_step():
        for i in insts:
            i.submit_all(srv.ctx)
            outstanding.append(list(i.tickets))
        return srv.ctx.epara_step(stream.cuda_stream, 0)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def drain():
        for tks in outstanding:
            for t in tks:
                st, _ = srv.ctx.epara_collect(t)
                if st != E.OK:
                    raise RuntimeError(f"request {t}: {E.lib.epara_strerror(st).decode()}")
        outstanding.clear()

    for _ in range(max(args.warmup, 3)):
        one_step()
        torch.cuda.synchronize()
        drain()

    check = None
    if args.check:
        # sampled parity of the resident step (a test mode: the comparison and its use of the CPU oracle live in
        # tests/stress_check.py; nothing of it runs inside the timed region)
        if not stress:
            raise SystemExit("--check goes with --workload stress (the mixed step has tests/test_gpu_step.py::"
                             "test_mixed_bench_workload_sampled_parity)")
        from tests import stress_check
        if rank == 0:
            check = stress_check.check_stress_step(insts, n_dec=8, n_img=2, log=lambda m: print(m, file=sys.stderr, flush=True))
            check["passed"] = True

    # ---- timed region: K steps, device-timed; every PROFILE_EVERY-th step (the last one among them)
    # brackets each launch with CUDA events for the per-kernel times.  The events keep a kernel from
    # starting under the tail of the one before it, so a bracketed step is some 7 % slower than a plain
    # one; sampling keeps the per-kernel times live in the timed region at a quarter of that cost. ----
    kinds = {k: [0.0, 0] for k in E.K_NAMES}
    launches = 0
    flops = wbytes = kvbytes = 0.0
    sampler = ClockSampler(local)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    infos = []
    for k in range(args.steps):
        srv.ctx.epara_set_profile((args.steps - 1 - k) % PROFILE_EVERY == 0)
        infos.append(one_step())
    ev1.record(stream)
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    drain()
    for info in infos:
        launches += info.launches
        flops += info.gemm_flops
        wbytes += info.weight_bytes
        kvbytes += info.kv_bytes
    # per-kind device time of the last timed step (every step launches the same kernels)
    prof = srv.ctx.epara_step_profile()
    srv.ctx.epara_set_profile(False)
    from paper_2511_00603_b200 import dp
    value = dp.whole_job_throughput(n_req * args.steps, ms_total, device=dev)   # all ranks' requests / slowest rank
    ms_total = world * n_req * args.steps / value * 1e3
    ms_step = ms_total / args.steps

    # ---- unprofiled repeat (shows what the event bracketing costs) ----
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        one_step()
    ev1.record(stream)
    barrier()
    ms_plain = ev0.elapsed_time(ev1) / args.steps
    drain()

    # ---- end to end: pinned host inputs -> device, step, results -> pinned host, every step ----
    h_in = [(i, i.x.cpu().pin_memory()) for i in insts if i.x is not None]
    h_out = [(i, torch.empty_like(i.logits, device="cpu").pin_memory(), torch.empty_like(i.argmax, device="cpu").pin_memory())
             for i in insts]
    h2d = sum(x.numel() * x.element_size() for _, x in h_in)
    d2h = sum(l.numel() * 2 + a.numel() * 4 for _, l, a in h_out)
    # E2E_BUFS device input buffers per instance: while step s computes, the inputs of step s + 1 travel on a
    # copy stream.  Every step still uploads all of its inputs and reads all of its results back into
    # pinned host memory; the host does not wait for a step before it submits the next one (the library
    # rotates its descriptor slots), so planning and launching overlap the previous step's kernels.
    # With only two buffers the upload for step s + 1 had to wait for step s - 1 to end, so it always started
    # at the very moment step s started and the step's small descriptor upload queued behind the images in
    # the copy engine (measured: 17.8 ms per step against 16.3 when the upload need not wait).  With four
    # buffers, and the host kept at most two steps ahead of the device, the buffer to fill was last read three
    # steps back: that step has ended, the upload starts at once, somewhere inside a step.
    for i in insts:
        i.make_bufs(E2E_BUFS)
    copy_stream = torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(E2E_BUFS)]
    ev_free = [None] * E2E_BUFS
    ev_out = [None] * E2E_BUFS
    step_done = []
    out_stream = torch.cuda.Stream(dev)

    def upload(buf):
        with torch.cuda.stream(copy_stream):
            if ev_free[buf] is not None:
                copy_stream.wait_event(ev_free[buf])      # the step that read this buffer has finished
            # in pieces of about 4 MB: a copy engine serves its queue in order, and the small descriptor
            # upload of the step that starts meanwhile must not wait behind 150 MB of images
            for i, hx in h_in:
                dst = i.x_bufs[buf]
                rows = max(1, (4 << 20) // max(1, hx[0].numel() * hx.element_size()))
                for r0 in range(0, hx.shape[0], rows):
                    dst[r0:r0 + rows].copy_(hx[r0:r0 + rows], non_blocking=True)
            ev_in[buf].record(copy_stream)

    barrier()
    t0 = time.perf_counter()
    upload(0)
    for s_i in range(args.steps):
        buf = s_i % E2E_BUFS
        if s_i >= 2:
            step_done[s_i - 2].synchronize()     # the host stays at most two steps ahead of the device
        stream.wait_event(ev_in[buf])
        if ev_out[buf] is not None:
            stream.wait_event(ev_out[buf])       # the results last written to this buffer set have been read back
        for i in insts:
            i.submit_all(srv.ctx, buf=buf)
            outstanding.append(list(i.tickets))
        srv.ctx.epara_step(stream.cuda_stream, 0)
        ev_free[buf] = torch.cuda.Event()
        ev_free[buf].record(stream)
        step_done.append(ev_free[buf])
        # (after the step is enqueued: its small descriptor upload must not queue behind the next step's
        # 150 MB of images in the host-to-device copy engine)
        if s_i + 1 < args.steps:
            upload((s_i + 1) % E2E_BUFS)
        # results of this step -> pinned host memory on a stream of its own, out of the step's own output
        # buffers (one set per input buffer), so that the next step does not wait for the read-back
        with torch.cuda.stream(out_stream):
            out_stream.wait_event(ev_free[buf])
            for i, hl, ha in h_out:
                hl.copy_(i.logits_bufs[buf], non_blocking=True)
                ha.copy_(i.argmax_bufs[buf], non_blocking=True)
            ev_out[buf] = torch.cuda.Event()
            ev_out[buf].record(out_stream)
    stream.synchronize()
    out_stream.synchronize()                # every step's results are on the host when the clock stops
    e2e_s = time.perf_counter() - t0
    drain()
    if world > 1:
        t = torch.tensor([e2e_s], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * n_req * args.steps / e2e_s

    if rank != 0:
        srv.close()
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel ----
    # The GEMM launches of a step are two kinds of work: tensor-core launches (tile pairs and one-CTA tiles),
    # judged against the tensor peak, and weight-streaming launches (groups of at most 16 rows), judged against
    # HBM.  The timed region is a fraction of a second; which bf16 peak applies depends on the clock it ran at,
    # so both fractions are given beside the sampled clock: the burst peak when the median SM clock stayed
    # within 10 % of the maximum, the sustained (power-capped) peak otherwise.
    per_step = lambda v: v / args.steps
    tc_ms, st_ms = prof["gemm"][0], prof["gemm_stream"][0]
    sflops = sum(i.stream_gemm_flops for i in infos)
    swbytes = sum(i.stream_weight_bytes for i in infos)
    near_max = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.9 * clocks["sm_max_mhz"])
    dom = max(("gemm", "attn_dec", "attn_enc", "norm"), key=lambda k: prof[k][0])
    if dom == "gemm":
        ach = per_step(flops - sflops) / (tc_ms / 1e3) / 1e12
        peak = peaks["bf16_tflops"] if near_max else peaks["bf16_tflops_sustained"]
        roof = {"kernel": "gemm_tc_pair_kernel + gemm_mlp_pair_kernel (the tensor-core GEMM launches of a step)", "bound": "tensor",
                "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                "frac_of_burst_peak": ach / peaks["bf16_tflops"], "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"],
                "sm_mhz_median": clocks.get("sm_mhz"), "launches_per_step": prof["gemm"][1], "ms_per_step": tc_ms,
                "traffic": None if (stress or GEMM_TC_TRAFFIC_PER_LAUNCH_MIXED is None) else GEMM_TC_TRAFFIC_PER_LAUNCH_MIXED,
                "traffic_source": None if stress else GEMM_TRAFFIC_SOURCE,
                "peak_source": peaks["source"] + (" (burst: median SM clock within 10 % of max)" if near_max else " (sustained)")}
    elif dom == "attn_dec":
        ach = per_step(kvbytes) / (prof["attn_dec"][0] / 1e3) / 1e9
        roof = {"kernel": "attn_decode_mma_kernel (all launches of a step)", "bound": "hbm", "achieved": ach,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": None,
                "peak_source": peaks["source"]}
    else:
        roof = {"kernel": dom, "bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": None, "traffic": None, "peak_source": peaks["source"]}
    kernels = {k: {"ms_per_step": prof[k][0], "launches_per_step": prof[k][1]} for k in prof if prof[k][1]}
    if prof["gemm"][1]:
        kernels["gemm"]["tflops"] = per_step(flops - sflops) / (tc_ms / 1e3) / 1e12
        kernels["gemm"]["frac_tensor_burst"] = kernels["gemm"]["tflops"] / peaks["bf16_tflops"]
        kernels["gemm"]["frac_tensor_sustained"] = kernels["gemm"]["tflops"] / peaks["bf16_tflops_sustained"]
    if prof["gemm_stream"][1]:
        kernels["gemm_stream"]["weight_gbs"] = per_step(swbytes) / (st_ms / 1e3) / 1e9
        kernels["gemm_stream"]["frac_hbm"] = kernels["gemm_stream"]["weight_gbs"] / peaks["hbm_gbs"]
    if prof["attn_dec"][1]:
        kernels["attn_dec"]["kv_gbs"] = per_step(kvbytes) / (prof["attn_dec"][0] / 1e3) / 1e9
        kernels["attn_dec"]["frac_hbm"] = kernels["attn_dec"]["kv_gbs"] / peaks["hbm_gbs"]

    poisson = None
    if not args.no_poisson and not stress:
        poisson = poisson_phase(srv, insts, E, W, torch)

    cpu = None
    if not args.no_cpu_baseline and not stress:
        cpu = cpu_baseline_leg()
    srv.close()
    del insts, srv
    torch.cuda.empty_cache()
    # whole steps of the single-model configurations, measured after (outside) the timed region
    cfg_steps = None
    if not args.no_config_steps and not stress:
        from paper_2511_00603_b200 import synth
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        cfg_steps = {"vit_b16": [measure_vit_step(torch, E, server, W, synth, peaks, W.VIT_B, b, 10, flush) for b in (1, 8, 64)],
                     "decoder_1b": [measure_decode_step(torch, E, server, W, synth, peaks, W.DEC_1B, b, 128, 4096, 10, flush)
                                    for b in (1, 32, 128)]}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": workload, "requests_per_step": n_req,
                       "l2": f"inputs larger than L2 ({kvbytes / args.steps / 1e9:.0f} GB of KV and {wbytes / args.steps / 1e9:.1f} GB of weights per step)",
                       "parallelism": f"replicas x{world}, no collective", "kv_clamp": clamp},
            "clocks": clocks, "gpu_launches": launches,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "roofline": roof, "cpu_baseline": cpu, "kernels": kernels, "ms_per_step_unprofiled": ms_plain,
            "ls_latency": poisson, "config_steps": cfg_steps}
    if check is not None:
        line["check"] = check
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------------------ whole steps of one model
def _timed_steps(torch, srv, inst, steps, flush):
    """Median device time of `steps` steps of one instance (L2 flushed before each), then one more step
    bracketed per launch for the per-kind split."""
    stream = torch.cuda.current_stream(srv.device)
    times, info = [], None
    for i in range(steps + 4):
        if i == steps + 3:
            srv.ctx.epara_set_profile(True)
        flush.zero_()
        inst.submit_all(srv.ctx)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        info = srv.ctx.epara_step(stream.cuda_stream, 0)
        e1.record(stream)
        torch.cuda.synchronize()
        for t in inst.tickets:
            srv.ctx.epara_collect(t)
        if 3 <= i < steps + 3:
            times.append(e0.elapsed_time(e1))
    prof = srv.ctx.epara_step_profile()
    return sorted(times)[len(times) // 2], info, {k: round(v[0], 4) for k, v in prof.items() if v[1]}


def measure_vit_step(torch, E, server, W, synth, peaks, cfgm, B, steps, flush):
    """Whole steps of one ViT at batch B (configs[1]: ViT-B/16 at batch 1 / 8 / 64, each its own step)."""
    srv = server.Server(device=torch.cuda.current_device(), workspace_bytes=2 << 30)
    inst = W.Instance(srv, synth.make_vit(seed=1, device=srv.device, **cfgm), E.CAT_FS, B, seed=11)
    ms, info, kinds = _timed_steps(torch, srv, inst, steps, flush)
    d, L, T = cfgm["d"], cfgm["n_layers"], 197
    fl = info.gemm_flops + 4.0 * T * T * d * L * B
    srv.close()
    return {"kernel": "vit step", "d": d, "B": B, "ms": ms, "launches": info.launches, "images_per_s": B / (ms / 1e3),
            "tflops_step": fl / (ms / 1e3) / 1e12, "frac_tensor_burst": fl / (ms / 1e3) / 1e12 / peaks["bf16_tflops"],
            "frac_tensor_sustained": fl / (ms / 1e3) / 1e12 / peaks["bf16_tflops_sustained"],
            "weight_gbs": info.weight_bytes / (ms / 1e3) / 1e9, "per_kind_ms": kinds}


def measure_decode_step(torch, E, server, W, synth, peaks, cfgm, B, lo, hi, steps, flush):
    """Whole decode steps of one decoder at batch B (configs[2]; the decoder of configs[4]) through the step API."""
    srv = server.Server(device=torch.cuda.current_device(), workspace_bytes=2 << 30)
    inst = W.Instance(srv, synth.make_decoder(seed=2, device=srv.device, **cfgm), E.CAT_FS, B, seed=21, kv_lo=lo, kv_hi=hi)
    ms, info, kinds = _timed_steps(torch, srv, inst, steps, flush)
    byt = info.weight_bytes + info.kv_bytes
    srv.close()
    return {"kernel": "decode step", "d": cfgm["d"], "B": B, "ms": ms, "launches": info.launches,
            "weight_gb": info.weight_bytes / 1e9, "kv_gb": info.kv_bytes / 1e9, "hbm_gbs": byt / (ms / 1e3) / 1e9,
            "frac_hbm": byt / (ms / 1e3) / 1e9 / peaks["hbm_gbs"], "tokens_per_s": B / (ms / 1e3), "per_kind_ms": kinds}


def measure_prefill_step(torch, E, server, synth, peaks, cfgm, n_prompts, n_tok, steps, flush):
    """Whole prefill steps of one decoder: n_prompts prompts of n_tok tokens each on an empty cache, one step
    (the prompts' chunks are the step's rows; every layer's GEMMs see n_prompts * n_tok rows).  Work counted:
    the step's GEMM flops as the library reports them plus the causal attention's 4 * hd * Hq * n (n + 1) / 2
    per prompt and layer."""
    import numpy as np
    dev = torch.device("cuda", torch.cuda.current_device())
    srv = server.Server(device=dev.index, workspace_bytes=6 << 30)
    p = synth.make_decoder(seed=2, device=dev, **cfgm)
    pages_per = (n_tok + 15) // 16
    pool = synth.make_kv_pool(cfgm["n_layers"], n_prompts * pages_per + 2, cfgm["n_kv_heads"], cfgm["head_dim"], seed=5, device=dev)
    m = srv.add_model(p, kv_pool=pool, max_kv_len=n_tok, max_batch=n_prompts * n_tok)
    rng = np.random.default_rng(7)
    prompts = [[int(t) for t in rng.integers(0, cfgm["vocab"], n_tok)] for _ in range(n_prompts)]
    perm = rng.permutation(n_prompts * pages_per).astype(np.int32)
    tables = [torch.as_tensor(perm[i * pages_per:(i + 1) * pages_per], device=dev) for i in range(n_prompts)]
    stream = torch.cuda.current_stream(dev)
    times, info = [], None
    for i in range(steps + 4):
        if i == steps + 3:
            srv.ctx.epara_set_profile(True)
        flush.zero_()
        ts = [srv.submit(m, E.CAT_FS, tokens=prompts[k], kv_len=0, table=tables[k]) for k in range(n_prompts)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        info = srv.step()
        e1.record(stream)
        torch.cuda.synchronize()
        for t in ts:
            st = srv.collect(t)[0]
            if st != E.OK:
                raise RuntimeError(f"prefill request: status {st}")
        if 3 <= i < steps + 3:
            times.append(e0.elapsed_time(e1))
    prof = srv.ctx.epara_step_profile()
    kinds = {k: round(v[0], 4) for k, v in prof.items() if v[1]}
    ms = sorted(times)[len(times) // 2]
    attn = 4.0 * cfgm["head_dim"] * cfgm["n_q_heads"] * n_tok * (n_tok + 1) / 2 * cfgm["n_layers"] * n_prompts
    fl = info.gemm_flops + attn
    gemm_ms = kinds.get("gemm", 0.0) + kinds.get("gemm_stream", 0.0)
    srv.close()
    return {"kernel": "prefill step", "d": cfgm["d"], "prompts": n_prompts, "tokens_per_prompt": n_tok, "ms": ms,
            "launches": info.launches, "prefill_tokens": info.prefill_tokens, "tokens_per_s": n_prompts * n_tok / (ms / 1e3),
            "tflops_step": fl / (ms / 1e3) / 1e12, "frac_tensor_burst": fl / (ms / 1e3) / 1e12 / peaks["bf16_tflops"],
            "frac_tensor_sustained": fl / (ms / 1e3) / 1e12 / peaks["bf16_tflops_sustained"],
            "gemm_tflops": (info.gemm_flops / (gemm_ms / 1e3) / 1e12) if gemm_ms else None,
            "gemm_frac_tensor_burst": (info.gemm_flops / (gemm_ms / 1e3) / 1e12 / peaks["bf16_tflops"]) if gemm_ms else None,
            "attn_prefill_tflops": (attn / (kinds["attn_prefill"] / 1e3) / 1e12) if kinds.get("attn_prefill") else None,
            "per_kind_ms": kinds}


# ------------------------------------------------------------------------------ single-kernel timings
MICRO_GEMM = {
    "vit_s": [(50432, 1152, 384, "bias"), (50432, 384, 384, "bias,resid"), (50432, 1536, 384, "bias,gelu"),
              (50432, 384, 1536, "bias,resid")],
    "vit_b": [(12608, 2304, 768, "bias"), (12608, 768, 768, "bias,resid"), (12608, 3072, 768, "bias,gelu"),
              (12608, 768, 3072, "bias,resid")],
    "dec_1b": [(128, 3072, 2048, ""), (128, 2048, 2048, "resid"), (128, 16384, 2048, "swiglu"), (128, 2048, 8192, "resid"),
               (128, 32000, 2048, "")],
    "dec_8b": [(256, 6144, 4096, ""), (256, 4096, 4096, "resid"), (256, 28672, 4096, "swiglu"), (256, 4096, 14336, "resid"),
               (256, 32000, 4096, "")],
    "square": [(8192, 8192, 8192, "")],
}


def run_micro(args):
    """Times one kernel through its C-ABI entry point on seeded inputs; one JSON line per case."""
    import torch
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara as E, synth
    peaks = read_peaks()
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    g = torch.Generator(device=dev).manual_seed(0)

    def timed(fn, reps):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        for a, b in ev:
            flush.zero_()                      # L2 flush between timed launches
            a.record(stream)
            fn()
            b.record(stream)
        torch.cuda.synchronize()
        ms = sorted(a.elapsed_time(b) for a, b in ev)
        return ms[len(ms) // 2]

    if args.micro == "gemm":
        for (M, N, K, fl) in MICRO_GEMM[args.case]:
            if args.m:
                M = args.m
            fl = set(x for x in fl.split(",") if x)
            A = torch.randn((M, K), generator=g, device=dev).to(torch.bfloat16)
            Wt = (torch.randn((N, K), generator=g, device=dev) * 0.02).to(torch.bfloat16)
            bias = torch.zeros(N, device=dev, dtype=torch.bfloat16) if "bias" in fl else None
            epi = (E.EPI_BIAS if "bias" in fl else 0) | (E.EPI_GELU if "gelu" in fl else 0) | \
                  (E.EPI_SWIGLU if "swiglu" in fl else 0) | (E.EPI_RESID_F32 if "resid" in fl else 0)
            ncol = N // 2 if "swiglu" in fl else N
            Cc = torch.zeros((M, ncol), device=dev, dtype=torch.float32 if "resid" in fl else torch.bfloat16)
            prob = [{"A": A, "W": Wt, "C": Cc, "bias": bias, "M": M, "N": N, "K": K, "epilogue": epi}]
            scratch = torch.empty(E.epara_gemm_scratch_bytes_for(prob), dtype=torch.uint8, device=dev)
            ms = timed(lambda: E.epara_grouped_gemm(prob, stream.cuda_stream, scratch), args.steps)
            tf = 2.0 * M * N * K / (ms / 1e3) / 1e12
            gbs = 2.0 * N * K / (ms / 1e3) / 1e9
            print(json.dumps({"kernel": "gemm_tc", "M": M, "N": N, "K": K, "epilogue": sorted(fl), "ms": ms, "tflops": tf,
                              "frac_tensor_burst": tf / peaks["bf16_tflops"], "weight_gbs": gbs,
                              "frac_hbm_weights": gbs / peaks["hbm_gbs"]}))
    elif args.micro == "attn_dec":
        import numpy as np
        Hq, Hkv, hd = (32, 8, 128) if args.case == "dec_8b" else (32, 8, 64)
        B = args.m or 128
        hi = 8192 if args.case == "dec_8b" else 4096
        toks, lens, tables, npages = synth.make_decode_batch(B, 128, hi, 32000, seed=2)
        lens = lens + 1
        stride = max(len(t) for t in tables)
        tb = np.zeros((B, stride), dtype=np.int32)
        for b, t in enumerate(tables):
            tb[b, :len(t)] = t
        pool = synth.make_kv_pool(1, npages, Hkv, hd, seed=3, device=dev)[0]
        q = torch.randn((B, Hq * hd), generator=g, device=dev).to(torch.bfloat16)
        out = torch.empty_like(q)
        max_len = int(lens.max())
        scratch = torch.empty(E.lib.epara_decode_attention_scratch_bytes(B, Hq, hd, max_len), dtype=torch.uint8, device=dev)
        lens_d, tb_d = torch.as_tensor(lens, device=dev), torch.as_tensor(tb, device=dev)
        ms = timed(lambda: E.epara_decode_attention(q, pool, lens_d, tb_d, out, Hq, Hkv, hd, max_len, scratch,
                                                    stream.cuda_stream), args.steps)
        kvb = float(lens.sum()) * 2 * Hkv * hd * 2
        print(json.dumps({"kernel": "attn_decode+combine", "B": B, "Hq": Hq, "Hkv": Hkv, "hd": hd, "tokens": int(lens.sum()),
                          "ms": ms, "kv_gbs": kvb / (ms / 1e3) / 1e9, "frac_hbm": kvb / (ms / 1e3) / 1e9 / peaks["hbm_gbs"]}))
    elif args.micro == "vit_step":
        from paper_2511_00603_b200 import server, workloads as W
        print(json.dumps(measure_vit_step(torch, E, server, W, synth, peaks, W.VIT_S if args.case == "vit_s" else W.VIT_B,
                                          args.m or 64, args.steps, flush)))
    elif args.micro == "prefill_step":
        from paper_2511_00603_b200 import server, configs
        big = args.case == "dec_8b"
        n_prompts, n_tok = (args.m or 4), args.tokens
        print(json.dumps(measure_prefill_step(torch, E, server, synth, peaks, configs.DEC_8B if big else configs.DEC_1B,
                                              n_prompts, n_tok, args.steps, flush)))
    elif args.micro == "decode_step":
        from paper_2511_00603_b200 import server, workloads as W
        big = args.case == "dec_8b"
        print(json.dumps(measure_decode_step(torch, E, server, W, synth, peaks, W.DEC_8B if big else W.DEC_1B, args.m or 128,
                                             512 if big else 128, 8192 if big else 4096, args.steps, flush)))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--micro", default=None, choices=["gemm", "attn_dec", "decode_step", "vit_step", "prefill_step"], help="time one kernel instead of the step")
    ap.add_argument("--case", default="vit_s")
    ap.add_argument("--m", type=int, default=0, help="override M (gemm) or B (attn_dec) of the micro case")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="epara", choices=["epara", "reference"])
    ap.add_argument("--workload", default="mixed", choices=["mixed", "stress"],
                    help="mixed: the co-resident step the metric is quoted on; stress: 8B decoder batch 256 + 16 ViT-B")
    ap.add_argument("--kv-hi", type=int, default=4096,
                    help="mixed workload: upper bound of the decoders' KV lengths (a short cache keeps a profiler capture small; "
                         "the GEMM launches do not depend on it)")
    ap.add_argument("--tokens", type=int, default=2048, help="prefill_step micro: tokens per prompt (--m prompts per step)")
    ap.add_argument("--check", action="store_true",
                    help="stress workload only: compare 8 decode requests and 2 images of the resident step with the "
                         "CPU oracle before timing (about a quarter of an hour)")
    ap.add_argument("--no-poisson", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-config-steps", action="store_true",
                    help="skip the whole-step timings of ViT-B/16 (batch 1/8/64) and the 1B decoder (batch 1/32/128)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.micro:
        return run_micro(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
