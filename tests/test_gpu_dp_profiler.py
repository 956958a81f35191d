"""GPU tests of the replica driver (two epara contexts, one host thread each; both on cuda:0 here, since one
GPU is what a test run has: replicas never wait for one another, so sharing a device only makes them slower)
and of the allocator's offline profiler on the real kernels."""
import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import synth
from tests.parity import assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def E():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara
    return epara


def test_two_replicas_serve_streams_in_frame_order(E):
    from paper_2511_00603_b200 import dp
    pm = synth.make_mlp([64, 128, 16], seed=700, device=DEV, std=0.1, perturb=0.2)
    pv = synth.make_vit(d=128, n_layers=1, n_heads=2, mlp=256, n_cls=10, seed=701, device=DEV, img=32, std=0.1)

    def build_models(srv):
        return [srv.add_model(pm, max_batch=8), srv.add_model(pv, max_batch=4)]

    reps = [dp.EparaReplica(0, build_models, workspace_bytes=128 << 20, cap_fs=8) for _ in range(2)]
    drv = dp.ReplicaDriver(reps, max_batch=8)
    xs = synth.make_mlp_inputs(24, 64, seed=702, device=DEV)
    imgs = synth.make_images(6, seed=703, device=DEV, img=32)
    for f in range(12):
        for s in (0, 1):                                   # two MLP streams, frames alternate between the replicas
            drv.submit(s, f, {"model": 0, "category": E.CAT_FS, "x": xs[s * 12 + f]})
    for f in range(6):                                     # one ViT stream
        drv.submit(2, f, {"model": 1, "category": E.CAT_FS, "x": imgs[f]})
    got = drv.drain(timeout=120)
    drv.close()
    vm, vv = synth.bits_view(pm), synth.bits_view(pv)
    seen = {0: [], 1: [], 2: []}
    for s, f, (status, logits, am) in got:
        assert status == E.OK
        seen[s].append(f)
        if s < 2:
            ref = O.mlp_forward(synth.to_bits(xs[s * 12 + f]), vm["W"], vm["b"])[0]
        else:
            ref = O.vit_forward(synth.to_bits(imgs[f]), vv)[0]
        assert_close(logits, ref, what=f"stream {s} frame {f}")
    assert seen[0] == list(range(12)) and seen[1] == list(range(12)) and seen[2] == list(range(6))
    for r in reps:
        r.close()


def test_profiler_sweeps_bs_and_mt_on_the_real_kernels(E, tmp_path):
    from paper_2511_00603_b200 import profiler
    services = {"mlp": synth.make_mlp([256, 512, 16], seed=710, device=DEV, std=0.1),
                "vit": synth.make_vit(d=128, n_layers=2, n_heads=2, mlp=256, n_cls=10, seed=711, device=DEV, img=64, std=0.1),
                "dec": synth.make_decoder(d=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=1000,
                                          seed=712, device=DEV, std=0.05)}
    measure = profiler.GpuMeasure(services, steps=3, warmup=1, kv_lo=16, kv_hi=200)
    table = profiler.sweep(list(services), measure, latency_slo_ms={"mlp": None, "vit": None, "dec": 50.0},
                           bs_range=[1, 2, 4, 8, 16], mt_range=[1, 2, 4])
    path = tmp_path / "c_ln.json"
    profiler.write_table(table, str(path))
    import json
    back = json.load(open(path))
    for name in services:
        t = back["services"][name]
        assert set(t["step_ms"]) == {"1", "2", "4", "8", "16"} and all(v is not None and v > 0 for v in t["step_ms"].values())
        assert t["best_bs"] in (1, 2, 4, 8, 16) and t["best_mt"] in (1, 2, 4)
        # batching pays on a GPU: a request costs less in a batch of 16 than alone (the paper's motivation for BS)
        assert t["c_ln_ms"]["16"] < t["c_ln_ms"]["1"]
        assert profiler.compute_ms(back, name, 3) == t["step_ms"]["4"]
        assert t["requests_per_s"] > 0
