"""GPU parity at the workload configurations' own sizes: ViT-B/16 at batch 1 / 8 / 64, the 1B decoder at
batch 1 / 32 / 128 with the model placed for exactly that batch (so that every GEMM kernel the batch
sizes select runs inside a checked step), a cut of the stress step (the 8B decoder at full depth placed
for batch 256, co-resident with ViT-B), and a step with multi-frame admission."""
import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import configs, synth
from tests.parity import assert_close, assert_parity, check_argmax, to_f64
from tests.test_gpu_step import _decoder_case, _finish, replay_layers

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def mods():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara, server
    return epara, server


@pytest.fixture(scope="module")
def vit_b():
    return synth.make_vit(seed=1, device=DEV, **configs.VIT_B)


@pytest.fixture(scope="module")
def dec_1b():
    return synth.make_decoder(seed=2, device=DEV, **configs.DEC_1B)


@pytest.mark.parametrize("batch", [1, 8, 64])
def test_config2_vit_b16_at_its_batch_sizes(mods, vit_b, batch):
    """ViT-B/16 as its own frequency-sensitive step at batch 1, 8 and 64, placed for that batch.  All images at
    batch 1 and 8; at 64 the first, the last and two in between.  Every image's argmax agrees with its logits."""
    E, server = mods
    srv = server.Server(workspace_bytes=2 << 30)
    imgs = synth.make_images(batch, seed=100 + batch, device=DEV)
    m = srv.add_model(vit_b, max_batch=batch)
    ts = [srv.submit(m, E.CAT_FS, x=imgs[i]) for i in range(batch)]
    info = srv.step()
    assert info.admitted[1] == batch
    res = _finish(srv, E, ts)
    v = synth.bits_view(vit_b)
    sample = range(batch) if batch <= 8 else [0, 21, 42, batch - 1]
    worst = 0.0
    for i in sample:
        ref, _, _ = O.vit_forward(synth.to_bits(imgs[i]), v)
        worst = max(worst, assert_close(res[i][0], ref, what=f"ViT-B batch {batch} image {i}"))
        check_argmax(res[i][1], res[i][0], ref)
    for logits, am in res:
        assert torch.isfinite(logits.float()).all() and am == int(logits.float().argmax())
    print(f"ViT-B batch {batch}: worst max relative error vs the fp64 oracle {worst:.3e}")
    srv.close()


@pytest.mark.parametrize("batch", [1, 32, 128])
def test_config3_decoder_1b_at_its_batch_sizes(mods, dec_1b, batch):
    """The 1B decoder (16 layers) decoding batch 1, 32 and 128 with KV ~U[128, 4096], max_batch equal to the
    batch: batch 1 runs the weight-streaming GEMM, 32 and 128 the GEMM kernels for 17 to 128 rows.  Checked
    requests: the shortest and the longest cache and one in between."""
    E, server = mods
    _, lens, _, _ = synth.make_decode_batch(batch, 128, 4096, dec_1b["vocab"], seed=300 + batch)
    order = np.argsort(lens, kind="stable")
    check = sorted({int(order[0]), int(order[len(order) // 2]), int(order[-1])})
    info, decided, errs = _decoder_case(E, server, dec_1b, B=batch, lo=128, hi=4096, seed=300 + batch, deep=True,
                                        max_batch=batch, check=check)
    assert info.admitted[1] == batch


def test_config5_stress_cut_full_depth(mods):
    """A cut of the stress step: the 8B-shaped decoder at its full 32 layers, placed for batch 256 (the kernels
    the stress step runs) and decoding 6 sequences with KV ~U[512, 8192], co-resident with one ViT-B/16 instance
    at batch 2, in one step.  Compared with the oracle: the shortest and the longest sequence and one image."""
    E, server = mods
    cfg = configs.DEC_8B
    p = synth.make_decoder(seed=400, device=DEV, **cfg)
    p["packed_layers"] = [synth.pack_decoder_layer(L) for L in p["layers"]]
    pv = synth.make_vit(seed=401, device=DEV, **configs.VIT_B)
    B = 6
    toks, lens, tables, npages = synth.make_decode_batch(B, 512, 8192, cfg["vocab"], seed=402)
    pool = synth.make_kv_pool_replicated(cfg["n_layers"], npages, cfg["n_kv_heads"], cfg["head_dim"], seed=403, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=3 << 30)
    trace = torch.zeros((cfg["n_layers"] + 1, 256, cfg["d"]), dtype=torch.float32, device=DEV)
    md = srv.add_model(p, kv_pool=pool, max_kv_len=8192, max_batch=256, trace=trace)
    mv = srv.add_model(pv, max_batch=32)
    imgs = synth.make_images(2, seed=404, device=DEV)
    tabs = [torch.as_tensor(t, device=DEV) for t in tables]
    td = [srv.submit(md, E.CAT_FS, token=int(toks[i]), kv_len=int(lens[i]), table=tabs[i]) for i in range(B)]
    tv = [srv.submit(mv, E.CAT_FS, x=imgs[i]) for i in range(2)]
    srv.step()
    rd, rv = _finish(srv, E, td), _finish(srv, E, tv)
    v = synth.bits_view({k: p[k] for k in p if k != "packed_layers"})
    fetch = lambda l, pg: synth.to_bits(pool0[l, pg])
    for i in sorted({int(np.argmin(lens)), int(np.argmax(lens))}):
        ra = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], fetch, v)
        rb = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], fetch, v, round_bf16=True)
        what = f"8B decoder request {i} (L={lens[i]})"
        assert_parity(rd[i][0], ra["logits"], rb["logits"], what=what, deep=True)
        check_argmax(rd[i][1], rd[i][0], rb["logits"])
        # strict tolerance layer by layer, each layer of the oracle fed the device's own input
        worst, head = replay_layers(v, trace, i, int(toks[i]), int(lens[i]), tables[i], fetch, pool, what)
        worst = max(worst, assert_close(rd[i][0], head, what=f"{what}: logits from the device's last residual"))
        print(f"{what}: layer-by-layer worst max relative error {worst:.3e}")
    ref, _, _ = O.vit_forward(synth.to_bits(imgs[1]), synth.bits_view(pv))
    assert_close(rv[1][0], ref, what="co-resident ViT-B image 1")
    check_argmax(rv[1][1], rv[1][0], ref)
    srv.close()


def test_step_with_multi_frame_admission(mods):
    """MF inside a step (mf_max = 3, frequency-sensitive cap 8): floor(8 / 3) = 2 streams are served, each
    with the same number of frames; the frames that ran equal the oracle, the rest stay queued and run in
    later steps."""
    E, server = mods
    srv = server.Server(workspace_bytes=64 << 20, cap_fs=8, mf_max=3)
    p = synth.make_mlp([64, 128, 16], seed=500, device=DEV, std=0.1, perturb=0.2)
    x = synth.make_mlp_inputs(12, 64, seed=501, device=DEV)
    m = srv.add_model(p)
    streams = [0, 1, 0, 2, 1, 0, 0, 2, 1, 1, 2, 0]              # arrival order; stream 0 has 5 frames, 1 has 4, 2 has 3
    ts = [srv.submit(m, E.CAT_FS, x=x[i], stream=streams[i]) for i in range(12)]
    queue = [{"ticket": ts[i], "deadline_ns": 0, "stream": streams[i]} for i in range(12)]
    exp, _ = O.admit(queue, 0, 8, 3)
    assert len(exp) == 6                                       # streams 0 and 1, three frames each
    info = srv.step(now_ns=0)
    assert info.admitted[1] == 6
    torch.cuda.synchronize()
    v = synth.bits_view(p)
    for i, t in enumerate(ts):
        s, logits, am = srv.collect(t)
        if t in exp:
            assert s == E.OK
            assert_close(logits, O.mlp_forward(synth.to_bits(x[i]), v["W"], v["b"])[0], what=f"frame {i}")
        else:
            assert s == E.PENDING
    left = [q for q in queue if q["ticket"] not in exp]
    exp2, _ = O.admit(left, 0, 8, 3)
    info = srv.step(now_ns=0)
    assert info.admitted[1] == len(exp2)
    torch.cuda.synchronize()
    for t in exp2:
        assert srv.collect(t)[0] == E.OK
    srv.close()
