"""GPU parity of whole serving steps (epara_register_model / submit / step / collect) against the
fp64 oracle, request by request, on the synthetic configurations."""
import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import synth
from tests.parity import assert_close, assert_parity, check_argmax, max_rel_err, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def mods():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara, server
    return epara, server


def _finish(srv, E, tickets):
    torch.cuda.synchronize()
    res = []
    for t in tickets:
        s, logits, am = srv.collect(t)
        assert s == E.OK, E.lib.epara_strerror(s)
        res.append((logits, int(am.item())))
    return res


@pytest.mark.parametrize("impl", ["simt", "tcgen05"])
def test_config1_two_mlps_one_step(mods, impl):
    """MLP-A 512->512->512->512->10 batch 8 (latency-sensitive) and MLP-B 256->1024->256 batch 32
    (frequency-sensitive) in ONE step, seed 0."""
    E, server = mods
    srv = server.Server(workspace_bytes=64 << 20, gemm_impl=E.GEMM_SIMT if impl == "simt" else E.GEMM_TCGEN05)
    pa = synth.make_mlp([512, 512, 512, 512, 10], seed=0, device=DEV)
    pb = synth.make_mlp([256, 1024, 256], seed=1, device=DEV)
    xa = synth.make_mlp_inputs(8, 512, seed=2, device=DEV)
    xb = synth.make_mlp_inputs(32, 256, seed=3, device=DEV)
    ma, mb = srv.add_model(pa), srv.add_model(pb)
    ta = [srv.submit(ma, E.CAT_LS, x=xa[i]) for i in range(4)]
    ta += [srv.submit(ma, E.CAT_FS, x=xa[i]) for i in range(4, 8)]   # one group may mix both categories
    tb = [srv.submit(mb, E.CAT_FS, x=xb[i]) for i in range(32)]
    info = srv.step()
    assert info.admitted[0] == 4 and info.admitted[1] == 36 and info.gemm_groups == 6
    ra, rb = _finish(srv, E, ta), _finish(srv, E, tb)
    va, vb = synth.bits_view(pa), synth.bits_view(pb)
    for i, (logits, am) in enumerate(ra):
        ref, ram = O.mlp_forward(synth.to_bits(xa[i]), va["W"], va["b"])
        assert_close(logits, ref, what=f"MLP-A req {i}")
        check_argmax(am, logits, ref)
    for i, (logits, am) in enumerate(rb):
        ref, ram = O.mlp_forward(synth.to_bits(xb[i]), vb["W"], vb["b"])
        assert_close(logits, ref, what=f"MLP-B req {i}")
        check_argmax(am, logits, ref)
    srv.close()


def test_mlp_with_biases_and_batch_invariance(mods):
    E, server = mods
    srv = server.Server(workspace_bytes=64 << 20)
    p = synth.make_mlp([256, 384, 72], seed=4, device=DEV, perturb=0.3, std=0.1)
    x = synth.make_mlp_inputs(9, 256, seed=5, device=DEV)
    m = srv.add_model(p)
    t_alone = [srv.submit(m, E.CAT_LS, x=x[3])]
    srv.step()
    alone = _finish(srv, E, t_alone)[0]
    ts = [srv.submit(m, E.CAT_FS, x=x[i]) for i in range(9)]
    srv.step()
    res = _finish(srv, E, ts)
    v = synth.bits_view(p)
    for i, (logits, am) in enumerate(res):
        ref, _ = O.mlp_forward(synth.to_bits(x[i]), v["W"], v["b"])
        assert_close(logits, ref, what=f"req {i}")
    assert torch.equal(alone[0], res[3][0]) and alone[1] == res[3][1]   # bit-identical alone vs in a batch
    srv.close()


def _vit_check(srv, E, p, imgs, mid, cat):
    ts = [srv.submit(mid, cat, x=imgs[i]) for i in range(imgs.shape[0])]
    srv.step()
    res = _finish(srv, E, ts)
    v = synth.bits_view(p)
    errs = []
    for i, (logits, am) in enumerate(res):
        ref, ram, _ = O.vit_forward(synth.to_bits(imgs[i]), v)
        errs.append(assert_close(logits, ref, what=f"ViT image {i}"))
        check_argmax(am, logits, ref)
    return res, errs


@pytest.mark.parametrize("impl", ["simt", "tcgen05"])
def test_small_vit_with_biases(mods, impl):
    E, server = mods
    srv = server.Server(workspace_bytes=256 << 20, gemm_impl=E.GEMM_SIMT if impl == "simt" else E.GEMM_TCGEN05)
    p = synth.make_vit(d=128, n_layers=2, n_heads=2, mlp=256, n_cls=10, seed=6, device=DEV, img=64, std=0.1, perturb=0.2)
    imgs = synth.make_images(3, seed=7, device=DEV, img=64)
    m = srv.add_model(p, max_batch=8)
    _vit_check(srv, E, p, imgs, m, E.CAT_FS)
    srv.close()


@pytest.mark.parametrize("img,patch,T", [(128, 16, 65), (176, 16, 122), (192, 16, 145), (208, 16, 170), (240, 16, 226)])
def test_vit_token_counts_around_the_attention_tiles(mods, img, patch, T):
    """Encoder attention at token counts on both sides of its tile edges: one 128-row query tile
    only partly filled (65, 122), a second tile with 17 and 42 rows (145, 170), key counts that are
    not multiples of 16, and 226 tokens, which is past the single-tile kernel's range and takes the
    flash-loop kernel.  Head size 64, three images so that the items do not fill the grid evenly."""
    E, server = mods
    srv = server.Server(workspace_bytes=256 << 20)
    p = synth.make_vit(d=128, n_layers=1, n_heads=2, mlp=256, n_cls=10, seed=60 + T, device=DEV, img=img, patch=patch,
                       std=0.1, perturb=0.2)
    assert p["T"] == T
    imgs = synth.make_images(3, seed=61 + T, device=DEV, img=img)
    m = srv.add_model(p, max_batch=4)
    _vit_check(srv, E, p, imgs, m, E.CAT_FS)
    srv.close()


def test_config2_vit_b16_batch_2(mods):
    """ViT-B/16 shape (197 tokens, d 768, 12 layers, 12 heads, MLP 3072, 1000 classes)."""
    E, server = mods
    srv = server.Server(workspace_bytes=1 << 30)
    p = synth.make_vit(d=768, n_layers=12, n_heads=12, mlp=3072, n_cls=1000, seed=1, device=DEV)
    imgs = synth.make_images(2, seed=11, device=DEV)
    m = srv.add_model(p, max_batch=8)
    res, _ = _vit_check(srv, E, p, imgs, m, E.CAT_FS)
    # batch invariance: image 1 alone reproduces its in-batch bits
    t = [srv.submit(m, E.CAT_LS, x=imgs[1])]
    srv.step()
    alone = _finish(srv, E, t)[0]
    assert torch.equal(alone[0], res[1][0])
    srv.close()


def replay_layers(p_bits, trace, row, token, kv_len, table, fetch, pool, what):
    """Strict check of a deep decoder, layer by layer.  trace [n_layers + 1, max_batch, d] holds the device's
    residual stream after the embedding and after every layer.  Each layer of the oracle (bf16 rounding at
    the storage points) is fed the DEVICE's own input of that layer, so the error of one layer cannot
    compound through the next: the layer's output, its appended k and v, and the logits computed from the
    device's last residual must each be within 2e-2 per element.  Returns the worst error seen."""
    worst = 0.0
    n_layers = len(p_bits["layers"])
    emb = O.bf16_to_f64(p_bits["Emb"][int(token)])
    assert np.array_equal(to_f64(trace[0, row]), emb), f"{what}: embedding row"          # a gather: bit-exact
    page, slot = int(table[kv_len // 16]), kv_len % 16
    for l in range(n_layers):
        x_in = to_f64(trace[l, row])
        x_out, k, v = O.decoder_layer(x_in, l, kv_len, table, fetch, p_bits, round_bf16=True)
        worst = max(worst, assert_close(trace[l + 1, row], x_out, what=f"{what}: residual after layer {l}"))
        worst = max(worst, assert_close(pool[l, page, 0, :, slot, :], k, what=f"{what}: appended k, layer {l}"))
        worst = max(worst, assert_close(pool[l, page, 1, :, slot, :], v, what=f"{what}: appended v, layer {l}"))
    return worst, O.decoder_head(to_f64(trace[n_layers, row]), p_bits, round_bf16=True)


def _decoder_case(E, server, p, B, lo, hi, seed, impl=None, n_check=None, deep=False, max_batch=None, check=None):
    """One decode step of B requests against the oracle.  `check` names the requests to compare (default:
    the first n_check, or all).  The cache is cloned on the device before the step: the oracle reads a
    request's pages from the clone, and the whole pool is compared with it afterwards, so that only the
    (page, slot) each block table names for the new token may have changed.
    deep: the model is several layers of the 1B / 8B shapes.  The strict element-wise tolerance is then checked
    layer by layer on the device's own layer inputs (replay_layers); the end-to-end logits are compared with
    both oracle evaluations under the rule of assert_parity(deep=True)."""
    toks, lens, tables, npages = synth.make_decode_batch(B, lo, hi, p["vocab"], seed=seed)
    pool = synth.make_kv_pool(p["n_layers"], npages, p["n_kv_heads"], p["head_dim"], seed=seed + 1, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=1 << 30, gemm_impl=impl if impl is not None else E.GEMM_TCGEN05)
    mb = max_batch if max_batch is not None else max(B, 4)
    trace = torch.zeros((p["n_layers"] + 1, mb, p["d"]), dtype=torch.float32, device=DEV) if deep else None
    m = srv.add_model(p, kv_pool=pool, max_kv_len=hi, max_batch=mb, trace=trace)
    tabs = [torch.as_tensor(t, device=DEV) for t in tables]
    ts = [srv.submit(m, E.CAT_FS, token=int(toks[i]), kv_len=int(lens[i]), table=tabs[i]) for i in range(B)]
    info = srv.step()
    res = _finish(srv, E, ts)
    v = synth.bits_view({k: p[k] for k in p if k != "packed_layers"})
    fetch = lambda l, pg: synth.to_bits(pool0[l, pg])
    decided = 0
    errs = []
    if check is None:
        check = range(B) if n_check is None else range(n_check)
    for i in check:
        r = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], fetch, v)
        rb = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], fetch, v, round_bf16=True)
        what = f"decoder req {i} (L={lens[i]})"
        e = assert_parity(res[i][0], r["logits"], rb["logits"], what=what, deep=deep)
        decided += check_argmax(res[i][1], res[i][0], rb["logits"])
        if deep:
            # strict tolerance, every layer on the device's own input; then the head on the device's last residual
            worst, head = replay_layers(v, trace, i, int(toks[i]), int(lens[i]), tables[i], fetch, pool, what)
            worst = max(worst, assert_close(res[i][0], head, what=f"{what}: logits from the device's last residual"))
            check_argmax(res[i][1], res[i][0], head)
            e["layerwise_worst_max_rel"] = worst
            print(f"{what}: layer-by-layer worst max relative error {worst:.3e}")
        else:
            for l, ap in enumerate(rb["appended"]):
                # the new k, v land in exactly the (page, slot) the block table names
                assert_close(pool[l, ap["page"], 0, :, ap["slot"], :], ap["k"], what=f"appended k req {i} layer {l}")
                assert_close(pool[l, ap["page"], 1, :, ap["slot"], :], ap["v"], what=f"appended v req {i} layer {l}")
        errs.append(e)
    touched = torch.zeros((pool.shape[0], pool.shape[1], pool.shape[4]), dtype=torch.bool, device=DEV)   # [layer, page, slot]
    for i in range(B):
        touched[:, int(tables[i][lens[i] // 16]), int(lens[i]) % 16] = True
    same = (pool.view(torch.int16) == pool0.view(torch.int16)).all(dim=5).all(dim=3).all(dim=2)          # [layer, page, slot]
    assert bool(same[~touched].all()), "a cache slot other than the appended ones changed"
    srv.close()
    return info, decided, errs


@pytest.mark.parametrize("impl", ["simt", "tcgen05"])
def test_small_decoder_step(mods, impl):
    E, server = mods
    p = synth.make_decoder(d=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=1000, seed=8,
                           device=DEV, std=0.05, perturb=0.2)
    _decoder_case(E, server, p, B=6, lo=0, hi=600, seed=9, impl=E.GEMM_SIMT if impl == "simt" else E.GEMM_TCGEN05)


def test_config3_decoder_1b_batch_4(mods):
    """Llama-style decoder d 2048, 16 layers, 32/8 heads (hd 64), FFN 8192, vocab 32000, KV lengths
    U[128, 4096], 16-token pages, permuted block tables."""
    E, server = mods
    p = synth.make_decoder(d=2048, n_layers=16, n_q_heads=32, n_kv_heads=8, head_dim=64, ffn=8192, vocab=32000,
                           seed=2, device=DEV)
    info, decided, _ = _decoder_case(E, server, p, B=4, lo=128, hi=4096, seed=21, n_check=2, deep=True)
    assert info.weight_bytes == pytest.approx(2 * (16 * (3072 * 2048 + 2048 * 2048 + 16384 * 2048 + 2048 * 8192)
                                                   + 32000 * 2048))


@pytest.mark.parametrize("n_layers", [1, 2])
def test_config3_shapes_shallow_strict(mods, n_layers):
    """The 1B decoder's layer shapes (d 2048, 32/8 heads, FFN 8192, vocab 32000): strict element-wise
    tolerance at depth 1; at depth 2 the amplification of single rounding differences already puts
    one logit in 32000 at the edge of 2e-2, so the deep-model rule applies."""
    E, server = mods
    p = synth.make_decoder(d=2048, n_layers=n_layers, n_q_heads=32, n_kv_heads=8, head_dim=64, ffn=8192, vocab=32000,
                           seed=2, device=DEV)
    _decoder_case(E, server, p, B=5, lo=128, hi=4096, seed=22, n_check=3, deep=n_layers > 1)


def test_config5_8b_layer_shapes_shallow_strict(mods):
    """The 8B decoder's layer shapes (d 4096, 32/8 heads of 128, FFN 14336, vocab 32000) at depth 1,
    KV lengths U[512, 8192]: strict element-wise tolerance."""
    E, server = mods
    p = synth.make_decoder(d=4096, n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=32000,
                           seed=4, device=DEV)
    _decoder_case(E, server, p, B=3, lo=512, hi=8192, seed=41, n_check=2)


def test_instance_buffer_sets_give_the_same_answers(mods):
    """The end-to-end loop of the benchmark rotates buffer sets (device inputs, outputs and request
    descriptors per set): a step fed from set 2 gives bit-identical results, in that set's own output
    buffers, to a step fed from set 0, and leaves the other sets' outputs alone."""
    E, server = mods
    from paper_2511_00603_b200 import workloads as W
    srv = server.Server(workspace_bytes=256 << 20)
    pm = synth.make_mlp([256, 384, 72], seed=70, device=DEV, perturb=0.3, std=0.1)
    pv = synth.make_vit(d=128, n_layers=1, n_heads=2, mlp=256, n_cls=10, seed=71, device=DEV, img=64, std=0.1)
    insts = [W.Instance(srv, pm, E.CAT_FS, 9, seed=72), W.Instance(srv, pv, E.CAT_LS, 3, seed=73)]
    stream = torch.cuda.current_stream().cuda_stream
    for i in insts:
        i.make_bufs(3)
        i.submit_all(srv.ctx)
    srv.ctx.epara_step(stream, 0)
    torch.cuda.synchronize()
    for i in insts:
        for t in i.tickets:
            assert srv.ctx.epara_collect(t)[0] == E.OK
        assert (i.argmax >= 0).all() and (i.argmax_bufs[2] == -1).all()
        i.x_bufs[2].copy_(i.x)
        i.x.zero_()                                   # set 0's inputs are not what the next step may read
        i.submit_all(srv.ctx, buf=2)
    srv.ctx.epara_step(stream, 0)
    torch.cuda.synchronize()
    for i in insts:
        for t in i.tickets:
            assert srv.ctx.epara_collect(t)[0] == E.OK
        assert torch.equal(i.logits_bufs[2], i.logits) and torch.equal(i.argmax_bufs[2], i.argmax)
        assert (i.argmax_bufs[1] == -1).all()
    srv.close()


def test_mixed_bench_workload_sampled_parity(mods):
    """The benchmark's own configuration (8 co-resident instances, full batches, one step): sampled
    requests of every instance against the oracle, plus properties that hold for all of them."""
    E, server = mods
    from paper_2511_00603_b200 import workloads as W
    srv = server.Server(workspace_bytes=3 << 30)
    insts = W.build_mixed(srv, seed=3)
    pools0 = {i: synth.to_bits(inst.kv_pool) for i, inst in enumerate(insts) if inst.kind == "decoder" and inst.n_req <= 8}
    for inst in insts:
        inst.submit_all(srv.ctx)
    info = srv.ctx.epara_step(torch.cuda.current_stream().cuda_stream, 0)
    torch.cuda.synchronize()
    assert info.admitted[0] == 12 and info.admitted[1] == 1280
    for k, inst in enumerate(insts):
        for t in inst.tickets:
            assert srv.ctx.epara_collect(t)[0] == E.OK
        lg = inst.logits.float()
        assert torch.isfinite(lg).all()
        # the argmax kernel agrees with its own logits for every request of the instance
        assert torch.equal(inst.argmax.long(), lg.argmax(dim=1))
        v = synth.bits_view({kk: inst.p[kk] for kk in inst.p if kk != "packed_layers"})
        if inst.kind == "mlp":
            for i in (0, inst.n_req // 2, inst.n_req - 1):
                ref, _ = O.mlp_forward(synth.to_bits(inst.x[i]), v["W"], v["b"])
                assert_close(inst.logits[i], ref, what=f"instance {k} MLP request {i}")
        elif inst.kind == "vit":
            for i in (0, inst.n_req - 1):
                ref, _, _ = O.vit_forward(synth.to_bits(inst.x[i]), v)
                assert_close(inst.logits[i], ref, what=f"instance {k} ViT-S image {i}")
                check_argmax(int(inst.argmax[i]), inst.logits[i], ref)
        elif k in pools0:
            i = 0                                     # latency-sensitive decoder: its cache copy fits the host
            pb = pools0[k]
            tb = inst.tables[i]
            ra = O.decoder_step(int(inst.tokens[i]), int(inst.lens[i]), tb, lambda l, pg: pb[l, pg], v)
            rb = O.decoder_step(int(inst.tokens[i]), int(inst.lens[i]), tb, lambda l, pg: pb[l, pg], v, round_bf16=True)
            assert_parity(inst.logits[i], ra["logits"], rb["logits"], what=f"instance {k} decoder request {i}", deep=True)
        else:
            # frequency-sensitive decoder (17 GB cache): the oracle reads one request's pages from the device
            i = int(np.argmin(inst.lens))
            tb = inst.tables[i]
            fetch = lambda l, pg: synth.to_bits(inst.kv_pool[l, pg])
            # the step appended this request's k, v at slot L: mask it out by giving the oracle L tokens only
            rb = O.decoder_step(int(inst.tokens[i]), int(inst.lens[i]), tb, fetch, v, round_bf16=True)
            ra = O.decoder_step(int(inst.tokens[i]), int(inst.lens[i]), tb, fetch, v)
            assert_parity(inst.logits[i], ra["logits"], rb["logits"], what=f"instance {k} decoder request {i}", deep=True)
    srv.close()


def test_decoder_batch_invariance_and_mixed_models(mods):
    """One step holding an MLP, a ViT and a decoder: every request equals the oracle, and the decoder
    request's bits do not depend on the co-resident models (MT)."""
    E, server = mods
    pd = synth.make_decoder(d=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=500, seed=30,
                            device=DEV, std=0.05)
    pm = synth.make_mlp([128, 256, 16], seed=31, device=DEV, std=0.1)
    pv = synth.make_vit(d=128, n_layers=1, n_heads=2, mlp=256, n_cls=10, seed=32, device=DEV, img=32, std=0.1)
    toks, lens, tables, npages = synth.make_decode_batch(3, 10, 300, 500, seed=33)
    pool = synth.make_kv_pool(2, npages, 2, 64, seed=34, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=512 << 20)
    md = srv.add_model(pd, kv_pool=pool, max_kv_len=300, max_batch=8)
    mm = srv.add_model(pm, max_batch=8)
    mv = srv.add_model(pv, max_batch=4)
    tabs = [torch.as_tensor(t, device=DEV) for t in tables]
    xs = synth.make_mlp_inputs(2, 128, seed=35, device=DEV)
    imgs = synth.make_images(2, seed=36, device=DEV, img=32)
    t_d = [srv.submit(md, E.CAT_FS, token=int(toks[i]), kv_len=int(lens[i]), table=tabs[i]) for i in range(3)]
    t_m = [srv.submit(mm, E.CAT_LS, x=xs[i]) for i in range(2)]
    t_v = [srv.submit(mv, E.CAT_FS, x=imgs[i]) for i in range(2)]
    srv.step()
    r_d, r_m, r_v = _finish(srv, E, t_d), _finish(srv, E, t_m), _finish(srv, E, t_v)
    pb = synth.to_bits(pool0)
    vd = synth.bits_view({k: pd[k] for k in pd if k != "packed_layers"})
    for i in range(3):
        r = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], lambda l, pg: pb[l, pg], vd)
        rb = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], lambda l, pg: pb[l, pg], vd, round_bf16=True)
        assert_parity(r_d[i][0], r["logits"], rb["logits"], what=f"decoder {i}")
    vm, vv = synth.bits_view(pm), synth.bits_view(pv)
    for i in range(2):
        assert_close(r_m[i][0], O.mlp_forward(synth.to_bits(xs[i]), vm["W"], vm["b"])[0], what=f"mlp {i}")
        assert_close(r_v[i][0], O.vit_forward(synth.to_bits(imgs[i]), vv)[0], what=f"vit {i}")
    # request 1 of the decoder alone, on a fresh copy of the cache
    pool.copy_(pool0)
    t = [srv.submit(md, E.CAT_LS, token=int(toks[1]), kv_len=int(lens[1]), table=tabs[1])]
    srv.step()
    alone = _finish(srv, E, t)[0]
    assert torch.equal(alone[0], r_d[1][0]) and alone[1] == r_d[1][1]
    srv.close()


def test_request_handler_answers(mods):
    """Timeout of an expired request, rejection of the >1 GPU categories, caps, pending tickets."""
    E, server = mods
    srv = server.Server(workspace_bytes=64 << 20, cap_ls=2, cap_fs=3)
    p = synth.make_mlp([64, 64, 8], seed=40, device=DEV, std=0.1)
    x = synth.make_mlp_inputs(8, 64, seed=41, device=DEV)
    m = srv.add_model(p)
    inp = E.Inputs()
    inp.input = x[0].data_ptr()
    out = torch.empty(8, dtype=torch.bfloat16, device=DEV)
    inp.out_logits = out.data_ptr()
    assert srv.ctx.epara_submit(m, E.CAT_LS_GT1, inp, raise_on_error=False)[0] == E.E_UNSUPPORTED
    assert srv.ctx.epara_submit(m, E.CAT_FS_GT1, inp, raise_on_error=False)[0] == E.E_UNSUPPORTED
    assert srv.ctx.epara_submit(m + 5, E.CAT_LS, inp, raise_on_error=False)[0] == E.E_INVALID
    assert srv.ctx.epara_submit(m, 7, inp, raise_on_error=False)[0] == E.E_INVALID
    late = srv.submit(m, E.CAT_LS, x=x[0], deadline_ns=1000)
    live = [srv.submit(m, E.CAT_LS, x=x[i], deadline_ns=5000) for i in range(1, 4)]
    fs = [srv.submit(m, E.CAT_FS, x=x[i]) for i in range(4, 8)]
    assert srv.collect(live[0])[0] == E.PENDING            # still queued
    info = srv.step(now_ns=2000)
    assert list(info.dropped) == [1, 0] and list(info.admitted) == [2, 3]
    torch.cuda.synchronize()
    assert srv.collect(late)[0] == E.E_TIMEOUT
    assert srv.collect(live[0])[0] == E.OK and srv.collect(live[1])[0] == E.OK
    assert srv.collect(live[2])[0] == E.PENDING            # beyond the LS cap: waits for the next step
    assert srv.collect(fs[3])[0] == E.PENDING
    info = srv.step(now_ns=6000)                           # live[2] expired meanwhile
    assert list(info.dropped) == [1, 0] and list(info.admitted) == [0, 1]
    torch.cuda.synchronize()
    assert srv.collect(live[2])[0] == E.E_TIMEOUT
    s, logits, am = srv.collect(fs[3])
    assert s == E.OK
    v = synth.bits_view(p)
    assert_close(logits, O.mlp_forward(synth.to_bits(x[7]), v["W"], v["b"])[0], what="late FS request")
    assert srv.ctx.epara_collect(fs[3])[0] == E.E_INVALID  # already collected
    srv.close()


def test_workspace_too_small_is_resource_insufficiency(mods):
    E, server = mods
    srv = server.Server(workspace_bytes=20 << 20)
    p = synth.make_vit(d=768, n_layers=1, n_heads=12, mlp=3072, n_cls=10, seed=50, device=DEV)
    with pytest.raises(E.EparaError) as ei:
        srv.add_model(p, max_batch=64)
    assert ei.value.status == E.E_RESOURCE
    srv.close()


@pytest.mark.parametrize("shape", [(384, 6, 1536, 2, 3, 224), (128, 2, 256, 2, 5, 96), (256, 4, 512, 1, 4, 128),
                                   (320, 5, 1280, 1, 2, 224)])
def test_fused_encoder_mlp_block_equals_the_unfused_kernels_and_the_oracle(mods, shape):
    """The fused FC1 -> GELU -> FC2 -> residual kernel (default placement of encoder blocks with d <= 384 and more than
    128 rows) against the same model placed with every GEMM as its own launch: same rounding points, same
    reduction order, so the logits must be bit-identical; and against the oracle for the first and last image.
    Shapes: ViT-S (two MMAs of N = 192 per k step), d 128 and 256 (one MMA), d 320 (two of 160; five k-blocks: a
    partly filled second ring slot), with row counts that leave a ragged last pair."""
    E, server = mods
    d, heads, mlp, layers, B, img = shape
    p = synth.make_vit(d=d, n_layers=layers, n_heads=heads, mlp=mlp, n_cls=100, seed=5, device=DEV, img=img, std=0.05,
                       perturb=0.2)
    imgs = synth.make_images(B, seed=6, device=DEV, img=img)

    def run(impl):
        srv = server.Server(workspace_bytes=1 << 30, gemm_impl=impl)
        m = srv.add_model(p, max_batch=B)
        ts = [srv.submit(m, E.CAT_FS, x=imgs[i]) for i in range(B)]
        info = srv.step()
        res = _finish(srv, E, ts)
        srv.close()
        return info, res

    fused_info, fused = run(E.GEMM_TCGEN05)
    plain_info, plain = run(E.GEMM_TCGEN05_UNFUSED)
    assert plain_info.launches - fused_info.launches == layers          # one launch less per block
    assert fused_info.gemm_flops == plain_info.gemm_flops
    for i in range(B):
        assert torch.equal(fused[i][0], plain[i][0]) and fused[i][1] == plain[i][1]
    v = synth.bits_view(p)
    for i in (0, B - 1):
        ref, _, _ = O.vit_forward(synth.to_bits(imgs[i]), v)
        assert_close(fused[i][0], ref, what=f"fused MLP block, d={d}, image {i}")
        check_argmax(fused[i][1], fused[i][0], ref)
