"""GPU parity of the decoder's prefill phase (prompt chunks through epara_submit with n_tokens > 1) against
the oracle's decoder_prefill: prompt lengths around the attention tile edges, chunked prefill on top of a
cached prefix, head size 128, prompt chunks and decode requests of one model mixed in one step, and the
hand-over from prefill to decode through the cache the prefill wrote."""
import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import configs, synth
from tests.parity import assert_close, assert_parity, check_argmax, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def mods():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara, server
    return epara, server


def _table(rng, n_tokens_total, offset=0):
    """A block table of ceil(n / 16) pages drawn from a permutation (offset: first page index to use)."""
    n = (n_tokens_total + 15) // 16
    return (rng.permutation(n) + offset).astype(np.int32)


def _check_prefill(p_bits, pool, pool0, res, tokens, kv_len, table, what, deep=False):
    """Last-token logits against both oracle evaluations, every appended k and v of every layer against the
    bf16-storage evaluation, and the positions they went to."""
    fetch = lambda l, pg: synth.to_bits(pool0[l, pg])
    ra = O.decoder_prefill(tokens, kv_len, table, fetch, p_bits)
    rb = O.decoder_prefill(tokens, kv_len, table, fetch, p_bits, round_bf16=True)
    e = assert_parity(res[0], ra["logits"], rb["logits"], what=what, deep=deep)
    check_argmax(res[1], res[0], rb["logits"])
    n = len(tokens)
    pos = kv_len + np.arange(n)
    pages, slots = torch.as_tensor(table[pos // 16].astype(np.int64), device=DEV), torch.as_tensor(pos % 16, device=DEV)
    for l, ap in enumerate(rb["appended"]):
        got_k = pool[l, pages, 0][:, :, :, :].permute(0, 2, 1, 3)[torch.arange(n, device=DEV), slots]     # [n, Hkv, hd]
        got_v = pool[l, pages, 1][:, :, :, :].permute(0, 2, 1, 3)[torch.arange(n, device=DEV), slots]
        assert_close(got_k, ap["k"], what=f"{what}: appended k, layer {l}")
        assert_close(got_v, ap["v"], what=f"{what}: appended v, layer {l}")
    return e


def _untouched_elsewhere(pool, pool0, touched_positions):
    """touched_positions: list of (page, slot).  Every other slot of every layer must be bit-identical."""
    touched = torch.zeros((pool.shape[1], pool.shape[4]), dtype=torch.bool, device=DEV)
    for pg, sl in touched_positions:
        touched[pg, sl] = True
    same = (pool.view(torch.int16) == pool0.view(torch.int16)).all(dim=5).all(dim=3).all(dim=2)          # [layer, page, slot]
    assert bool(same[:, ~touched].all()), "a cache slot outside the chunk's positions changed"


@pytest.mark.parametrize("n", [2, 63, 64, 65, 127, 128, 129, 1000])
def test_prefill_of_a_whole_prompt_at_the_1b_layer_shapes(mods, n):
    """One layer of the 1B decoder's shapes (strict element-wise tolerance), prompts of n tokens on an empty
    cache: n on both sides of the 64-token query tile and key block edges, and 1000."""
    E, server = mods
    cfg = dict(configs.DEC_1B, n_layers=1)
    p = synth.make_decoder(seed=2, device=DEV, **cfg)
    rng = np.random.default_rng(800 + n)
    tokens = [int(t) for t in rng.integers(0, cfg["vocab"], n)]
    table = _table(rng, n)
    pool = synth.make_kv_pool(1, len(table) + 2, cfg["n_kv_heads"], cfg["head_dim"], seed=801, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=1 << 30)
    m = srv.add_model(p, kv_pool=pool, max_kv_len=1024, max_batch=1024)
    t = srv.submit(m, E.CAT_FS, tokens=tokens, kv_len=0, table=torch.as_tensor(table, device=DEV))
    info = srv.step()
    assert info.prefill_tokens == n and info.admitted[1] == 1
    torch.cuda.synchronize()
    s, logits, am = srv.collect(t)
    assert s == E.OK
    v = synth.bits_view({k: p[k] for k in p if k != "packed_layers"})
    e = _check_prefill(v, pool, pool0, (logits, int(am.item())), tokens, 0, table, f"prompt of {n} tokens")
    print(f"prompt of {n}: {e}")
    _untouched_elsewhere(pool, pool0, [(int(table[q // 16]), q % 16) for q in range(n)])
    srv.close()


def test_chunked_prefill_on_a_cached_prefix_and_head_size_128(mods):
    """A later chunk of a chunked prefill: 300 tokens already cached (random cache contents), a chunk of 200
    tokens on top; one layer of the 8B decoder's shapes (head size 128, KV heads shared by 4 query heads)."""
    E, server = mods
    cfg = dict(configs.DEC_8B, n_layers=1)
    p = synth.make_decoder(seed=4, device=DEV, **cfg)
    rng = np.random.default_rng(810)
    kv0, n = 300, 200
    tokens = [int(t) for t in rng.integers(0, cfg["vocab"], n)]
    table = _table(rng, kv0 + n, offset=3)
    pool = synth.make_kv_pool(1, len(table) + 5, cfg["n_kv_heads"], cfg["head_dim"], seed=811, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=2 << 30)
    m = srv.add_model(p, kv_pool=pool, max_kv_len=1024, max_batch=256)
    t = srv.submit(m, E.CAT_LS, tokens=tokens, kv_len=kv0, table=torch.as_tensor(table, device=DEV))
    srv.step()
    torch.cuda.synchronize()
    s, logits, am = srv.collect(t)
    assert s == E.OK
    v = synth.bits_view({k: p[k] for k in p if k != "packed_layers"})
    _check_prefill(v, pool, pool0, (logits, int(am.item())), tokens, kv0, table, "chunk of 200 after 300 cached")
    _untouched_elsewhere(pool, pool0, [(int(table[q // 16]), q % 16) for q in range(kv0, kv0 + n)])
    srv.close()


def test_prompt_chunks_and_decode_requests_share_a_step(mods):
    """One decoder serving, in ONE step, two prompt chunks (37 tokens on an empty cache; 90 tokens after 21
    cached) and three decode requests, co-resident with a ViT.  Every request equals the oracle; and a
    request's bits do not depend on what shares its step: each is repeated alone on a fresh copy of the cache."""
    E, server = mods
    p = synth.make_decoder(d=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=500, seed=820,
                           device=DEV, std=0.05, perturb=0.2)
    pv = synth.make_vit(d=128, n_layers=1, n_heads=2, mlp=256, n_cls=10, seed=821, device=DEV, img=32, std=0.1)
    rng = np.random.default_rng(822)
    toks, lens, tables, npages = synth.make_decode_batch(3, 10, 300, 500, seed=823)
    chunks = [([int(t) for t in rng.integers(0, 500, 37)], 0), ([int(t) for t in rng.integers(0, 500, 90)], 21)]
    ctabs, off = [], npages
    for tk, kv0 in chunks:
        ctabs.append(_table(rng, kv0 + len(tk), offset=off))
        off += len(ctabs[-1])
    pool = synth.make_kv_pool(2, off + 1, 2, 64, seed=824, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=512 << 20)
    md = srv.add_model(p, kv_pool=pool, max_kv_len=320, max_batch=160)
    mv = srv.add_model(pv, max_batch=4)
    imgs = synth.make_images(2, seed=825, device=DEV, img=32)
    dtabs = [torch.as_tensor(t, device=DEV) for t in tables]
    ptabs = [torch.as_tensor(t, device=DEV) for t in ctabs]

    def submit_all():
        tp0 = srv.submit(md, E.CAT_FS, tokens=chunks[0][0], kv_len=chunks[0][1], table=ptabs[0])
        td = [srv.submit(md, E.CAT_FS, token=int(toks[i]), kv_len=int(lens[i]), table=dtabs[i]) for i in range(3)]
        tp1 = srv.submit(md, E.CAT_FS, tokens=chunks[1][0], kv_len=chunks[1][1], table=ptabs[1])
        tv = [srv.submit(mv, E.CAT_FS, x=imgs[i]) for i in range(2)]
        return [tp0] + td + [tp1], tv

    def finish(ts):
        torch.cuda.synchronize()
        out = []
        for t in ts:
            s, logits, am = srv.collect(t)
            assert s == E.OK
            out.append((logits, int(am.item())))
        return out

    ts, tv = submit_all()
    info = srv.step()
    assert info.prefill_tokens == 127 and info.admitted[1] == 7
    res, resv = finish(ts), finish(tv)
    v = synth.bits_view({k: p[k] for k in p if k != "packed_layers"})
    fetch = lambda l, pg: synth.to_bits(pool0[l, pg])
    _check_prefill(v, pool, pool0, res[0], chunks[0][0], 0, ctabs[0], "chunk 0")
    _check_prefill(v, pool, pool0, res[4], chunks[1][0], 21, ctabs[1], "chunk 1")
    for i in range(3):
        ra = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], fetch, v)
        rb = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], fetch, v, round_bf16=True)
        assert_parity(res[1 + i][0], ra["logits"], rb["logits"], what=f"decode request {i}")
    vv = synth.bits_view(pv)
    for i in range(2):
        assert_close(resv[i][0], O.vit_forward(synth.to_bits(imgs[i]), vv)[0], what=f"ViT image {i}")
    # each decoder request alone, on a fresh copy of the cache: bit-identical
    mixed_pool = pool.clone()
    singles = ([dict(tokens=chunks[0][0], kv_len=0, table=ptabs[0])] +
               [dict(token=int(toks[i]), kv_len=int(lens[i]), table=dtabs[i]) for i in range(3)] +
               [dict(tokens=chunks[1][0], kv_len=21, table=ptabs[1])])
    for k, kw in enumerate(singles):
        pool.copy_(pool0)
        t = srv.submit(md, E.CAT_LS, **kw)
        srv.step()
        alone = finish([t])[0]
        assert torch.equal(alone[0], res[k][0]) and alone[1] == res[k][1], f"request {k} depends on its step's company"
    assert mixed_pool.shape == pool.shape
    srv.close()


def test_decode_continues_from_the_cache_a_prefill_wrote(mods):
    """Prefill of a 50-token prompt, then a decode step of the next token on the same sequence: the decode step
    must equal the oracle's decode step over the cache as the device's prefill left it."""
    E, server = mods
    p = synth.make_decoder(d=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=500, seed=830,
                           device=DEV, std=0.05, perturb=0.2)
    rng = np.random.default_rng(831)
    n = 50
    tokens = [int(t) for t in rng.integers(0, 500, n)]
    table = _table(rng, n + 1)
    pool = synth.make_kv_pool(2, len(table), 2, 64, seed=832, device=DEV)
    srv = server.Server(workspace_bytes=256 << 20)
    m = srv.add_model(p, kv_pool=pool, max_kv_len=100, max_batch=64)
    tab = torch.as_tensor(table, device=DEV)
    t = srv.submit(m, E.CAT_FS, tokens=tokens, kv_len=0, table=tab)
    srv.step()
    torch.cuda.synchronize()
    s, logits, am = srv.collect(t)
    assert s == E.OK
    nxt = int(am.item())                                           # greedy: the argmax is the next token
    after_prefill = pool.clone()
    t = srv.submit(m, E.CAT_FS, token=nxt, kv_len=n, table=tab)
    srv.step()
    torch.cuda.synchronize()
    s, logits2, am2 = srv.collect(t)
    assert s == E.OK
    v = synth.bits_view({k: p[k] for k in p if k != "packed_layers"})
    fetch = lambda l, pg: synth.to_bits(after_prefill[l, pg])
    ra = O.decoder_step(nxt, n, table, fetch, v)
    rb = O.decoder_step(nxt, n, table, fetch, v, round_bf16=True)
    assert_parity(logits2, ra["logits"], rb["logits"], what="decode after prefill")
    check_argmax(int(am2.item()), logits2, rb["logits"])
    srv.close()


def test_prefill_admission_by_token_rows_and_rejections(mods):
    """A decoder placed for 64 token rows: chunks of 40 and 30 tokens cannot share a step (the second waits),
    a chunk of 65 is refused at submit (resource insufficiency), a chunk whose positions pass max_kv_len or
    whose table is too short is invalid, and a model with head size 16 does not take prompt chunks."""
    E, server = mods
    p = synth.make_decoder(d=128, n_layers=1, n_q_heads=2, n_kv_heads=1, head_dim=64, ffn=256, vocab=100, seed=840,
                           device=DEV, std=0.05)
    pool = synth.make_kv_pool(1, 16, 1, 64, seed=841, device=DEV)
    srv = server.Server(workspace_bytes=128 << 20)
    m = srv.add_model(p, kv_pool=pool, max_kv_len=200, max_batch=64)
    tab_a = torch.arange(0, 4, dtype=torch.int32, device=DEV)
    tab_b = torch.arange(4, 8, dtype=torch.int32, device=DEV)
    ta = srv.submit(m, E.CAT_FS, tokens=list(range(40)), kv_len=0, table=tab_a)
    tb = srv.submit(m, E.CAT_FS, tokens=list(range(30)), kv_len=0, table=tab_b)
    info = srv.step()
    assert info.admitted[1] == 1 and info.prefill_tokens == 40
    torch.cuda.synchronize()
    assert srv.collect(ta)[0] == E.OK and srv.collect(tb)[0] == E.PENDING
    info = srv.step()
    assert info.admitted[1] == 1 and info.prefill_tokens == 30
    torch.cuda.synchronize()
    assert srv.collect(tb)[0] == E.OK

    def status(**kw):
        inp = E.Inputs()
        toks = kw.pop("tokens")
        arr = (E.C.c_int32 * len(toks))(*toks)
        inp.tokens, inp.n_tokens = arr, len(toks)
        inp.kv_len, inp.block_table, inp.n_blocks = kw["kv_len"], kw["table"].data_ptr(), kw["table"].numel()
        out = torch.empty(100, dtype=torch.bfloat16, device=DEV)
        inp.out_logits = out.data_ptr()
        return srv.ctx.epara_submit(kw.get("model", m), E.CAT_FS, inp, raise_on_error=False)[0]

    big = torch.arange(0, 16, dtype=torch.int32, device=DEV)
    assert status(tokens=list(range(65)), kv_len=0, table=big) == E.E_RESOURCE
    assert status(tokens=list(range(20)), kv_len=190, table=big) == E.E_INVALID          # positions pass max_kv_len
    assert status(tokens=list(range(40)), kv_len=0, table=tab_a[:2]) == E.E_INVALID       # 40 tokens need 3 pages
    assert status(tokens=[5, 100], kv_len=0, table=big) == E.E_INVALID                    # token id out of range
    p16 = synth.make_decoder(d=64, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=128, vocab=100, seed=842,
                             device=DEV, std=0.05)
    pool16 = synth.make_kv_pool(1, 16, 2, 16, seed=843, device=DEV)
    m16 = srv.add_model(p16, kv_pool=pool16, max_kv_len=200, max_batch=64)
    assert status(tokens=[1, 2, 3], kv_len=0, table=big, model=m16) == E.E_UNSUPPORTED
    srv.close()
