"""Error paths on the GPU, none of which faults, traps or hangs the device: block tables that name pages
outside the pool (skipped and reported), a bounded wait that runs out by design, lengths outside the range
the scratch was sized for (clamped), and steps that fail on the host after admission."""
import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import synth
from tests.parity import assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def mods():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara, server
    return epara, server


def test_page_id_outside_the_declared_pool_is_reported_not_dereferenced(mods):
    """The model is placed with kv_pages = 40 although the pool tensor holds 64 pages per layer.  One request's
    block table names pages 40..63: outside what the library may touch, but inside the allocation, so that
    not even a missing check could reach foreign memory.  The step completes, every request of it answers
    DEVICE with the code of the skipped access, and the pages past the declared range are untouched.  The
    next step has a status word of its own and answers OK, equal to the oracle."""
    E, server = mods
    p = synth.make_decoder(d=256, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=500, seed=600,
                           device=DEV, std=0.05)
    declared, actual = 40, 64
    pool = synth.make_kv_pool(2, actual, 2, 64, seed=601, device=DEV)
    pool0 = pool.clone()
    srv = server.Server(workspace_bytes=256 << 20)
    m = srv.add_model(p, kv_pool=pool, max_kv_len=300, max_batch=8, kv_pages=declared)
    good = torch.arange(0, 10, dtype=torch.int32, device=DEV)          # pages 0..9
    bad = torch.arange(40, 60, dtype=torch.int32, device=DEV)          # outside [0, 40)
    t_good = srv.submit(m, E.CAT_FS, token=7, kv_len=100, table=good)
    t_bad = srv.submit(m, E.CAT_FS, token=9, kv_len=200, table=bad)
    srv.step()
    torch.cuda.synchronize()
    for t in (t_good, t_bad):
        s, out = srv.ctx.epara_collect(t)
        assert s == E.E_DEVICE and out.status == E.E_DEVICE
        assert out.device_error in (E.ERR_PAGE_APPEND, E.ERR_PAGE_ATTEND)
    # as the library sees the pool, layer l starts at page l * declared of the flat tensor: flat pages 80..127 are
    # past its two layers, and within a layer the bad request's pages were never written
    flat, flat0 = pool.view(torch.int16).reshape(2 * actual, -1), pool0.view(torch.int16).reshape(2 * actual, -1)
    assert torch.equal(flat[2 * declared:], flat0[2 * declared:])
    changed = (flat != flat0).any(dim=1).nonzero().flatten().tolist()
    assert set(changed) <= {6, declared + 6}, changed                  # only the good request's page 100 // 16 = 6, per layer
    # a clean step afterwards: not marked by the earlier error
    t2 = srv.submit(m, E.CAT_FS, token=11, kv_len=50, table=good)
    srv.step()
    torch.cuda.synchronize()
    s, out = srv.ctx.epara_collect(t2)
    assert s == E.OK and out.device_error == 0
    srv.close()


def test_bounded_wait_runs_out_and_reports(mods):
    """A wait on a barrier nothing arrives at, limited to 1 ms: the kernel returns by itself, the status word
    holds the self-test's code, the entry answers DEVICE, and the context stays usable."""
    E, _ = mods
    word = torch.zeros(1, dtype=torch.int32, device=DEV)
    s, code = E.epara_selftest_bounded_wait(word, torch.cuda.current_stream().cuda_stream, limit_ns=1_000_000)
    assert s == E.E_DEVICE and code == E.ERR_SELFTEST_WAIT
    assert int(word.item()) == E.ERR_SELFTEST_WAIT
    assert E.lib.epara_selftest_bounded_wait(0, None, 0, word.data_ptr(), None) == E.E_INVALID
    assert float((torch.ones(8, device=DEV) * 2).sum().item()) == 16.0     # the device still answers


def _attn_case(B, lens, Hq, Hkv, hd, seed, extra_pages=0):
    lens = np.asarray(lens, dtype=np.int32)
    need = [(int(L) + 15) // 16 for L in lens]
    npages = sum(need) + extra_pages
    perm = np.random.default_rng(seed).permutation(sum(need)).astype(np.int32)
    tables = np.zeros((B, max(need)), dtype=np.int32)
    o = 0
    for b, n in enumerate(need):
        tables[b, :n] = perm[o:o + n]
        o += n
    pool = synth.make_kv_pool(1, npages, Hkv, hd, seed=seed + 1, device=DEV)[0]
    q = torch.randn((B, Hq * hd), generator=torch.Generator(device=DEV).manual_seed(seed + 2), device=DEV).to(torch.bfloat16)
    return q, pool, lens, tables


def test_decode_attention_entry_reports_bad_pages_and_clamps_lengths(mods):
    E, _ = mods
    stream = torch.cuda.current_stream().cuda_stream
    Hq, Hkv, hd = 8, 2, 64
    q, pool, lens, tables = _attn_case(4, [300, 40, 513, 700], Hq, Hkv, hd, seed=610, extra_pages=8)
    n_used = pool.shape[0] - 8
    max_len = 700
    scratch = torch.zeros(E.lib.epara_decode_attention_scratch_bytes(4, Hq, hd, max_len), dtype=torch.uint8, device=DEV)
    lens_d, tabs_d = torch.as_tensor(lens, device=DEV), torch.as_tensor(tables, device=DEV)
    ref = torch.empty_like(q)
    E.epara_decode_attention(q, pool, lens_d, tabs_d, ref, Hq, Hkv, hd, max_len, scratch, stream)
    torch.cuda.synchronize()
    status = lambda: int(scratch[E.DECODE_STATUS_OFFSET:E.DECODE_STATUS_OFFSET + 4].view(torch.int32).item())
    assert status() == 0
    # (a) lengths past max_len are clamped to it: request 3 claims 5000 tokens and is served as 700
    over = lens.copy()
    over[3] = 5000
    got = torch.empty_like(q)
    E.epara_decode_attention(q, pool, torch.as_tensor(over, device=DEV), tabs_d, got, Hq, Hkv, hd, max_len, scratch, stream)
    torch.cuda.synchronize()
    assert status() == 0 and torch.equal(got, ref)
    # a negative length is served as 0: the row is left as it was
    neg = lens.copy()
    neg[1] = -5
    got = torch.full_like(q, 3.0)
    E.epara_decode_attention(q, pool, torch.as_tensor(neg, device=DEV), tabs_d, got, Hq, Hkv, hd, max_len, scratch, stream)
    torch.cuda.synchronize()
    assert torch.equal(got[[0, 2, 3]], ref[[0, 2, 3]]) and bool((got[1] == 3.0).all())
    # (b) page ids outside the declared page count (but inside the tensor): reported, other requests unaffected
    bad = tables.copy()
    bad[1, 0] = n_used + 3
    got = torch.empty_like(q)
    E.epara_decode_attention(q, pool, lens_d, torch.as_tensor(bad, device=DEV), got, Hq, Hkv, hd, max_len, scratch, stream,
                             kv_pages=n_used)
    torch.cuda.synchronize()
    assert status() == E.ERR_PAGE_ATTEND
    assert torch.equal(got[[0, 2, 3]], ref[[0, 2, 3]])
    bad[1, 0] = -1
    E.epara_decode_attention(q, pool, lens_d, torch.as_tensor(bad, device=DEV), got, Hq, Hkv, hd, max_len, scratch, stream,
                             kv_pages=n_used)
    torch.cuda.synchronize()
    assert status() == E.ERR_PAGE_ATTEND
    # the status word is cleared by the next call
    E.epara_decode_attention(q, pool, lens_d, tabs_d, got, Hq, Hkv, hd, max_len, scratch, stream)
    torch.cuda.synchronize()
    assert status() == 0 and torch.equal(got, ref)


def test_step_that_fails_on_the_host_answers_its_requests(mods):
    """A profiled step with more launches than the profile may hold runs nothing: the step answers RESOURCE,
    and so does every request it had admitted (they neither stay pending for ever nor answer OK).  The same
    requests submitted again run normally."""
    E, server = mods
    srv = server.Server(workspace_bytes=64 << 20, profile=True)
    p = synth.make_mlp([64, 128, 16], seed=620, device=DEV, std=0.1)
    x = synth.make_mlp_inputs(3, 64, seed=621, device=DEV)
    m = srv.add_model(p)
    assert E.lib.epara_set_max_profile_launches(srv.ctx.h, 2) == E.OK       # the step needs 4 launches
    ts = [srv.submit(m, E.CAT_LS, x=x[i]) for i in range(3)]
    with pytest.raises(E.EparaError) as ei:
        srv.step()
    assert ei.value.status == E.E_RESOURCE
    torch.cuda.synchronize()
    for t in ts:
        s, out = srv.ctx.epara_collect(t)
        assert s == E.E_RESOURCE and out.status == E.E_RESOURCE
        assert srv.ctx.epara_collect(t)[0] == E.E_INVALID                   # answered once
    assert E.lib.epara_set_max_profile_launches(srv.ctx.h, 4096) == E.OK
    ts = [srv.submit(m, E.CAT_LS, x=x[i]) for i in range(3)]
    srv.step()
    torch.cuda.synchronize()
    v = synth.bits_view(p)
    for i, t in enumerate(ts):
        s, logits, am = srv.collect(t)
        assert s == E.OK
        assert_close(logits, O.mlp_forward(synth.to_bits(x[i]), v["W"], v["b"])[0], what=f"request {i}")
    srv.close()


def test_answers_survive_many_later_steps(mods):
    """A request collected long after its step (more steps later than the library keeps step records) still
    answers OK once, with its outputs in place."""
    E, server = mods
    srv = server.Server(workspace_bytes=64 << 20)
    p = synth.make_mlp([64, 128, 16], seed=630, device=DEV, std=0.1)
    x = synth.make_mlp_inputs(8, 64, seed=631, device=DEV)
    m = srv.add_model(p)
    first = srv.submit(m, E.CAT_LS, x=x[0])
    srv.step()
    later = []
    for i in range(1, 8):
        later.append(srv.submit(m, E.CAT_LS, x=x[i]))
        srv.step()
    torch.cuda.synchronize()
    v = synth.bits_view(p)
    s, logits, am = srv.collect(first)
    assert s == E.OK
    assert_close(logits, O.mlp_forward(synth.to_bits(x[0]), v["W"], v["b"])[0], what="first request")
    for t in later:
        assert srv.collect(t)[0] == E.OK
    srv.close()
