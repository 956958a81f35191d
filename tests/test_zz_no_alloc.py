"""The allocation-free decode-attention entry point against the ordinary one.

epara_decode_attention_static is for embedders that cannot hand the library a scratch buffer
because they cannot allocate one (the device belongs to a framework's memory pool, or a
cudaMalloc would stall a latency-critical loop).  It must give what epara_decode_attention gives,
call after call, although all its calls share one built-in scratch array that keeps the previous
call's contents (only its chunk counters are cleared per call).
This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2511_00603_b200 import synth
from tests.parity import assert_close, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def E():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara
    return epara


def _case(E, B, lens, Hq, Hkv, hd, seed):
    dev = torch.device("cuda")
    lens = np.asarray(lens, dtype=np.int32)
    need = [(int(L) + 15) // 16 for L in lens]
    npages = sum(need) + 2
    perm = np.random.default_rng(seed).permutation(npages).astype(np.int32)
    tables = np.zeros((B, max(need)), dtype=np.int32)
    o = 0
    for b, n in enumerate(need):
        tables[b, :n] = perm[o:o + n]
        o += n
    pool = synth.make_kv_pool(1, npages, Hkv, hd, seed=seed + 1, device=dev)[0]
    q = torch.randn((B, Hq * hd), generator=torch.Generator(device=dev).manual_seed(seed + 2), device=dev).to(torch.bfloat16)
    return q, pool, torch.as_tensor(lens, device=dev), torch.as_tensor(tables, device=dev), int(lens.max())


def test_static_scratch_entry_matches_the_ordinary_entry_twice_in_a_row(E):
    stream = torch.cuda.current_stream().cuda_stream
    # different problems back to back: each call finds the previous one's leftovers in the array; the third
    # repeats the first (several chunks per request, merged by the last block to arrive) after the second,
    # so it runs on chunk counters that the earlier calls must have left at zero
    problems = [(6, [700, 1, 256, 257, 40, 1023], 8, 2, 64, 70), (3, [300, 17, 513], 8, 2, 128, 80),
                (6, [700, 1, 256, 257, 40, 1023], 8, 2, 64, 70)]
    for n, (B, lens, Hq, Hkv, hd, seed) in enumerate(problems):
        q, pool, lens_d, tabs_d, max_len = _case(E, B, lens, Hq, Hkv, hd, seed)
        ref = torch.empty_like(q)
        scratch = torch.empty(E.lib.epara_decode_attention_scratch_bytes(B, Hq, hd, max_len), dtype=torch.uint8,
                              device=q.device)
        E.epara_decode_attention(q, pool, lens_d, tabs_d, ref, Hq, Hkv, hd, max_len, scratch, stream)
        got = torch.full_like(q, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        E.epara_decode_attention_static(q, pool, lens_d, tabs_d, got, Hq, Hkv, hd, max_len, stream)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if n > 0:
            # (the first call may load the kernels; from the second on the call must leave the device's free
            # memory exactly as it found it)
            assert free_after == free_before, f"call {n}: free device memory changed by {free_before - free_after} bytes"
        assert_close(got, to_f64(ref), what=f"static-scratch decode attention B={B} hd={hd}")
        assert torch.equal(got, ref)          # same kernels, same reduction order


def test_static_scratch_entry_rejects_what_does_not_fit(E):
    assert E.lib.epara_static_scratch_bytes() == 8 << 20
    stream = torch.cuda.current_stream().cuda_stream
    q, pool, lens_d, tabs_d, max_len = _case(E, 2, [30, 50], 8, 2, 64, 90)
    out = torch.empty_like(q)
    # claim a batch and length whose partials need far more than the built-in array holds
    s = E.lib.epara_decode_attention_static(0, stream, q.data_ptr(), q.stride(0), pool.data_ptr(), pool.shape[0],
                                            lens_d.data_ptr(), tabs_d.data_ptr(), tabs_d.stride(0), out.data_ptr(), 4096, 32,
                                            8, 64, 8192)
    assert s == E.E_RESOURCE
    assert E.lib.epara_decode_attention_static(0, stream, None, 0, None, 1, None, None, 0, None, 1, 8, 2, 64, 16) == E.E_INVALID
