"""GPU parity of the single kernels against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import synth
from tests.parity import assert_close, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def E():
    from paper_2511_00603_b200 import build
    build.build()
    from paper_2511_00603_b200 import epara
    return epara


def _stream():
    return torch.cuda.current_stream().cuda_stream


GEMM_CASES = [
    # M, N, K, epilogue flags (names)
    (8, 512, 512, ("bias", "gelu")),
    (32, 1024, 256, ("bias",)),
    (197, 2304, 768, ("bias",)),
    (1, 3072, 2048, ()),
    (130, 10, 512, ("bias",)),          # N below one tile, not a multiple of 8
    (300, 1000, 768, ("bias",)),        # ragged M and N
    (33, 512, 256, ("swiglu",)),
    (77, 768, 3072, ("bias", "resid")),
    (0, 64, 64, ()),                    # empty group
    (257, 136, 64, ("gelu", "bias")),   # single k-block, N tail of 8
    (40, 1024, 1024, ("swiglu",)),      # split along K with a SwiGLU epilogue
    (256, 2048, 4096, ("resid",)),      # two row tiles, long K
    (64, 512, 8192, ("bias", "resid")), # few tiles, very long K: split along K with the last-arriver reduction
    (20, 768, 4096, ("gelu", "bias")),  # split along K, bf16 output
    (9, 256, 5120, ("swiglu",)),        # split along K, SwiGLU, uneven ranges
    # at most 16 rows: the weight-streaming kernel (16 W rows per block, k-blocks of 32 dealt to 8 warps)
    (16, 1000, 776, ("bias",)),         # ragged N, K not a multiple of 32
    (3, 10, 512, ("bias",)),            # N below one block
    (5, 64, 8, ()),                     # a single 16-byte piece of K
    (12, 2048, 8192, ("resid",)),       # long K, fp32 residual
    (2, 512, 2048, ("swiglu",)),
    (1, 32000, 2048, ()),               # LM head of one request
]


def _run_gemm(E, impl, cases, seed=0):
    dev = torch.device("cuda")
    g = torch.Generator(device=dev).manual_seed(seed)
    probs, refs = [], []
    for (M, N, K, fl) in cases:
        A = torch.randn((max(M, 1), K), generator=g, device=dev).to(torch.bfloat16)
        W = (torch.randn((N, K), generator=g, device=dev) * 0.05).to(torch.bfloat16)
        bias = (torch.randn((N,), generator=g, device=dev) * 0.5).to(torch.bfloat16) if "bias" in fl else None
        epi = (E.EPI_BIAS if "bias" in fl else 0) | (E.EPI_GELU if "gelu" in fl else 0) | \
              (E.EPI_SWIGLU if "swiglu" in fl else 0) | (E.EPI_RESID_F32 if "resid" in fl else 0)
        ldc = ((N // 2 if "swiglu" in fl else N) + 7) // 8 * 8
        if "resid" in fl:
            Cc = torch.randn((max(M, 1), ldc), generator=g, device=dev, dtype=torch.float32)
        else:
            Cc = torch.full((max(M, 1), ldc), float("nan"), device=dev, dtype=torch.bfloat16)
        C0 = Cc.clone()
        probs.append({"A": A, "W": W, "C": Cc, "bias": bias, "M": M, "N": N, "K": K, "epilogue": epi})
        # oracle
        y = O.linear(O.bf16_to_f64(synth.to_bits(A))[:M], O.bf16_to_f64(synth.to_bits(W)),
                     O.bf16_to_f64(synth.to_bits(bias)) if bias is not None else None)
        if "gelu" in fl:
            y = O.gelu(y)
        if "swiglu" in fl:
            y = O.silu(y[:, 0::2]) * y[:, 1::2]
        if "resid" in fl:
            y = C0[:M, :N].double().cpu().numpy() + y
        refs.append(y)
    scratch = torch.empty(E.epara_gemm_scratch_bytes_for(probs), dtype=torch.uint8, device=dev)
    E.epara_grouped_gemm(probs, _stream(), scratch, impl=impl)
    torch.cuda.synchronize()
    status = int(scratch[:4].view(torch.int32).item())
    assert status == 0, f"device status {status}"
    return probs, refs


@pytest.mark.parametrize("impl", ["simt", "tcgen05"])
def test_grouped_gemm_matches_oracle(E, impl):
    probs, refs = _run_gemm(E, E.GEMM_SIMT if impl == "simt" else E.GEMM_TCGEN05, GEMM_CASES)
    for p, ref, case in zip(probs, refs, GEMM_CASES):
        M, ncols = ref.shape
        if M == 0:
            continue
        assert_close(p["C"][:M, :ncols], ref, what=f"{impl} gemm {case}")
        if impl == "simt" and p["C"].dtype == torch.bfloat16 and p["C"].shape[1] > ncols:
            # (the tensor-core kernel stores through TMA in 16-byte units and may fill the pad
            # columns up to the next multiple of 8, which the C ABI allows)
            assert torch.isnan(p["C"][:M, ncols:].float()).all(), "wrote beyond N"


def test_grouped_gemm_many_tiles_and_group_independence(E):
    """More tiles than SMs, several k-blocks beyond the stage ring, and the same problem alone vs
    among others gives bit-identical output (no dependence on co-resident groups)."""
    big = [(1576, 768, 768, ("bias",)), (640, 3072, 768, ("bias", "gelu")), (1000, 768, 3072, ("bias", "resid"))]
    probs, refs = _run_gemm(E, E.GEMM_TCGEN05, big, seed=3)
    for p, ref, case in zip(probs, refs, big):
        assert_close(p["C"][:ref.shape[0], :ref.shape[1]], ref, what=f"gemm {case}")
    alone, _ = _run_gemm(E, E.GEMM_TCGEN05, big[:1], seed=3)
    assert torch.equal(alone[0]["C"], probs[0]["C"])


def test_grouped_gemm_tile_pairs(E):
    """Dense bf16-output problems (more than 256 rows, 256-wide tiles) run as 256-row tiles on CTA pairs:
    ragged last pair (one CTA with no valid row), N tails inside the first and the second half of the W
    rows, SwiGLU, one k-block, a long K beyond the six-stage ring, more pairs than SM pairs, fp32-residual
    outputs with 192- and 256-wide tiles, 128-wide tiles of problems with 129 to 256 rows, N below one tile."""
    cases = [(1000, 1152, 384, ("bias",)), (513, 2048, 256, ("swiglu",)), (700, 264, 1536, ("bias", "gelu")),
             (257, 392, 64, ()), (20000, 512, 128, ("bias",)), (384, 256, 4096, ("gelu", "bias")),
             (900, 384, 384, ("bias", "resid")), (515, 768, 1536, ("resid",)), (1300, 576, 192, ("bias", "resid")),
             (200, 512, 512, ("bias", "gelu")), (256, 2048, 2048, ("resid",)), (129, 10, 512, ("bias",))]
    probs, refs = _run_gemm(E, E.GEMM_TCGEN05, cases, seed=9)
    for p, ref, case in zip(probs, refs, cases):
        assert_close(p["C"][:ref.shape[0], :ref.shape[1]], ref, what=f"pair gemm {case}")
    alone, _ = _run_gemm(E, E.GEMM_TCGEN05, cases[:1], seed=9)
    assert torch.equal(alone[0]["C"], probs[0]["C"])


def test_grouped_gemm_swapped_operands_17_to_128_rows(E):
    """Problems of 17 to 128 rows run with W as the tensor core's 128-row operand and the batch as its N, a cluster
    of 1, 2, 4 or 8 CTAs per tile of 128 output columns splitting K (reduced through distributed shared memory in
    rank order): every epilogue, N below and not a multiple of a tile, K not a multiple of a k-block, batch sizes
    on both sides of the multiples of 16, one k-block, and the decode shapes of the 1B decoder.  The same problem
    alone and among others gives the same bits."""
    cases = [(17, 10, 512, ("bias",)), (128, 3072, 2048, ()), (100, 1000, 776, ("bias",)), (48, 2048, 8192, ("resid",)),
             (33, 512, 256, ("swiglu",)), (64, 2048, 2048, ("resid", "bias")), (127, 16384, 2048, ("swiglu",)),
             (32, 1024, 256, ("bias", "gelu")), (96, 136, 64, ("gelu", "bias")), (20, 768, 4096, ("gelu", "bias")),
             (128, 32000, 2048, ()), (31, 264, 1536, ("bias", "resid")), (80, 4096, 4096, ("swiglu",))]
    probs, refs = _run_gemm(E, E.GEMM_TCGEN05, cases, seed=11)
    for p, ref, case in zip(probs, refs, cases):
        assert_close(p["C"][:ref.shape[0], :ref.shape[1]], ref, what=f"swapped gemm {case}")
    alone, _ = _run_gemm(E, E.GEMM_TCGEN05, cases[:2], seed=11)
    assert torch.equal(alone[1]["C"], probs[1]["C"])
    # fewer live rows than the capacity the tile was sized for leave the other rows' outputs untouched
    M, N, K = 128, 512, 512
    g = torch.Generator(device="cuda").manual_seed(12)
    A = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((N, K), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    full = torch.zeros((M, N), device="cuda", dtype=torch.bfloat16)
    part = torch.full((M, N), 7.0, device="cuda", dtype=torch.bfloat16)
    for C_, rows in ((full, M), (part, 40)):
        pr = [{"A": A, "W": W, "C": C_, "bias": None, "M": rows, "N": N, "K": K, "epilogue": 0}]
        sc = torch.empty(E.epara_gemm_scratch_bytes_for(pr), dtype=torch.uint8, device="cuda")
        E.epara_grouped_gemm(pr, _stream(), sc)
    torch.cuda.synchronize()
    assert bool((part[40:] == 7.0).all())
    assert_close(part[:40], to_f64(full[:40]), what="first 40 rows", tol=1e-6)


def test_grouped_gemm_rejects_bad_arguments(E):
    dev = torch.device("cuda")
    A = torch.zeros((8, 64), device=dev, dtype=torch.bfloat16)
    W = torch.zeros((8, 64), device=dev, dtype=torch.bfloat16)
    Cc = torch.zeros((8, 8), device=dev, dtype=torch.bfloat16)
    scratch = torch.empty(4096, dtype=torch.uint8, device=dev)
    bad = {"A": A[:, 1:], "W": W, "C": Cc, "M": 8, "N": 8, "K": 63, "epilogue": 0}
    with pytest.raises(E.EparaError) as ei:
        E.epara_grouped_gemm([bad], _stream(), scratch)
    assert ei.value.status == E.E_INVALID
    small = torch.empty(256, dtype=torch.uint8, device=dev)
    ok = {"A": A, "W": W, "C": Cc, "M": 8, "N": 8, "K": 64, "epilogue": 0}
    with pytest.raises(E.EparaError) as ei:
        E.epara_grouped_gemm([ok], _stream(), small)
    assert ei.value.status == E.E_RESOURCE


@pytest.mark.parametrize("Hq,Hkv,hd", [(8, 2, 64), (8, 2, 128), (4, 4, 64), (4, 2, 16)])
def test_decode_attention_matches_oracle(E, Hq, Hkv, hd):
    dev = torch.device("cuda")
    lens = np.array([1, 16, 17, 255, 256, 257, 700, 1023], dtype=np.int32)
    B = len(lens)
    need = [(int(L) + 15) // 16 for L in lens]
    npages = sum(need) + 3
    rng = np.random.default_rng(5)
    perm = rng.permutation(npages).astype(np.int32)
    stride = max(need)
    tables = np.zeros((B, stride), dtype=np.int32)
    o = 0
    for b, n in enumerate(need):
        tables[b, :n] = perm[o:o + n]
        o += n
    pool = synth.make_kv_pool(1, npages, Hkv, hd, seed=6, device=dev)[0]
    # poison the slots past each request's length: they must never be read
    pool_ref = synth.to_bits(pool)
    for b, L in enumerate(lens):
        if L % 16:
            pool[int(tables[b, need[b] - 1]), :, :, L % 16:, :] = float("nan")
    q = torch.randn((B, Hq * hd), generator=torch.Generator(device=dev).manual_seed(7), device=dev).to(torch.bfloat16)
    out = torch.empty((B, Hq * hd), device=dev, dtype=torch.bfloat16)
    max_len = int(lens.max())
    scratch = torch.empty(E.lib.epara_decode_attention_scratch_bytes(B, Hq, hd, max_len), dtype=torch.uint8, device=dev)
    E.epara_decode_attention(q, pool, torch.as_tensor(lens, device=dev), torch.as_tensor(tables, device=dev), out,
                             Hq, Hkv, hd, max_len, scratch, _stream())
    torch.cuda.synchronize()
    qf = O.bf16_to_f64(synth.to_bits(q)).reshape(B, Hq, hd)
    for b, L in enumerate(lens):
        K, V = O.gather_kv(lambda l, pg: pool_ref[pg], 0, tables[b], int(L))
        ref = np.stack([O.attention(qf[b, h], K[h // (Hq // Hkv)], V[h // (Hq // Hkv)]) for h in range(Hq)])
        assert_close(out[b].reshape(Hq, hd), ref, what=f"decode attention b={b} L={L}")


@pytest.mark.parametrize("rows", [16, 100, 200, 1024])
def test_gelu_epilogue_sweep_through_identity_gemm(E, rows):
    """The device GELU over its whole range: x swept over [-8, 8] (every bf16 value of a fine grid) goes through a
    GEMM with the identity as weights, so the accumulator holds x exactly and the epilogue alone decides the
    output.  Bound: the fitted form's 2.6e-5, the hardware tanh's relative error 2^-11 scaled by 0.5 |x|
    (2.5e-4 |x|), and the rounding of the bf16 store (half an ulp: at most 2^-8 of the result).  The row counts select the
    weight-streaming kernel, the swapped-operand kernel, the one-CTA tile kernel and the tile-pair kernel."""
    dev = torch.device("cuda")
    K = N = 256
    x = torch.linspace(-8.0, 8.0, rows * K, device=dev).reshape(rows, K)
    x = x[:, torch.randperm(K, generator=torch.Generator(device=dev).manual_seed(rows), device=dev)].to(torch.bfloat16)
    W = torch.eye(N, K, device=dev).to(torch.bfloat16)
    C = torch.full((rows, N), float("nan"), device=dev, dtype=torch.bfloat16)
    prob = [{"A": x, "W": W, "C": C, "bias": None, "M": rows, "N": N, "K": K, "epilogue": E.EPI_GELU}]
    scratch = torch.empty(E.epara_gemm_scratch_bytes_for(prob), dtype=torch.uint8, device=dev)
    E.epara_grouped_gemm(prob, _stream(), scratch, impl=E.GEMM_TCGEN05)
    torch.cuda.synchronize()
    assert int(scratch[:4].view(torch.int32).item()) == 0
    xs = O.bf16_to_f64(synth.to_bits(x))
    ref = O.gelu(xs)
    got = to_f64(C)
    bound = 2.6e-5 + 2.5e-4 * np.abs(xs) + 2.0 ** -8 * np.abs(ref) + 1e-7
    bad = np.abs(got - ref) > bound
    assert not bad.any(), f"{int(bad.sum())} of {bad.size} outside the bound; worst excess " \
                          f"{float(np.max(np.abs(got - ref) - bound)):.3e} at x = {float(xs[np.unravel_index(np.argmax(np.abs(got - ref) - bound), xs.shape)])}"
