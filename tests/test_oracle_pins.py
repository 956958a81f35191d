"""Pins of the CPU oracle against things other than itself: brute force, closed forms,
invariants, special cases that reduce to library routines, and the paper's worked example."""
import math

import numpy as np
import pytest
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import synth


def bits(x):
    """fp values that are exactly representable in bf16 -> bit patterns."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    assert torch.equal(t.float(), torch.as_tensor(np.asarray(x, dtype=np.float32)))
    return synth.to_bits(t)


def rbits(shape, seed, std=1.0):
    g = torch.Generator().manual_seed(seed)
    return synth.to_bits((torch.randn(shape, generator=g) * std).to(torch.bfloat16))


# ------------------------------------------------------------------- bf16 codec
def test_bf16_decode_known_patterns():
    u = np.array([0x3F80, 0xBF80, 0x4000, 0x3F00, 0x0000, 0x4049, 0x7F80], dtype=np.uint16)
    got = O.bf16_to_f64(u)
    assert got.tolist()[:5] == [1.0, -1.0, 2.0, 0.5, 0.0]
    assert got[5] == 3.140625 and np.isinf(got[6])


def test_bf16_round_to_nearest_even():
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7: ties to even (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert O.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8 + 2.0 ** -12]))[0] == 0x3F81
    x = torch.randn(4096, generator=torch.Generator().manual_seed(1), dtype=torch.float64)
    ref = synth.to_bits(x.float().to(torch.bfloat16))
    assert np.array_equal(O.f64_to_bf16_bits(x.numpy()), ref)


# ------------------------------------------------------------------- P1 brute force
def test_linear_brute_force_tiny():
    x = np.array([1.0, -2.0, 3.0])
    W = np.array([[1.0, 0.0, 2.0], [0.0, -1.0, 1.0]])
    b = np.array([0.5, -0.5])
    # hand-expanded: [1*1 + 0 + 3*2 + .5, 2 + 3 - .5]
    assert O.linear(x, W, b).tolist() == [7.5, 4.5]
    # a transposed operand would fail this non-square case
    rng = np.random.default_rng(0)
    X = rng.integers(-3, 4, (4, 3)).astype(np.float64)
    Wm = rng.integers(-3, 4, (2, 3)).astype(np.float64)
    ref = [[sum(X[i, k] * Wm[j, k] for k in range(3)) for j in range(2)] for i in range(4)]
    assert O.linear(X, Wm).tolist() == ref


def test_mlp_brute_force_integer_weights():
    x = bits([1, 2, -1, 0.5])
    W0 = bits([[1, 0, 0, 2], [0, 1, 1, 0], [-1, 0, 2, 0]])
    b0 = bits([0.5, 0, -1])
    W1 = bits([[-1, -1, 2], [0.5, 0.5, 0]])
    b1 = bits([0, 1])
    h = [1 + 1 + 0.5, 2 - 1, -1 - 2 - 1]
    ge = [0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in h]
    ref = [-ge[0] - ge[1] + 2 * ge[2], 0.5 * ge[0] + 0.5 * ge[1] + 1]
    y, am = O.mlp_forward(x, [W0, W1], [b0, b1])
    assert np.allclose(y, ref, rtol=0, atol=1e-15)
    assert am == 1  # no activation after the last layer: ref[0] < 0 < ref[1]
    assert ref[0] < -3 and y[0] < -3


# ------------------------------------------------------------------- P2 / P3
def test_identity_and_zero_mlp():
    x = rbits((8,), 3)
    I = bits(np.eye(8))
    z = bits(np.zeros(8))
    y, _ = O.mlp_forward(x, [I], [z])
    assert np.array_equal(y, O.bf16_to_f64(x))           # single layer: no activation
    y2, _ = O.mlp_forward(x, [I, I], [z, z])
    xv = O.bf16_to_f64(x)
    ref = np.array([0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in xv])
    assert np.allclose(y2, ref, rtol=0, atol=1e-15)      # GELU between layers only
    y0, am = O.mlp_forward(z, [rbits((8, 8), 4), rbits((5, 8), 5)], [z, bits(np.zeros(5))])
    assert np.all(y0 == 0) and am == 0                   # GELU(0) = 0; ties -> lowest index


def test_gelu_values():
    # known values of the exact (erf) form; the tanh approximation differs in the 4th digit
    assert abs(O.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15
    assert abs(O.gelu(np.array([-1.0]))[0] + 0.15865525393145707) < 1e-15
    assert O.gelu(np.array([0.0]))[0] == 0.0
    x = torch.linspace(-6, 6, 101, dtype=torch.float64)
    assert np.allclose(O.gelu(x.numpy()), torch.nn.functional.gelu(x).numpy(), atol=1e-15)


def test_device_gelu_formula_stays_within_its_stated_bound_of_the_erf_form():
    """The CUDA epilogue evaluates GELU as 0.5 x (1 + tanh(x P(x^2))), P(t) = a + b t + c t^2 with t clamped at
    64 (csrc/common.cuh).  With an exact tanh that formula is within 2.6e-5 of the erf form for every x; the
    coefficients are read from the source file, so a change there is checked here."""
    import os
    import re
    src = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2511_00603_b200", "csrc",
                            "common.cuh")).read()
    body = src[src.index("float gelu_erf(float x)"):]
    body = body[:body.index("silu_f")]
    c2, c1 = [float(v) for v in re.search(r"fmaf\(t, (-?[0-9.e+-]+)f, (-?[0-9.e+-]+)f\)", body).groups()]
    c0 = float(re.search(r"fmaf\(t, p, (-?[0-9.e+-]+)f\)", body).group(1))
    assert abs(c0 - math.sqrt(2 / math.pi)) < 1e-3            # leading term of erf(x / sqrt 2) ~ tanh(sqrt(2/pi) x)
    x = np.linspace(-12.0, 12.0, 480001)
    t = np.minimum(x * x, 64.0)
    dev = 0.5 * x * (1.0 + np.tanh(x * (c0 + t * (c1 + t * c2))))
    err = np.abs(dev - O.gelu(x))
    assert err.max() <= 2.6e-5, err.max()
    assert err[np.abs(x) > 8].max() <= 1e-10                  # saturated on both sides: x or 0


def test_silu_values():
    assert abs(O.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16
    x = torch.linspace(-8, 8, 77, dtype=torch.float64)
    assert np.allclose(O.silu(x.numpy()), torch.nn.functional.silu(x).numpy(), atol=1e-15)


# ------------------------------------------------------------------- P6 norms
def test_layernorm_closed_forms():
    d = 64
    g = np.linspace(0.5, 1.5, d)
    b = np.linspace(-1, 1, d)
    assert np.allclose(O.layernorm(np.full(d, 3.7), g, b), b, atol=1e-12)   # constant -> beta
    x = np.random.default_rng(0).normal(2.0, 3.0, d)
    y = O.layernorm(x, np.ones(d), np.zeros(d), eps=1e-6)
    assert abs(y.mean()) < 1e-13
    var = x.var()
    assert abs(y.var() - var / (var + 1e-6)) < 1e-12
    xt = torch.tensor(x)
    ref = torch.nn.functional.layer_norm(xt, (d,), torch.tensor(g), torch.tensor(b), eps=1e-6).numpy()
    assert np.allclose(O.layernorm(x, g, b), ref, atol=1e-13)


def test_rmsnorm_closed_forms():
    d = 32
    c = 2.5
    x = np.array([c if i % 2 else -c for i in range(d)])
    y = O.rmsnorm(x, np.ones(d), eps=1e-5)
    assert np.allclose(y, x / math.sqrt(c * c + 1e-5), atol=1e-15)
    assert np.all(O.rmsnorm(np.zeros(d), np.ones(d)) == 0)
    xr = np.random.default_rng(1).normal(size=d)
    g = np.linspace(0.5, 2, d)
    ref = torch.nn.functional.rms_norm(torch.tensor(xr), (d,), torch.tensor(g), eps=1e-5).numpy()
    assert np.allclose(O.rmsnorm(xr, g), ref, atol=1e-14)


# ------------------------------------------------------------------- P8 RoPE
def test_rope_properties():
    rng = np.random.default_rng(2)
    hd = 64
    q, k = rng.normal(size=hd), rng.normal(size=hd)
    assert np.array_equal(O.rope(q, 0), q)                                  # position 0 = identity
    r = O.rope(q, 1234)
    assert np.allclose(r[0::2] ** 2 + r[1::2] ** 2, q[0::2] ** 2 + q[1::2] ** 2, atol=1e-12)
    assert abs(O.rope(q, 77) @ O.rope(k, 77) - q @ k) < 1e-11
    assert abs(O.rope(q, 300) @ O.rope(k, 100) - O.rope(q, 200) @ k) < 1e-10  # relative position
    # explicit angle of pair j at position p: p * 10000^(-2j/hd); the last pair turns slowest
    p = 5
    j = hd // 2 - 1
    th = p * 10000.0 ** (-2.0 * j / hd)
    e = np.zeros(hd)
    e[2 * j] = 1.0
    rr = O.rope(e, p)
    assert abs(rr[2 * j] - math.cos(th)) < 1e-15 and abs(rr[2 * j + 1] - math.sin(th)) < 1e-15
    e0 = np.zeros(hd)
    e0[0] = 1.0
    r0 = O.rope(e0, p)
    assert abs(r0[0] - math.cos(5.0)) < 1e-15 and abs(r0[1] - math.sin(5.0)) < 1e-15


# ------------------------------------------------------------------- P4 / P5 / P11 attention
def test_attention_single_token_and_uniform():
    rng = np.random.default_rng(3)
    q = rng.normal(size=16)
    V = rng.normal(size=(7, 16))
    assert np.allclose(O.attention(q, rng.normal(size=(1, 16)), V[:1]), V[0], atol=0)
    K = np.tile(rng.normal(size=(1, 16)), (7, 1))
    assert np.allclose(O.attention(q, K, V), V.mean(axis=0), atol=1e-14)    # equal keys -> mean of V
    K2 = rng.normal(size=(7, 16))
    K2[4] = q * 1e3                                                          # one dominant key
    assert np.allclose(O.attention(q, K2, V), V[4], atol=1e-12)


def test_attention_scale_and_library():
    rng = np.random.default_rng(4)
    Q, K, V = rng.normal(size=(5, 8)), rng.normal(size=(9, 8)), rng.normal(size=(9, 8))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(Q)[None], torch.tensor(K)[None], torch.tensor(V)[None])[0].numpy()
    assert np.allclose(O.attention(Q, K, V), ref, atol=1e-13)
    # brute force with the 1/sqrt(hd) scale written out
    s = [[sum(Q[i, c] * K[t, c] for c in range(8)) / math.sqrt(8) for t in range(9)] for i in range(5)]
    for i in range(5):
        w = [math.exp(v - max(s[i])) for v in s[i]]
        o = [sum(w[t] * V[t, c] for t in range(9)) / sum(w) for c in range(8)]
        assert np.allclose(O.attention(Q, K, V)[i], o, atol=1e-14)


def test_softmax_shift_sum_and_split_merge():
    rng = np.random.default_rng(5)
    s = rng.normal(size=(3, 50)) * 5
    p = O.softmax(s)
    assert np.allclose(p.sum(-1), 1, atol=1e-15)
    assert np.allclose(O.softmax(s + 123.0), p, atol=1e-14)
    # attention over a split key set merged by log-sum-exp equals the unsplit result
    q, K, V = rng.normal(size=8), rng.normal(size=(50, 8)), rng.normal(size=(50, 8))
    parts = []
    for a, b in [(0, 13), (13, 14), (14, 50)]:
        sc = K[a:b] @ q / math.sqrt(8)
        m = sc.max()
        w = np.exp(sc - m)
        parts.append((m, w.sum(), w @ V[a:b]))
    M = max(m for m, _, _ in parts)
    l = sum(ls * math.exp(m - M) for m, ls, _ in parts)
    o = sum(ov * math.exp(m - M) for m, _, ov in parts) / l
    assert np.allclose(O.attention(q, K, V), o, atol=1e-14)


def test_argmax_lowest_index_on_ties():
    assert O.argmax_lowest(np.array([1.0, 3.0, 3.0, 2.0])) == 1
    assert O.argmax_lowest(np.zeros(9)) == 0


# ------------------------------------------------------------------- ViT
def test_patchify_index_rule():
    img = np.arange(3 * 32 * 48, dtype=np.float64).reshape(3, 32, 48)
    P = O.patchify(img, 16)
    assert P.shape == (6, 768)
    for (i, j, c, u, v) in [(0, 0, 0, 0, 0), (1, 2, 2, 15, 3), (0, 1, 1, 7, 9), (1, 0, 0, 0, 15)]:
        assert P[i * 3 + j, c * 256 + u * 16 + v] == img[c, 16 * i + u, 16 * j + v]
    t = torch.tensor(img)[None]
    ref = torch.nn.functional.unfold(t, kernel_size=16, stride=16)[0].T.numpy()
    assert np.array_equal(P, ref)


def _torch_bf16(t):
    """Storage rounding by the library's own bf16 cast (fp64 -> fp32 -> bf16 -> fp64)."""
    return t.float().to(torch.bfloat16).double()


def _torch_vit(img, p, rnd=lambda t: t):
    """Independent fp64 evaluation with torch library routines (conv patch embedding,
    layer_norm, scaled_dot_product_attention, gelu).  rnd is applied to every tensor the device
    contract stores as bf16 (identity: the unrounded evaluation)."""
    F = torch.nn.functional
    f = lambda t: t.double()
    d, H, ps = p["d"], p["n_heads"], p["patch"]
    x = rnd(F.conv2d(f(img)[None], f(p["W_pe"]).reshape(d, 3, ps, ps), f(p["b_pe"]), stride=ps))
    x = x.flatten(2).transpose(1, 2)
    z = torch.cat([f(p["cls"])[None, None], x], dim=1) + f(p["pos"])[None]
    T = z.shape[1]
    for L in p["layers"]:
        h = rnd(F.layer_norm(z, (d,), f(L["ln1_g"]), f(L["ln1_b"]), eps=1e-6))
        qkv = rnd(F.linear(h, f(L["Wqkv"]), f(L["bqkv"]))).reshape(1, T, 3, H, d // H).permute(2, 0, 3, 1, 4)
        o = rnd(F.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2]).transpose(1, 2).reshape(1, T, d))
        z = z + F.linear(o, f(L["Wo"]), f(L["bo"]))
        h = rnd(F.layer_norm(z, (d,), f(L["ln2_g"]), f(L["ln2_b"]), eps=1e-6))
        z = z + F.linear(rnd(F.gelu(F.linear(h, f(L["W1"]), f(L["b1"])))), f(L["W2"]), f(L["b2"]))
    c = rnd(F.layer_norm(z[0, 0], (d,), f(p["lnf_g"]), f(p["lnf_b"]), eps=1e-6))
    return rnd(F.linear(c, f(p["Whead"]), f(p["bhead"]))).numpy()


def test_vit_matches_torch_library_evaluation():
    p = synth.make_vit(d=64, n_layers=2, n_heads=4, mlp=128, n_cls=10, seed=7, img=64, std=0.2, perturb=0.3)
    img = synth.make_images(1, seed=8, img=64)[0]
    logits, am, _ = O.vit_forward(synth.to_bits(img), synth.bits_view(p))
    ref = _torch_vit(img, p)
    assert np.allclose(logits, ref, rtol=1e-10, atol=1e-12)
    assert am == int(ref.argmax())


def test_vit_zero_image_depends_only_on_cls_pos_and_biases():
    p = synth.make_vit(d=32, n_layers=1, n_heads=2, mlp=64, n_cls=5, seed=9, img=32)
    z = np.zeros((3, 32, 32), dtype=np.uint16)
    a, _, _ = O.vit_forward(z, synth.bits_view(p))
    p2 = dict(p)
    p2["W_pe"] = p["W_pe"] * 3.0          # patch weights cannot matter for a zero image
    b, _, _ = O.vit_forward(z, synth.bits_view(p2))
    assert np.array_equal(a, b)


# ------------------------------------------------------------------- decoder
def _pool_fetch(pool_bits):
    return lambda layer, page: pool_bits[layer, page]


def _torch_decoder(token, L, table, pool, p, rnd=lambda t: t):
    """Independent fp64 evaluation: contiguous K/V rebuilt with torch indexing, complex-number
    RoPE, library rms_norm / sdpa / silu.  rnd is applied to every tensor the device contract stores
    as bf16 (identity: the unrounded evaluation)."""
    F = torch.nn.functional
    f = lambda t: t.double()
    Hq, Hkv, hd = p["n_q_heads"], p["n_kv_heads"], p["head_dim"]
    x = f(p["Emb"][token])
    ang = L * (10000.0 ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd))
    rot = torch.polar(torch.ones_like(ang), ang)

    def rope(t):
        c = torch.view_as_complex(t.reshape(-1, hd // 2, 2).contiguous()) * rot
        return torch.view_as_real(c).reshape(-1, hd)

    tb = torch.as_tensor(table.astype(np.int64))
    for li, Lw in enumerate(p["layers"]):
        h = rnd(F.rms_norm(x, (p["d"],), f(Lw["g1"]), eps=1e-5))
        q = rnd(rope(rnd(F.linear(h, f(Lw["Wq"]))).reshape(Hq, hd)))
        k = rnd(rope(rnd(F.linear(h, f(Lw["Wk"]))).reshape(Hkv, hd)))
        v = rnd(F.linear(h, f(Lw["Wv"]))).reshape(Hkv, hd)
        pages = f(pool[li][tb])                               # [n, 2, Hkv, 16, hd]
        Kc = pages[:, 0].permute(1, 0, 2, 3).reshape(Hkv, -1, hd)[:, :L]
        Vc = pages[:, 1].permute(1, 0, 2, 3).reshape(Hkv, -1, hd)[:, :L]
        K = torch.cat([Kc, k[:, None]], dim=1).repeat_interleave(Hq // Hkv, dim=0)
        V = torch.cat([Vc, v[:, None]], dim=1).repeat_interleave(Hq // Hkv, dim=0)
        o = rnd(F.scaled_dot_product_attention(q[:, None], K, V).reshape(-1))
        x = x + F.linear(o, f(Lw["Wo"]))
        h = rnd(F.rms_norm(x, (p["d"],), f(Lw["g2"]), eps=1e-5))
        x = x + F.linear(rnd(F.silu(F.linear(h, f(Lw["Wg"]))) * F.linear(h, f(Lw["Wu"]))), f(Lw["Wd"]))
    return rnd(F.linear(rnd(F.rms_norm(x, (p["d"],), f(p["gf"]), eps=1e-5)), f(p["Wlm"]))).numpy()


def _small_decoder(seed=11, perturb=0.2):
    return synth.make_decoder(d=64, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=50,
                              seed=seed, std=0.2, perturb=perturb)


def test_decoder_matches_torch_library_evaluation():
    p = _small_decoder()
    toks, lens, tables, npages = synth.make_decode_batch(3, 5, 40, 50, seed=12)
    pool = synth.make_kv_pool(2, npages, 2, 16, seed=13)
    pb = synth.to_bits(pool)
    for i in range(3):
        r = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], _pool_fetch(pb), synth.bits_view(p))
        ref = _torch_decoder(int(toks[i]), int(lens[i]), tables[i], pool, p)
        assert np.allclose(r["logits"], ref, rtol=1e-10, atol=1e-12)
        assert r["argmax"] == int(ref.argmax())
        assert r["appended"][0]["page"] == int(tables[i][lens[i] // 16])
        assert r["appended"][0]["slot"] == int(lens[i]) % 16


def test_decoder_empty_cache_attention_is_v():
    """kv_len = 0: the only key is the new token, so attention returns v (rope at 0 = identity)
    and the layer reduces to x + Wo v_rep + FFN."""
    p = _small_decoder(perturb=0.0)
    pv = synth.bits_view(p)
    D = O.bf16_to_f64
    r = O.decoder_step(3, 0, np.array([0], dtype=np.int32), lambda l, pg: (_ for _ in ()).throw(AssertionError), pv)
    x = D(pv["Emb"][3])
    for L in pv["layers"]:
        h = O.rmsnorm(x, D(L["g1"]))
        v = (D(L["Wv"]) @ h).reshape(2, 16)
        o = np.repeat(v, 2, axis=0).reshape(-1)       # q head hq uses kv head hq // 2
        x = x + D(L["Wo"]) @ o
        h = O.rmsnorm(x, D(L["g2"]))
        x = x + D(L["Wd"]) @ (O.silu(D(L["Wg"]) @ h) * (D(L["Wu"]) @ h))
    ref = D(pv["Wlm"]) @ O.rmsnorm(x, D(pv["gf"]))
    assert np.allclose(r["logits"], ref, rtol=1e-12, atol=1e-14)


def test_decoder_zero_embedding_row_gives_zero_logits():
    p = _small_decoder(perturb=0.0)
    p["Emb"][7] = 0
    toks, lens, tables, npages = synth.make_decode_batch(1, 20, 20, 50, seed=14)
    pool = synth.to_bits(synth.make_kv_pool(2, npages, 2, 16, seed=15))
    r = O.decoder_step(7, 20, tables[0], _pool_fetch(pool), synth.bits_view(p))
    # RMSNorm(0) = 0 -> q = k = v = 0 -> scores uniform -> attention = mean of cached V (not 0);
    # so only layer-0's projections vanish.  With Wo = 0 as well the whole stream stays 0.
    for L in p["layers"]:
        L["Wo"].zero_()
    r = O.decoder_step(7, 20, tables[0], _pool_fetch(pool), synth.bits_view(p))
    assert np.all(r["logits"] == 0) and r["argmax"] == 0


def test_decoder_paging_invariance_and_gqa():
    p = _small_decoder()
    pv = synth.bits_view(p)
    toks, lens, tables, npages = synth.make_decode_batch(2, 30, 45, 50, seed=16)
    pool = synth.to_bits(synth.make_kv_pool(2, npages, 2, 16, seed=17))
    base = O.decoder_step(int(toks[0]), int(lens[0]), tables[0], _pool_fetch(pool), pv)
    # permute physical pages together with the table: nothing changes
    perm = np.random.default_rng(0).permutation(npages)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(npages)
    pool2 = pool[:, perm]
    r2 = O.decoder_step(int(toks[0]), int(lens[0]), inv[tables[0]].astype(np.int32), _pool_fetch(pool2), pv)
    assert np.array_equal(base["logits"], r2["logits"])
    # batch invariance: another request's pages and tokens cannot matter
    pool3 = pool.copy()
    pool3[:, tables[1]] = 0
    r3 = O.decoder_step(int(toks[0]), int(lens[0]), tables[0], _pool_fetch(pool3), pv)
    assert np.array_equal(base["logits"], r3["logits"])
    # slots at and beyond kv_len in the last page are never read
    pool4 = pool.copy()
    L0 = int(lens[0])
    pool4[:, tables[0][L0 // 16], :, :, L0 % 16:, :] = 0x7FC0  # NaN
    r4 = O.decoder_step(int(toks[0]), L0, tables[0], _pool_fetch(pool4), pv)
    assert np.array_equal(base["logits"], r4["logits"])


def test_gqa_query_heads_read_their_groups_kv_head():
    """GQA against a model without it: the decoder with 4 query heads over 2 KV heads must equal the
    multi-head decoder (4 KV heads) whose K and V projections and cache hold, for query head h, a copy of
    KV head h // 2.  A wrong head-to-group mapping (h % 2, say) fails: the two KV heads differ."""
    p = _small_decoder(seed=23)
    toks, lens, tables, npages = synth.make_decode_batch(2, 20, 45, 50, seed=24)
    pool = synth.make_kv_pool(2, npages, 2, 16, seed=25)
    wide = {k: v for k, v in p.items()}
    wide["n_kv_heads"] = 4
    wide["layers"] = []
    for L in p["layers"]:
        W = dict(L)
        for name in ("Wk", "Wv"):
            W[name] = L[name].reshape(2, 16, -1).repeat_interleave(2, dim=0).reshape(64, -1).contiguous()
        wide["layers"].append(W)
    pool_wide = pool.repeat_interleave(2, dim=3).contiguous()          # [layer, page, 2, Hkv -> 4, 16, hd]
    for i in range(2):
        a = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], _pool_fetch(synth.to_bits(pool)), synth.bits_view(p))
        b = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], _pool_fetch(synth.to_bits(pool_wide)), synth.bits_view(wide))
        assert np.allclose(a["logits"], b["logits"], rtol=1e-12, atol=1e-14)
        # and the mapping matters for this input: swapping the two KV heads changes the answer
        swapped = synth.to_bits(pool.flip(3).contiguous())
        c = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], _pool_fetch(swapped), synth.bits_view(p))
        assert np.max(np.abs(a["logits"] - c["logits"])) > 1e-3


def test_bf16_storage_mode_matches_torch_evaluation_with_library_casts():
    """Mode B (bf16 rounding at the device contract's storage points) is what the decoder parity tests
    compare with.  It is pinned against the independent torch evaluation with the library's own bf16 cast at
    those points: norm outputs, q / k / v before and after the rotation, attention output, SwiGLU output,
    logits; the residual stream stays unrounded.  (An evaluation that rounded somewhere else, or not at all,
    differs by about 1e-3 relative; agreement here is to 1e-9.)"""
    p = _small_decoder(seed=26)
    toks, lens, tables, npages = synth.make_decode_batch(3, 5, 40, 50, seed=27)
    pool = synth.make_kv_pool(2, npages, 2, 16, seed=28)
    pb = synth.to_bits(pool)
    for i in range(3):
        r = O.decoder_step(int(toks[i]), int(lens[i]), tables[i], _pool_fetch(pb), synth.bits_view(p), round_bf16=True)
        ref = _torch_decoder(int(toks[i]), int(lens[i]), tables[i], pool, p, rnd=_torch_bf16)
        assert np.allclose(r["logits"], ref, rtol=1e-9, atol=1e-12)
        unrounded = _torch_decoder(int(toks[i]), int(lens[i]), tables[i], pool, p)
        assert np.max(np.abs(unrounded - ref)) > 1e-5
    pv = synth.make_vit(d=64, n_layers=2, n_heads=4, mlp=128, n_cls=10, seed=29, img=64, std=0.2, perturb=0.3)
    img = synth.make_images(1, seed=30, img=64)[0]
    logits, am, _ = O.vit_forward(synth.to_bits(img), synth.bits_view(pv), round_bf16=True)
    assert np.allclose(logits, _torch_vit(img, pv, rnd=_torch_bf16), rtol=1e-9, atol=1e-12)


def test_mode_b_is_close_to_mode_a():
    p = _small_decoder()
    toks, lens, tables, npages = synth.make_decode_batch(1, 30, 30, 50, seed=18)
    pool = synth.to_bits(synth.make_kv_pool(2, npages, 2, 16, seed=19))
    a = O.decoder_step(int(toks[0]), 30, tables[0], _pool_fetch(pool), synth.bits_view(p))["logits"]
    b = O.decoder_step(int(toks[0]), 30, tables[0], _pool_fetch(pool), synth.bits_view(p), round_bf16=True)["logits"]
    rho = math.sqrt(np.mean(a * a))
    assert 0 < np.max(np.abs(a - b)) < 2e-2 * rho


@pytest.mark.parametrize("n_layers,l2_lo,l2_hi,max_hi", [(1, 2e-3, 1.2e-2, 5e-2), (2, 3e-3, 1.5e-2, 6e-2), (16, 8e-3, 4e-2, 1.5e-1)])
def test_mode_a_vs_mode_b_gap_at_the_1b_layer_shapes(n_layers, l2_lo, l2_hi, max_hi):
    """How far apart two correct evaluations of one decode request are at the 1B decoder's layer shapes
    (d 2048, 32 / 8 heads of 64, FFN 8192, vocab 32000): the unrounded fp64 evaluation against the one that
    rounds to bf16 at the storage points.  This gap, not a kernel, is why a deep random-weight decoder
    cannot meet 2e-2 element-wise against the unrounded evaluation; the GPU tests bound the device by a
    fraction of each request's own gap and rely on the ceilings checked here.  Measured (seed 2, KV length
    600): relative L2 5.9e-3 / 7.3e-3 / 1.8e-2 and worst element 2.5e-2 / 2.9e-2 / 7.9e-2 of the tensor's
    scale at 1 / 2 / 16 layers."""
    from paper_2511_00603_b200 import configs
    from tests.parity import DEEP_GAP_L2_CEIL, DEEP_GAP_MAX_CEIL, max_rel_err, rel_l2_err
    cfg = dict(configs.DEC_1B, n_layers=n_layers)
    p = synth.bits_view(synth.make_decoder(seed=2, **cfg))
    toks, lens, tables, npages = synth.make_decode_batch(1, 600, 600, cfg["vocab"], seed=31)
    pool = synth.to_bits(synth.make_kv_pool(n_layers, npages, cfg["n_kv_heads"], cfg["head_dim"], seed=32))
    a = O.decoder_step(int(toks[0]), 600, tables[0], _pool_fetch(pool), p)["logits"]
    b = O.decoder_step(int(toks[0]), 600, tables[0], _pool_fetch(pool), p, round_bf16=True)["logits"]
    l2, mx = rel_l2_err(a, b), max_rel_err(a, b)
    print(f"1B layer shapes, {n_layers} layers: mode A vs mode B relative L2 {l2:.3e}, max relative {mx:.3e}")
    assert l2_lo <= l2 <= l2_hi and mx <= max_hi
    assert l2 <= DEEP_GAP_L2_CEIL and mx <= DEEP_GAP_MAX_CEIL
    if n_layers >= 2:
        assert mx > 2e-2          # the strict element-wise reading is out of reach for any implementation


# ------------------------------------------------------------------- prefill
class _GrowingCache:
    """A paged cache as bf16 bits that decode steps append to: fetch(layer, page) serves the oracle."""

    def __init__(self, pool_bits):
        self.pool = pool_bits.copy()

    def fetch(self, layer, page):
        return self.pool[layer, page]

    def append(self, layer, page, slot, k, v):
        self.pool[layer, page, 0, :, slot, :] = O.f64_to_bf16_bits(k)
        self.pool[layer, page, 1, :, slot, :] = O.f64_to_bf16_bits(v)


def test_prefill_equals_successive_decode_steps_on_a_growing_cache():
    """The identity that defines prefill: feeding the chunk's tokens one at a time through decoder_step, each
    step's k, v stored in the cache before the next, gives the same appended k, v, residuals and final
    logits.  With bf16 storage (mode B) the cache holds exactly what was appended, so the identity is exact
    up to summation order; both a fresh prompt (kv_len 0) and a chunk after 21 cached tokens."""
    p = synth.bits_view(_small_decoder(seed=40))
    for kv0, n in [(0, 9), (21, 14)]:
        toks, lens, tables, npages = synth.make_decode_batch(1, kv0 + n, kv0 + n, 50, seed=41 + kv0)
        pool = synth.to_bits(synth.make_kv_pool(2, npages, 2, 16, seed=42))
        tokens = [int(t) for t in np.random.default_rng(43).integers(0, 50, n)]
        pre = O.decoder_prefill(tokens, kv0, tables[0], _pool_fetch(pool), p, round_bf16=True)
        cache = _GrowingCache(pool)
        for t, tok in enumerate(tokens):
            r = O.decoder_step(tok, kv0 + t, tables[0], cache.fetch, p, round_bf16=True)
            for l, ap in enumerate(r["appended"]):
                assert np.allclose(ap["k"], pre["appended"][l]["k"][t], rtol=1e-12, atol=1e-14)
                assert np.allclose(ap["v"], pre["appended"][l]["v"][t], rtol=1e-12, atol=1e-14)
                cache.append(l, ap["page"], ap["slot"], ap["k"], ap["v"])
            for l in range(3):
                assert np.allclose(r["residual"][l], pre["residual"][l][t], rtol=1e-11, atol=1e-13)
        assert np.allclose(r["logits"], pre["logits"], rtol=1e-11, atol=1e-13)
        assert r["argmax"] == pre["argmax"]


def test_prefill_is_causal_and_its_first_token_sees_only_itself():
    p = synth.bits_view(_small_decoder(seed=44, perturb=0.0))
    table = np.arange(2, dtype=np.int32)
    nofetch = lambda l, pg: (_ for _ in ()).throw(AssertionError("no cached token exists"))
    a = O.decoder_prefill([5, 17, 3, 8], 0, table, nofetch, p)
    # changing a later token leaves every earlier token's k, v and residual untouched
    b = O.decoder_prefill([5, 17, 30, 41], 0, table, nofetch, p)
    for l in range(2):
        assert np.array_equal(a["appended"][l]["k"][:2], b["appended"][l]["k"][:2])
        assert np.array_equal(a["residual"][l + 1][:2], b["residual"][l + 1][:2])
        assert not np.array_equal(a["residual"][l + 1][3], b["residual"][l + 1][3])
    # the first token attends to itself only: its attention output is its own v (closed form, as for an empty cache)
    one = O.decoder_step(5, 0, table, nofetch, p)
    assert np.allclose(a["residual"][2][0], one["residual"][2], rtol=1e-13, atol=1e-15)
    # and a prompt of one token is a decode step
    assert np.array_equal(O.decoder_prefill([5], 0, table, nofetch, p)["logits"], one["logits"])


def test_prefill_matches_a_causal_torch_evaluation():
    """Independent route: all tokens at once with the library's causal scaled_dot_product_attention."""
    F = torch.nn.functional
    pt = _small_decoder(seed=45)
    p = synth.bits_view(pt)
    n, hd, Hq, Hkv, d = 11, 16, 4, 2, 64
    tokens = [int(t) for t in np.random.default_rng(46).integers(0, 50, n)]
    got = O.decoder_prefill(tokens, 0, np.arange(1, dtype=np.int32), None, p)
    f = lambda t: t.double()
    x = f(pt["Emb"][torch.tensor(tokens)])
    pos = torch.arange(n, dtype=torch.float64)[:, None]
    ang = pos * (10000.0 ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd))[None]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]                       # [n, 1, hd/2]

    def rope(t):                                                                  # t [n, H, hd]
        c = torch.view_as_complex(t.reshape(n, -1, hd // 2, 2).contiguous()) * rot
        return torch.view_as_real(c).reshape(n, -1, hd)

    for Lw in pt["layers"]:
        h = F.rms_norm(x, (d,), f(Lw["g1"]), eps=1e-5)
        q = rope(F.linear(h, f(Lw["Wq"])).reshape(n, Hq, hd)).transpose(0, 1)
        k = rope(F.linear(h, f(Lw["Wk"])).reshape(n, Hkv, hd)).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
        v = F.linear(h, f(Lw["Wv"])).reshape(n, Hkv, hd).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
        o = F.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(0, 1).reshape(n, -1)
        x = x + F.linear(o, f(Lw["Wo"]))
        h = F.rms_norm(x, (d,), f(Lw["g2"]), eps=1e-5)
        x = x + F.linear(F.silu(F.linear(h, f(Lw["Wg"]))) * F.linear(h, f(Lw["Wu"])), f(Lw["Wd"]))
    ref = F.linear(F.rms_norm(x[-1], (d,), f(pt["gf"]), eps=1e-5), f(pt["Wlm"])).numpy()
    assert np.allclose(got["logits"], ref, rtol=1e-10, atol=1e-12)


# ------------------------------------------------------------------- host policy
def test_eq4_eq5_and_goodput_example():
    assert O.dp_group_count(97, 49) == 2 and O.dp_group_count(98, 49) == 2 and O.dp_group_count(99, 49) == 3
    assert O.inter_request_count(256, 8) == 32 and O.inter_request_count(4, 8) == 0
    assert O.inter_request_count(10, 4) == 2
    # worked example in the paper's Section 3.3: 120 frames, 60 fps required, 30 fps achieved -> 60
    line = open(__file__.replace("test_oracle_pins.py", "golden/fs_goodput_example.txt")).read().split("\n")
    vals = [float(v) for v in line[-2].split()]
    assert O.fs_satisfied(vals[0], vals[1], vals[2]) == vals[3] == 60.0
    assert O.fs_satisfied(120, 60, 90) == 120


def _q(*items):
    return [{"ticket": t, "deadline_ns": d, "stream": s} for (t, d, s) in items]


def test_admission_rules():
    # timeout rule, then oldest-first up to the cap
    q = _q((1, 50, 0), (2, 0, 0), (3, 200, 0), (4, 100, 0), (5, 0, 0))
    assert O.admit(q, now_ns=100, cap=2) == ([2, 3], [1])      # deadline == now is still live
    assert O.admit(q, now_ns=101, cap=9) == ([2, 3, 5], [1, 4])
    # MF: cap 4, mf 2 -> 2 streams, identical frame count = min(2, fewest waiting)
    q = _q((1, 0, 7), (2, 0, 8), (3, 0, 7), (4, 0, 9), (5, 0, 7), (6, 0, 8))
    assert O.admit(q, 0, cap=4, mf_max=2) == ([1, 3, 2, 6], [])
    q = _q((1, 0, 7), (2, 0, 8), (3, 0, 7), (4, 0, 9), (5, 0, 7))
    assert O.admit(q, 0, cap=4, mf_max=2) == ([1, 2], [])       # stream 8 has one frame -> f = 1
    assert O.admit(q, 0, cap=1, mf_max=2) == ([], [])           # Eq. 5: floor(1/2) = 0 streams
