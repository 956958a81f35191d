"""Plain fp64 CPU oracle for one categorized serving step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of
what one serving step computes.  It shares no code with the CUDA library, never
imports it, and is imported only by the tests, the smoke check and the CPU-baseline
leg of the benchmark.  The product path never calls it.

What the step is (paper Section 3.1): on one GPU the allocator combines batching
(BS: several tasks of one service in a batch), multi-task (MT: tasks of different
services at once) and multi-frame (MF: equal frame counts from homogeneous streams)
for the two "<1 GPU" categories.  The paper treats the model execution itself as a
profiled latency; the forward passes below are therefore the textbook definitions
of the three model families the workloads name (GELU MLP, ViT encoder,
Llama-style decoder step over a paged KV cache), evaluated per request, in fp64,
with no intermediate rounding ("mode A").  `round_bf16=True` ("mode B") rounds to
bf16 at the tensor-storage points of the device contract and exists only to tell
"kernel wrong" from "storage noise".

Every request is computed on its own: a request's result cannot depend on which
other requests or models share its step (batch invariance).

Weights, inputs and the KV pool arrive as raw bf16 bit patterns (numpy uint16);
token ids, block tables and lengths as integers.

Parity pins (tests/test_oracle_pins.py): brute-force tiny matmuls, identity weights,
zero inputs, single-token attention equals V, uniform attention equals mean(V),
norm closed forms, RoPE relative-position property, GQA and paging invariances,
softmax shift invariance and split/merge, cross-check of every family against an
independent fp64 torch evaluation; the prefill against successive decode steps on a growing
cache, a causal torch evaluation, and causality itself (a later token cannot change an earlier one).  The host-logic functions (admission, Eq. 4,
Eq. 5, goodput rule) are pinned by the paper's worked example (120 frames,
60 fps required, 30 fps achieved -> 60 satisfied) and by hand-computed cases.
No function here is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf as _erf

PAGE = 16  # tokens per KV page (workload definition)


# --------------------------------------------------------------------------- bf16
def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> fp64: the 16 bits are the top half of an IEEE fp32."""
    u = np.ascontiguousarray(u16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 -> bf16 bits, round to nearest even (mode B storage points)."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def _store(x: np.ndarray, round_bf16: bool) -> np.ndarray:
    return bf16_to_f64(f64_to_bf16_bits(x)) if round_bf16 else x


# ------------------------------------------------------------------ elementary ops
def gelu(x: np.ndarray) -> np.ndarray:
    """Exact GELU, 0.5 x (1 + erf(x / sqrt 2))."""
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def softmax(s: np.ndarray) -> np.ndarray:
    """Softmax over the last axis."""
    e = np.exp(s - np.max(s, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def layernorm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """LayerNorm over the last axis with the biased variance."""
    mu = np.mean(x, axis=-1, keepdims=True)
    var = np.mean((x - mu) ** 2, axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * gamma + beta


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * g


def linear(x: np.ndarray, W: np.ndarray, b: Optional[np.ndarray] = None) -> np.ndarray:
    """y = x W^T (+ b); W is [out_features, in_features]."""
    y = x @ W.T
    return y if b is None else y + b


def argmax_lowest(v: np.ndarray) -> int:
    """Index of the maximum; the lowest index wins a tie."""
    return int(np.argmax(v))  # numpy returns the first maximal element


def rope(x: np.ndarray, pos: int, base: float = 10000.0) -> np.ndarray:
    """Rotary embedding of one head vector x[hd] at position pos.

    Pairs are interleaved, (x[2j], x[2j+1]), rotated by the angle pos * base^(-2j/hd).
    """
    hd = x.shape[-1]
    j = np.arange(hd // 2, dtype=np.float64)
    ang = float(pos) * base ** (-2.0 * j / hd)
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * c - x[..., 1::2] * s
    out[..., 1::2] = x[..., 0::2] * s + x[..., 1::2] * c
    return out


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """softmax(q K^T / sqrt(hd)) V for q[..., hd], K[T, hd], V[T, hd]."""
    hd = q.shape[-1]
    return softmax((q @ K.T) / math.sqrt(hd)) @ V


# ------------------------------------------------------------------------- MLP
def mlp_forward(x_bits: np.ndarray, Ws: Sequence[np.ndarray], bs: Sequence[np.ndarray],
                round_bf16: bool = False) -> Tuple[np.ndarray, int]:
    """One request through a GELU MLP: GELU between layers, none after the last.

    x_bits: uint16 [K0]; Ws[l]: uint16 [N_l, K_l]; bs[l]: uint16 [N_l].
    Returns (output vector fp64 [N_last], argmax).
    """
    y = bf16_to_f64(x_bits)
    n = len(Ws)
    for l in range(n):
        y = linear(y, bf16_to_f64(Ws[l]), bf16_to_f64(bs[l]))
        if l + 1 < n:
            y = gelu(y)
        y = _store(y, round_bf16)
    return y, argmax_lowest(y)


# ------------------------------------------------------------------------- ViT
def patchify(img: np.ndarray, patch: int = 16) -> np.ndarray:
    """[C, H, W] -> [H/p * W/p, C*p*p]; patch (i, j) row-major, element c*p*p + u*p + v."""
    C, H, W = img.shape
    gh, gw = H // patch, W // patch
    out = np.empty((gh * gw, C * patch * patch), dtype=img.dtype)
    for i in range(gh):
        for j in range(gw):
            out[i * gw + j] = img[:, i * patch:(i + 1) * patch, j * patch:(j + 1) * patch].reshape(-1)
    return out


def vit_forward(img_bits: np.ndarray, p: Dict, round_bf16: bool = False) -> Tuple[np.ndarray, int, np.ndarray]:
    """One image through a pre-LN ViT encoder and a linear classification head.

    img_bits: uint16 [3, H, W].  p holds bf16-bit arrays: W_pe [d, 3*16*16], b_pe, cls [d],
    pos [T, d], layers[l] = {ln1_g, ln1_b, Wqkv [3d, d] (rows q;k;v), bqkv, Wo, bo, ln2_g,
    ln2_b, W1 [mlp, d], b1, W2 [d, mlp], b2}, lnf_g, lnf_b, Whead [n_cls, d], bhead, and the
    integer n_heads.  Returns (logits, argmax, final-LN CLS vector).
    """
    D = bf16_to_f64
    H = int(p["n_heads"])
    patches = patchify(D(img_bits))
    z = np.concatenate([D(p["cls"])[None, :],
                        _store(linear(patches, D(p["W_pe"]), D(p["b_pe"])), round_bf16)], axis=0)
    z = z + D(p["pos"])
    T, d = z.shape
    hd = d // H
    for L in p["layers"]:
        h = _store(layernorm(z, D(L["ln1_g"]), D(L["ln1_b"])), round_bf16)
        qkv = _store(linear(h, D(L["Wqkv"]), D(L["bqkv"])), round_bf16)
        q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
        o = np.empty((T, d))
        for hh in range(H):
            sl = slice(hh * hd, (hh + 1) * hd)
            o[:, sl] = attention(q[:, sl], k[:, sl], v[:, sl])
        o = _store(o, round_bf16)
        z = z + linear(o, D(L["Wo"]), D(L["bo"]))
        h = _store(layernorm(z, D(L["ln2_g"]), D(L["ln2_b"])), round_bf16)
        f = _store(gelu(linear(h, D(L["W1"]), D(L["b1"]))), round_bf16)
        z = z + linear(f, D(L["W2"]), D(L["b2"]))
    c = _store(layernorm(z[0], D(p["lnf_g"]), D(p["lnf_b"])), round_bf16)
    logits = _store(linear(c, D(p["Whead"]), D(p["bhead"])), round_bf16)
    return logits, argmax_lowest(logits), c


# --------------------------------------------------------------------- decoder
def gather_kv(fetch_page: Callable[[int, int], np.ndarray], layer: int, table: np.ndarray,
              n_tokens: int) -> Tuple[np.ndarray, np.ndarray]:
    """Cached K and V of one request in one layer, tokens 0..n_tokens-1.

    fetch_page(layer, page_id) returns that page as uint16 [2, Hkv, PAGE, hd]
    (index 0 = K, 1 = V).  Token t lives in page table[t // PAGE], slot t % PAGE.
    Returns K, V as fp64 [Hkv, n_tokens, hd].
    """
    ks, vs = [], []
    for j in range((n_tokens + PAGE - 1) // PAGE):
        pg = bf16_to_f64(fetch_page(layer, int(table[j])))
        ks.append(pg[0])
        vs.append(pg[1])
    if not ks:
        return None, None
    K = np.concatenate(ks, axis=1)[:, :n_tokens]
    V = np.concatenate(vs, axis=1)[:, :n_tokens]
    return K, V


def decoder_layer(x: np.ndarray, li: int, kv_len: int, table: np.ndarray,
                  fetch_page: Callable[[int, int], np.ndarray], p: Dict,
                  round_bf16: bool = False) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Layer li of a Llama-style decoder for one new token at position kv_len.

    x is the residual stream entering the layer (fp64 [d]).  Pre-norm attention block, then pre-norm
    SwiGLU block: x += Wo attn(rope(Wq h), [cache; rope(Wk h)], [cache; Wv h]) with h = RMSNorm(x);
    x += Wd (silu(Wg h) * (Wu h)) with h = RMSNorm(x).  Query head hq reads KV head hq // (Hq / Hkv).
    Returns (x leaving the layer, the new token's k [Hkv, hd] after rotation, its v [Hkv, hd]).
    """
    D = bf16_to_f64
    Hq, Hkv, hd = int(p["n_q_heads"]), int(p["n_kv_heads"]), int(p["head_dim"])
    grp = Hq // Hkv
    L = p["layers"][li]
    h = _store(rmsnorm(x, D(L["g1"])), round_bf16)
    q = _store(linear(h, D(L["Wq"])), round_bf16).reshape(Hq, hd)
    k = _store(linear(h, D(L["Wk"])), round_bf16).reshape(Hkv, hd)
    v = _store(linear(h, D(L["Wv"])), round_bf16).reshape(Hkv, hd)
    q = _store(rope(q, kv_len), round_bf16)
    k = _store(rope(k, kv_len), round_bf16)
    Kc, Vc = gather_kv(fetch_page, li, table, kv_len)
    o = np.empty((Hq, hd))
    for hq in range(Hq):
        g = hq // grp
        Kh = k[g][None, :] if Kc is None else np.concatenate([Kc[g], k[g][None, :]], axis=0)
        Vh = v[g][None, :] if Vc is None else np.concatenate([Vc[g], v[g][None, :]], axis=0)
        o[hq] = attention(q[hq], Kh, Vh)
    o = _store(o.reshape(-1), round_bf16)
    x = x + linear(o, D(L["Wo"]))
    h = _store(rmsnorm(x, D(L["g2"])), round_bf16)
    f = _store(silu(linear(h, D(L["Wg"]))) * linear(h, D(L["Wu"])), round_bf16)
    x = x + linear(f, D(L["Wd"]))
    return x, k, v


def decoder_head(x: np.ndarray, p: Dict, round_bf16: bool = False) -> np.ndarray:
    """Final RMSNorm and LM head: logits [vocab] of the residual stream x [d]."""
    D = bf16_to_f64
    h = _store(rmsnorm(x, D(p["gf"])), round_bf16)
    return _store(linear(h, D(p["Wlm"])), round_bf16)


def decoder_step(token: int, kv_len: int, table: np.ndarray,
                 fetch_page: Callable[[int, int], np.ndarray], p: Dict,
                 round_bf16: bool = False) -> Dict:
    """One decode step of one sequence through a Llama-style decoder.

    The new token sits at position kv_len: its q and k are rotated at that position,
    its k, v are appended at cache slot kv_len (page table[kv_len // PAGE], slot
    kv_len % PAGE) and the query attends over positions 0..kv_len (kv_len + 1 tokens).
    The cached keys are taken as already rotated.

    p: Emb [V, d], layers[l] = {g1, Wq [Hq*hd, d], Wk [Hkv*hd, d], Wv, Wo [d, Hq*hd], g2,
    Wg [F, d], Wu [F, d], Wd [d, F]}, gf, Wlm [V, d] as bf16 bits; ints n_q_heads,
    n_kv_heads, head_dim.  Returns logits, argmax, per layer the appended k, v
    (fp64 [Hkv, hd]) with the (page, slot) they go to, and the residual stream after the
    embedding and after every layer ("residual", n_layers + 1 vectors).
    """
    x = bf16_to_f64(p["Emb"][int(token)])
    appended = []
    residual = [x]
    for li in range(len(p["layers"])):
        x, k, v = decoder_layer(x, li, kv_len, table, fetch_page, p, round_bf16)
        residual.append(x)
        appended.append({"k": k, "v": v, "page": int(table[kv_len // PAGE]), "slot": kv_len % PAGE})
    logits = decoder_head(x, p, round_bf16)
    return {"logits": logits, "argmax": argmax_lowest(logits), "appended": appended, "residual": residual}


def decoder_prefill(tokens: Sequence[int], kv_len: int, table: np.ndarray,
                    fetch_page: Callable[[int, int], np.ndarray], p: Dict,
                    round_bf16: bool = False) -> Dict:
    """A prompt chunk of n tokens through a Llama-style decoder (the prefill phase of an LLM request,
    Section 4.3; with kv_len > 0 it is one chunk of a chunked prefill).

    Token t of the chunk sits at position kv_len + t.  In every layer each token gets its own q, k, v
    (rotated at its own position); its k, v go to cache slot kv_len + t; its query attends causally:
    over the cached positions 0 .. kv_len - 1 and the chunk's tokens 0 .. t.  Everything else is
    token-wise, exactly as in decoder_layer.  With n = 1 this is decoder_step.
    Returns the last token's logits and argmax, per layer the chunk's appended k and v
    (fp64 [n, Hkv, hd]), and the residual stream after the embedding and after every layer ([n, d] each).
    """
    D = bf16_to_f64
    Hq, Hkv, hd = int(p["n_q_heads"]), int(p["n_kv_heads"]), int(p["head_dim"])
    grp = Hq // Hkv
    n = len(tokens)
    X = np.stack([D(p["Emb"][int(t)]) for t in tokens])
    appended = []
    residual = [X]
    for li, L in enumerate(p["layers"]):
        H = _store(rmsnorm(X, D(L["g1"])), round_bf16)
        Q = _store(linear(H, D(L["Wq"])), round_bf16).reshape(n, Hq, hd)
        K = _store(linear(H, D(L["Wk"])), round_bf16).reshape(n, Hkv, hd)
        V = _store(linear(H, D(L["Wv"])), round_bf16).reshape(n, Hkv, hd)
        Q = np.stack([_store(rope(Q[t], kv_len + t), round_bf16) for t in range(n)])
        K = np.stack([_store(rope(K[t], kv_len + t), round_bf16) for t in range(n)])
        Kc, Vc = gather_kv(fetch_page, li, table, kv_len)
        Oa = np.empty((n, Hq, hd))
        for t in range(n):
            for hq in range(Hq):
                g = hq // grp
                Kh = K[:t + 1, g] if Kc is None else np.concatenate([Kc[g], K[:t + 1, g]], axis=0)
                Vh = V[:t + 1, g] if Vc is None else np.concatenate([Vc[g], V[:t + 1, g]], axis=0)
                Oa[t, hq] = attention(Q[t, hq], Kh, Vh)
        Oa = _store(Oa.reshape(n, -1), round_bf16)
        X = X + linear(Oa, D(L["Wo"]))
        H = _store(rmsnorm(X, D(L["g2"])), round_bf16)
        F = _store(silu(linear(H, D(L["Wg"]))) * linear(H, D(L["Wu"])), round_bf16)
        X = X + linear(F, D(L["Wd"]))
        residual.append(X)
        appended.append({"k": K, "v": V})
    logits = decoder_head(X[n - 1], p, round_bf16)
    return {"logits": logits, "argmax": argmax_lowest(logits), "appended": appended, "residual": residual}


# ------------------------------------------------------------ host-side policy
def dp_group_count(required_fps: float, group_fps: float) -> int:
    """Eq. 4: ceil(frame-rate requirement / frame rate of one DP group)."""
    return int(math.ceil(required_fps / group_fps))


def inter_request_count(bs: int, mf_max: int) -> int:
    """Eq. 5: floor(batch size / max inter-frame count)."""
    return int(bs // mf_max)


def fs_satisfied(frames: float, required_fps: float, achieved_fps: float) -> float:
    """Goodput credit of a frequency-sensitive request (Section 3.3, text before Eq. 2):
    frames x achieved / required, never above the frame count."""
    return frames * min(1.0, achieved_fps / required_fps)


def admit(queue: List[Dict], now_ns: int, cap: int, mf_max: int = 0) -> Tuple[List[int], List[int]]:
    """Admission of one (model, category) queue for one step.

    queue: requests in arrival order, each {"ticket", "deadline_ns" (0 = none), "stream"}.
    1. A request whose deadline has passed is not processed and reports a timeout
       (Section 3.2, first handler rule).
    2. mf_max == 0 (latency-sensitive, or no multi-frame): the oldest `cap` live requests
       are taken (BS).
    3. mf_max > 0 (MF, Section 3.1 and Eq. 5): at most floor(cap / mf_max) distinct streams
       are served, chosen by their oldest waiting frame; every chosen stream contributes
       the same number of frames f = min(mf_max, fewest waiting frames among the chosen
       streams), oldest first, stream by stream in the order the streams were chosen.
    Returns (admitted tickets in batch order, dropped tickets).
    """
    dropped = [r["ticket"] for r in queue if r["deadline_ns"] != 0 and r["deadline_ns"] < now_ns]
    live = [r for r in queue if not (r["deadline_ns"] != 0 and r["deadline_ns"] < now_ns)]
    if mf_max <= 0:
        return [r["ticket"] for r in live[:cap]], dropped
    n_streams = inter_request_count(cap, mf_max)
    order: List[int] = []
    for r in live:
        if r["stream"] not in order:
            order.append(r["stream"])
    chosen = order[:n_streams]
    if not chosen:
        return [], dropped
    f = min(mf_max, min(sum(1 for r in live if r["stream"] == s) for s in chosen))
    out: List[int] = []
    for s in chosen:
        out += [r["ticket"] for r in live if r["stream"] == s][:f]
    return out, dropped
