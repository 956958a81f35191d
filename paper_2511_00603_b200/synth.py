"""Seeded synthetic workloads: model parameters, images, KV pools, decode batches, arrivals.

This module only draws random numbers and arranges bytes.  It contains none of the
forward-pass arithmetic and is the one piece of code that both the CUDA library's callers
and the CPU oracle's callers use, so that both sides consume identical bytes.

Matrices, embeddings, cls and pos are N(0, std) (std 0.02 unless stated); norm gains are 1 and
biases 0 unless `perturb` is given, in which case gains are 1 + N(0, perturb) and biases
N(0, perturb) so that the bias/gain paths carry signal.  Everything is stored as bf16.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np
import torch

PAGE = 16


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, std, g, device) -> torch.Tensor:
    return (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def _gain(n, perturb, g, device) -> torch.Tensor:
    if perturb:
        return (1.0 + torch.randn(n, generator=g, device=device) * perturb).to(torch.bfloat16)
    return torch.ones(n, device=device, dtype=torch.bfloat16)


def _bias(n, perturb, g, device) -> torch.Tensor:
    if perturb:
        return (torch.randn(n, generator=g, device=device) * perturb).to(torch.bfloat16)
    return torch.zeros(n, device=device, dtype=torch.bfloat16)


# ------------------------------------------------------------------ models
def make_mlp(dims: List[int], seed: int, device="cpu", std: float = 0.02, perturb: float = 0.0) -> Dict:
    """dims = [K0, N1, ..., N_last]; layer l has W [dims[l+1], dims[l]] and b [dims[l+1]]."""
    g = _gen(seed, device)
    Ws = [_normal((dims[i + 1], dims[i]), std, g, device) for i in range(len(dims) - 1)]
    bs = [_bias(dims[i + 1], perturb, g, device) for i in range(len(dims) - 1)]
    return {"kind": "mlp", "dims": list(dims), "W": Ws, "b": bs}


def make_vit(d: int, n_layers: int, n_heads: int, mlp: int, n_cls: int, seed: int, device="cpu",
             img: int = 224, patch: int = 16, std: float = 0.02, perturb: float = 0.0) -> Dict:
    g = _gen(seed, device)
    T = (img // patch) ** 2 + 1
    p = {"kind": "vit", "d": d, "n_layers": n_layers, "n_heads": n_heads, "mlp": mlp, "n_cls": n_cls,
         "img": img, "patch": patch, "T": T,
         "W_pe": _normal((d, 3 * patch * patch), std, g, device), "b_pe": _bias(d, perturb, g, device),
         "cls": _normal((d,), std, g, device), "pos": _normal((T, d), std, g, device), "layers": []}
    for _ in range(n_layers):
        p["layers"].append({
            "ln1_g": _gain(d, perturb, g, device), "ln1_b": _bias(d, perturb, g, device),
            "Wqkv": _normal((3 * d, d), std, g, device), "bqkv": _bias(3 * d, perturb, g, device),
            "Wo": _normal((d, d), std, g, device), "bo": _bias(d, perturb, g, device),
            "ln2_g": _gain(d, perturb, g, device), "ln2_b": _bias(d, perturb, g, device),
            "W1": _normal((mlp, d), std, g, device), "b1": _bias(mlp, perturb, g, device),
            "W2": _normal((d, mlp), std, g, device), "b2": _bias(d, perturb, g, device)})
    p["lnf_g"] = _gain(d, perturb, g, device)
    p["lnf_b"] = _bias(d, perturb, g, device)
    p["Whead"] = _normal((n_cls, d), std, g, device)
    p["bhead"] = _bias(n_cls, perturb, g, device)
    return p


def make_decoder(d: int, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, ffn: int,
                 vocab: int, seed: int, device="cpu", std: float = 0.02, perturb: float = 0.0) -> Dict:
    g = _gen(seed, device)
    p = {"kind": "decoder", "d": d, "n_layers": n_layers, "n_q_heads": n_q_heads, "n_kv_heads": n_kv_heads,
         "head_dim": head_dim, "ffn": ffn, "vocab": vocab,
         "Emb": _normal((vocab, d), std, g, device), "layers": []}
    for _ in range(n_layers):
        p["layers"].append({
            "g1": _gain(d, perturb, g, device),
            "Wq": _normal((n_q_heads * head_dim, d), std, g, device),
            "Wk": _normal((n_kv_heads * head_dim, d), std, g, device),
            "Wv": _normal((n_kv_heads * head_dim, d), std, g, device),
            "Wo": _normal((d, n_q_heads * head_dim), std, g, device),
            "g2": _gain(d, perturb, g, device),
            "Wg": _normal((ffn, d), std, g, device), "Wu": _normal((ffn, d), std, g, device),
            "Wd": _normal((d, ffn), std, g, device)})
    p["gf"] = _gain(d, perturb, g, device)
    p["Wlm"] = _normal((vocab, d), std, g, device)
    return p


def pack_decoder_layer(L: Dict) -> Dict:
    """Device layout of one decoder layer: Wqkv = rows [Wq; Wk; Wv]; Wgu has gate row j at
    2j and up row j at 2j+1 so a gate/up pair is adjacent in the GEMM's output columns."""
    F, d = L["Wg"].shape
    Wgu = torch.stack([L["Wg"], L["Wu"]], dim=1).reshape(2 * F, d).contiguous()
    return {"g1": L["g1"], "Wqkv": torch.cat([L["Wq"], L["Wk"], L["Wv"]], dim=0).contiguous(),
            "Wo": L["Wo"], "g2": L["g2"], "Wgu": Wgu, "Wd": L["Wd"]}


# ------------------------------------------------------------------ inputs
def make_mlp_inputs(batch: int, k: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randn((batch, k), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def make_images(batch: int, seed: int, device="cpu", img: int = 224) -> torch.Tensor:
    """U(0,1) fp32 images cast once to bf16; both sides consume the bf16 bytes."""
    g = _gen(seed, device)
    return torch.rand((batch, 3, img, img), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def make_kv_pool(n_layers: int, num_pages: int, n_kv_heads: int, head_dim: int, seed: int,
                 device="cpu") -> torch.Tensor:
    """bf16 N(0,1) pool [n_layers, num_pages, 2, Hkv, PAGE, hd], filled layer by layer."""
    g = _gen(seed, device)
    pool = torch.empty((n_layers, num_pages, 2, n_kv_heads, PAGE, head_dim), device=device, dtype=torch.bfloat16)
    for l in range(n_layers):
        step = max(1, (1 << 28) // (2 * n_kv_heads * PAGE * head_dim))
        for s in range(0, num_pages, step):
            e = min(num_pages, s + step)
            pool[l, s:e] = torch.randn((e - s, 2, n_kv_heads, PAGE, head_dim), generator=g, device=device,
                                       dtype=torch.float32).to(torch.bfloat16)
    return pool


def make_kv_pool_replicated(n_layers: int, num_pages: int, n_kv_heads: int, head_dim: int, seed: int,
                            device="cpu") -> torch.Tensor:
    """Pool of the same shape and distribution for very large caches: layer 0 is drawn N(0,1) as in
    make_kv_pool; layer l holds layer 0's pages rotated by 7919 * l positions (a copy, not a new draw),
    so filling 100+ GB takes seconds and any page of any layer can be recomputed from layer 0."""
    pool = torch.empty((n_layers, num_pages, 2, n_kv_heads, PAGE, head_dim), device=device, dtype=torch.bfloat16)
    pool[0] = make_kv_pool(1, num_pages, n_kv_heads, head_dim, seed, device=device)[0]
    for l in range(1, n_layers):
        sh = (7919 * l) % num_pages
        pool[l, sh:] = pool[0, :num_pages - sh]
        pool[l, :sh] = pool[0, num_pages - sh:]
    return pool


def make_decode_batch(batch: int, len_lo: int, len_hi: int, vocab: int, seed: int
                      ) -> Tuple[np.ndarray, np.ndarray, List[np.ndarray], int]:
    """Tokens ~U[0,vocab), KV lengths ~U[len_lo,len_hi] (inclusive), and per-request block
    tables that are disjoint slices of one seeded permutation of the page pool.  A request
    of length L owns ceil((L+1)/PAGE) pages (room for the appended token).
    Returns (tokens int32 [B], kv_lens int32 [B], tables list of int32 arrays, num_pages)."""
    rng = np.random.default_rng(seed)
    tokens = rng.integers(0, vocab, size=batch, dtype=np.int64).astype(np.int32)
    lens = rng.integers(len_lo, len_hi + 1, size=batch, dtype=np.int64).astype(np.int32)
    need = [(int(L) + 1 + PAGE - 1) // PAGE for L in lens]
    num_pages = int(sum(need))
    perm = rng.permutation(num_pages).astype(np.int32)
    tables, o = [], 0
    for n in need:
        tables.append(perm[o:o + n].copy())
        o += n
    return tokens, lens, tables, num_pages


def poisson_arrivals(rate_per_s: float, horizon_s: float, seed: int) -> np.ndarray:
    """Arrival times in ns over [0, horizon) with exponential inter-arrival gaps."""
    rng = np.random.default_rng(seed)
    n = int(rate_per_s * horizon_s * 1.5) + 16
    t = np.cumsum(rng.exponential(1.0 / rate_per_s, size=n))
    return (t[t < horizon_s] * 1e9).astype(np.int64)


# ------------------------------------------------------------------ byte views
def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def bits_view(p):
    """Recursively replace bf16 tensors by uint16 bit arrays (what the oracle reads)."""
    if isinstance(p, torch.Tensor):
        return to_bits(p) if p.dtype == torch.bfloat16 else p.detach().cpu().numpy()
    if isinstance(p, dict):
        return {k: bits_view(v) for k, v in p.items()}
    if isinstance(p, (list, tuple)):
        return [bits_view(v) for v in p]
    return p
