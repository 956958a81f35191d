"""The synthetic serving workloads: which models are co-resident, their categories, batches and
inputs.  Only placement and argument marshalling happen here; every forward pass runs in the
library's kernels.

mixed step (the co-resident configuration): 8 instances -- 3x MLP-A (512->512->512->512->10),
3x ViT-S/16 (d 384, 6 heads, 12 layers, MLP 1536, 1000 classes), 2x Llama-style 1B decoder
(d 2048, 16 layers, 32/8 heads, hd 64, FFN 8192, vocab 32000).  Per family the first instance
is latency-sensitive (batch <= 4, 20 ms deadline), the others frequency-sensitive (batch <= 256).
Decoder requests have KV lengths ~U[128, 4096] in a paged cache filled N(0,1) with permuted
block tables.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List

import numpy as np
import torch

from . import epara as E
from . import synth

from .configs import (DEC_1B, DEC_8B, LS_DEADLINE_NS, MIXED_RATES, MLP_A, STRESS_DEC_BATCH, STRESS_KV_HI, STRESS_KV_LO,  # noqa: F401
                      STRESS_VIT_BATCH, STRESS_VITS, VIT_B, VIT_S)


class Instance:
    """One placed model with a pool of ready-made requests (inputs, outputs, ctypes descriptors)."""

    def __init__(self, srv, p: Dict, category: int, n_req: int, seed: int, kv_lo: int = 128, kv_hi: int = 4096,
                 max_batch: int = 0, kv_replicate_layers: bool = False):
        dev = srv.device
        self.p, self.category, self.n_req, self.kind = p, category, n_req, p["kind"]
        self.kv_pool = None
        self.tokens = self.lens = self.tables = None
        if self.kind == "mlp":
            self.x = synth.make_mlp_inputs(n_req, p["dims"][0], seed, device=dev)
            self.n_out = p["dims"][-1]
        elif self.kind == "vit":
            self.x = synth.make_images(n_req, seed, device=dev, img=p["img"])
            self.n_out = p["n_cls"]
        else:
            self.x = None
            self.n_out = p["vocab"]
            self.tokens, self.lens, self.tables, npages = synth.make_decode_batch(n_req, kv_lo, kv_hi, p["vocab"], seed)
            if kv_replicate_layers:
                self.kv_pool = synth.make_kv_pool_replicated(p["n_layers"], npages, p["n_kv_heads"], p["head_dim"],
                                                             seed + 1, device=dev)
            else:
                self.kv_pool = synth.make_kv_pool(p["n_layers"], npages, p["n_kv_heads"], p["head_dim"], seed + 1,
                                                  device=dev)
            flat = np.concatenate(self.tables)
            self.tables_dev = torch.as_tensor(flat, device=dev)
            self.table_off = np.concatenate([[0], np.cumsum([len(t) for t in self.tables])])
        self.mid = srv.add_model(p, kv_pool=self.kv_pool, max_kv_len=kv_hi, max_batch=max_batch or n_req)
        self.logits = torch.zeros((n_req, self.n_out), dtype=torch.bfloat16, device=dev)
        self.argmax = torch.full((n_req,), -1, dtype=torch.int32, device=dev)
        self.inputs = (E.Inputs * n_req)()
        self.tickets = (C.c_uint64 * n_req)()
        for i in range(n_req):
            self.fill(self.inputs[i], i, i)

    def fill(self, inp: "E.Inputs", req: int, out_slot: int, deadline_ns: int = 0, arrival_ns: int = 0, stream: int = 0):
        """Request `req` of the pool, writing its result to output row `out_slot`."""
        if self.kind == "decoder":
            inp.input = None
            inp.token, inp.kv_len = int(self.tokens[req]), int(self.lens[req])
            inp.block_table = self.tables_dev.data_ptr() + 4 * int(self.table_off[req])
            inp.n_blocks = int(self.table_off[req + 1] - self.table_off[req])
        else:
            inp.input = self.x[req].data_ptr()
        inp.deadline_ns, inp.arrival_ns, inp.stream = deadline_ns, arrival_ns, stream
        inp.out_logits = self.logits[out_slot].data_ptr()
        inp.out_argmax = self.argmax.data_ptr() + 4 * out_slot

    def submit_all(self, ctx: "E.Context", buf: int = 0):
        """Submits the whole pool; buf = k takes inputs, outputs and descriptors from buffer set k (make_bufs)."""
        ctx.epara_submit_many(self.mid, self.category, self.inputs_bufs[buf] if buf else self.inputs, self.n_req,
                              self.tickets)

    def make_bufs(self, n: int):
        """n buffer sets (set 0 is self.x / self.logits / self.argmax), each with its own request
        descriptors: device inputs, so that the inputs of later steps can be uploaded while earlier steps
        still read theirs, and device outputs, so that a step's results can be read back while the next
        step runs."""
        self.x_bufs, self.inputs_bufs = [self.x], [self.inputs]
        self.logits_bufs, self.argmax_bufs = [self.logits], [self.argmax]
        for _ in range(1, n):
            xb = None if self.x is None else torch.empty_like(self.x)
            lb, ab = torch.zeros_like(self.logits), torch.full_like(self.argmax, -1)
            ib = (E.Inputs * self.n_req)()
            for i in range(self.n_req):
                C.memmove(C.byref(ib[i]), C.byref(self.inputs[i]), C.sizeof(E.Inputs))
                if xb is not None:
                    ib[i].input = xb[i].data_ptr()
                ib[i].out_logits = lb[i].data_ptr()
                ib[i].out_argmax = ab.data_ptr() + 4 * i
            self.x_bufs.append(xb)
            self.inputs_bufs.append(ib)
            self.logits_bufs.append(lb)
            self.argmax_bufs.append(ab)

    def input_bytes(self) -> int:
        return 0 if self.x is None else self.x.numel() * self.x.element_size()

    def output_bytes(self) -> int:
        return self.logits.numel() * 2 + self.argmax.numel() * 4


def workspace_bytes_mixed(ls_batch: int, fs_batch: int) -> int:
    # ViT-S activations dominate: ~8.5 KB per token, 197 tokens per image
    vit = lambda b: (b * 197 + 128) * 10 * 1024
    dec = lambda b: (b + 128) * (2048 * 6 + 3072 * 2 + 2048 * 2 + 8192 * 2 + 32000 * 2) + b * 32 * 17 * 66 * 4
    return int(64 << 20) + vit(ls_batch) + 2 * vit(fs_batch) + dec(ls_batch) + dec(fs_batch) + (64 << 20)


def build_mixed(srv, seed: int = 3, ls_batch: int = 4, fs_batch: int = 256, kv_lo: int = 128, kv_hi: int = 4096
                ) -> List[Instance]:
    """The 8 co-resident instances with one full batch of requests each."""
    dev = srv.device
    out: List[Instance] = []
    k = 0
    for i in range(3):
        cat, n = (E.CAT_LS, ls_batch) if i == 0 else (E.CAT_FS, fs_batch)
        out.append(Instance(srv, synth.make_mlp(MLP_A, seed=seed * 100 + k, device=dev), cat, n, seed * 1000 + k))
        k += 1
    for i in range(3):
        cat, n = (E.CAT_LS, ls_batch) if i == 0 else (E.CAT_FS, fs_batch)
        out.append(Instance(srv, synth.make_vit(seed=seed * 100 + k, device=dev, **VIT_S), cat, n, seed * 1000 + k))
        k += 1
    for i in range(2):
        cat, n = (E.CAT_LS, ls_batch) if i == 0 else (E.CAT_FS, fs_batch)
        out.append(Instance(srv, synth.make_decoder(seed=seed * 100 + k, device=dev, **DEC_1B), cat, n,
                            seed * 1000 + k, kv_lo=kv_lo, kv_hi=kv_hi))
        k += 1
    return out


# ------------------------------------------------------------------ stress step

def stress_bytes(kv_hi: int, n_vits: int = STRESS_VITS, vit_batch: int = STRESS_VIT_BATCH,
                 dec_batch: int = STRESS_DEC_BATCH, kv_lo: int = STRESS_KV_LO) -> Dict[str, float]:
    """Device bytes the stress step needs for a KV upper bound (expected value of the seeded lengths)."""
    d = DEC_8B
    per_tok = 2 * d["n_kv_heads"] * d["head_dim"] * 2 * d["n_layers"]
    mean_pages = ((kv_lo + kv_hi) / 2 + 1 + synth.PAGE) / synth.PAGE
    kv = dec_batch * mean_pages * synth.PAGE * per_tok
    dec_w = 2.0 * (2 * d["vocab"] * d["d"] + d["n_layers"] * (
        (d["n_q_heads"] + 2 * d["n_kv_heads"]) * d["head_dim"] * d["d"] + d["d"] * d["n_q_heads"] * d["head_dim"] +
        3 * d["ffn"] * d["d"]))
    vit_w = n_vits * 2.0 * 86.6e6
    rows = vit_batch * 197 + 128
    ws = n_vits * rows * (768 * 4 + 768 * 2 * 2 + 2304 * 2 + 3072 * 2) + (dec_batch + 128) * (
        4096 * 6 + 6144 * 2 + 14336 * 2 + 32000 * 2) + dec_batch * 32 * (kv_hi // 256 + 2) * 130 * 4 + (256 << 20)
    imgs = n_vits * vit_batch * 3 * 224 * 224 * 2
    return {"kv": kv, "decoder_weights": dec_w, "vit_weights": vit_w, "workspace": float(ws), "images": float(imgs),
            "total": kv + dec_w + vit_w + ws + imgs}


def build_stress(srv, seed: int = 4, kv_hi: int = STRESS_KV_HI, n_vits: int = STRESS_VITS,
                 vit_batch: int = STRESS_VIT_BATCH, dec_batch: int = STRESS_DEC_BATCH, kv_lo: int = STRESS_KV_LO
                 ) -> List[Instance]:
    """The stress configuration: one 8B-shaped decoder decoding `dec_batch` sequences with KV lengths
    ~U[kv_lo, kv_hi], co-resident with `n_vits` ViT-B/16 instances at batch `vit_batch`, all
    frequency-sensitive.  The decoder's unpacked weight copies are dropped once the packed layout exists;
    the KV pool is drawn for layer 0 and rotated for the other layers (see make_kv_pool_replicated)."""
    dev = srv.device
    out: List[Instance] = []
    p = synth.make_decoder(seed=seed * 100, device=dev, **DEC_8B)
    p["packed_layers"] = [synth.pack_decoder_layer(L) for L in p["layers"]]
    p["layers"] = None                      # the packed layout is all the library reads
    out.append(Instance(srv, p, E.CAT_FS, dec_batch, seed * 1000, kv_lo=kv_lo, kv_hi=kv_hi, kv_replicate_layers=True))
    for i in range(n_vits):
        out.append(Instance(srv, synth.make_vit(seed=seed * 100 + 1 + i, device=dev, **VIT_B), E.CAT_FS, vit_batch,
                            seed * 1000 + 1 + i))
    return out
