"""Sampled parity of the resident stress step (8B-shaped decoder, batch 256, co-resident ViT-B/16 instances).

The workload keeps only the packed device layout of the decoder's weights and a KV cache of 100+ GB, so the
oracle cannot be handed copies: it reads one layer's weights at a time out of the packed tensors and the
pages of the checked request out of the device pool after the step.  A step writes a request's new k, v at
slot kv_len only, and the oracle attends to the kv_len slots before it, so the pool after the step serves.

Used by tests/test_gpu_configs.py on a cut of the configuration and by `bench.py --workload stress --check`
on the configuration itself (about a quarter of an hour of oracle time for 8 requests at 32 layers)."""
import time
from typing import Dict, List

import numpy as np
import torch

from oracle import epara_oracle as O
from paper_2511_00603_b200 import synth
from tests.parity import assert_close, assert_parity, check_argmax


class PackedLayers:
    """The decoder's layers as the oracle names them (Wq, Wk, Wv, Wg, Wu separately), cut out of the packed
    device layout (Wqkv rows [q; k; v], Wgu rows gate/up interleaved) one layer at a time."""

    def __init__(self, packed: List[Dict], n_q_heads: int, n_kv_heads: int, head_dim: int):
        self.packed, self.nq, self.nkv = packed, n_q_heads * head_dim, n_kv_heads * head_dim
        self._last = (-1, None)

    def __len__(self):
        return len(self.packed)

    def __getitem__(self, l: int) -> Dict:
        if self._last[0] != l:
            P = self.packed[l]
            qkv, gu = P["Wqkv"], P["Wgu"]
            L = {"g1": P["g1"], "Wq": qkv[:self.nq], "Wk": qkv[self.nq:self.nq + self.nkv], "Wv": qkv[self.nq + self.nkv:],
                 "Wo": P["Wo"], "g2": P["g2"], "Wg": gu[0::2], "Wu": gu[1::2], "Wd": P["Wd"]}
            self._last = (l, synth.bits_view({k: v.contiguous() for k, v in L.items()}))
        return self._last[1]


def decoder_view(p: Dict) -> Dict:
    v = synth.bits_view({k: p[k] for k in p if k not in ("packed_layers", "layers")})
    v["layers"] = PackedLayers(p["packed_layers"], p["n_q_heads"], p["n_kv_heads"], p["head_dim"])
    return v


def pick_requests(lens: np.ndarray, n: int) -> List[int]:
    """n requests spread over the KV lengths of the batch, the shortest and the longest among them."""
    order = np.argsort(lens, kind="stable")
    idx = np.unique(np.round(np.linspace(0, len(order) - 1, min(n, len(order)))).astype(int))
    return [int(order[i]) for i in idx]


def check_stress_step(insts, n_dec: int = 8, n_img: int = 2, log=print) -> Dict:
    """Compares sampled outputs of one executed step of the stress instances (workloads.build_stress) with
    the oracle: n_dec decode requests under the deep-model rule of assert_parity, n_img images of the
    first and of the last ViT instance at the stated tolerance.  Returns the measured errors."""
    out = {"decoder": [], "vit": []}
    for k, inst in enumerate(insts):
        lg = inst.logits.float()
        assert torch.isfinite(lg).all(), f"instance {k}: non-finite logits"
        assert torch.equal(inst.argmax.long(), lg.argmax(dim=1)), f"instance {k}: argmax kernel disagrees with its logits"
    dec = [i for i in insts if i.kind == "decoder"]
    vits = [i for i in insts if i.kind == "vit"]
    for inst in dec:
        v = decoder_view(inst.p)
        fetch = lambda l, pg: synth.to_bits(inst.kv_pool[l, pg])
        for i in pick_requests(np.asarray(inst.lens), n_dec):
            t0 = time.time()
            tok, L, tb = int(inst.tokens[i]), int(inst.lens[i]), inst.tables[i]
            ra = O.decoder_step(tok, L, tb, fetch, v)
            rb = O.decoder_step(tok, L, tb, fetch, v, round_bf16=True)
            what = f"stress decoder request {i} (L={L})"
            e = assert_parity(inst.logits[i], ra["logits"], rb["logits"], what=what, deep=True)
            e["decided_by_gap"] = bool(check_argmax(int(inst.argmax[i]), inst.logits[i], rb["logits"]))
            e.update({"request": i, "kv_len": L, "oracle_s": round(time.time() - t0, 1)})
            # the k, v the step appended at slot L of every layer, against the bf16-storage evaluation
            worst = 0.0
            for l, ap in enumerate(rb["appended"]):
                worst = max(worst, assert_close(inst.kv_pool[l, ap["page"], 0, :, ap["slot"], :], ap["k"], tol=1.5e-1,
                                                what=f"{what}: appended k, layer {l}"))
                worst = max(worst, assert_close(inst.kv_pool[l, ap["page"], 1, :, ap["slot"], :], ap["v"], tol=1.5e-1,
                                                what=f"{what}: appended v, layer {l}"))
            e["appended_kv_worst_max_rel"] = worst
            out["decoder"].append(e)
            log(f"{what}: " + ", ".join(f"{kk} {vv:.3e}" if isinstance(vv, float) else f"{kk} {vv}" for kk, vv in e.items()))
    for inst in ([vits[0], vits[-1]] if len(vits) > 1 else vits)[:max(n_img, 1)]:
        pv = synth.bits_view(inst.p)
        for i in ([0] if n_img <= 2 and len(vits) > 1 else list(range(min(n_img, inst.n_req)))):
            ref, _, _ = O.vit_forward(synth.to_bits(inst.x[i]), pv)
            e = assert_close(inst.logits[i], ref, what=f"stress ViT-B instance, image {i}")
            check_argmax(int(inst.argmax[i]), inst.logits[i], ref)
            out["vit"].append({"image": i, "max_rel": e})
            log(f"stress ViT-B image {i}: max relative error {e:.3e}")
    return out
