"""Convenience layer over the binding: owns the torch buffers a caller must keep alive
(workspace, per-request outputs, block tables) and turns torch tensors into epara_inputs.
All computation still happens inside the library's kernels."""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

from . import epara as E
from . import synth


class Server:
    def __init__(self, device: int = 0, workspace_bytes: int = 1 << 30, **cfg):
        self.device = torch.device("cuda", device)
        self.dev_index = device
        self.workspace = torch.empty(workspace_bytes, dtype=torch.uint8, device=self.device)
        self.ctx = E.Context(self.workspace, device=device, **cfg)
        self.models: List[Dict] = []
        self.pending: Dict[int, Tuple] = {}

    # ------------------------------------------------------------- placement
    def add_model(self, p: Dict, kv_pool: Optional[torch.Tensor] = None, max_kv_len: int = 0,
                  max_batch: int = 0, kv_pages: int = 0, trace: Optional[torch.Tensor] = None) -> int:
        """p: a synth model whose tensors are on this device.  Decoders are packed here."""
        if p["kind"] == "decoder" and "packed_layers" not in p:
            p["packed_layers"] = [synth.pack_decoder_layer(L) for L in p["layers"]]
        desc, keep = E.make_model_desc(p, kv_pool=kv_pool, max_kv_len=max_kv_len, max_batch=max_batch, kv_pages=kv_pages,
                                       trace=trace)
        mid = self.ctx.epara_register_model(desc, keep)
        n_out = p["dims"][-1] if p["kind"] == "mlp" else (p["n_cls"] if p["kind"] == "vit" else p["vocab"])
        self.models.append({"p": p, "n_out": n_out})
        return mid

    # ------------------------------------------------------------- requests
    def _outs(self, mid: int):
        n = self.models[mid]["n_out"]
        return (torch.empty(n, dtype=torch.bfloat16, device=self.device),
                torch.full((1,), -1, dtype=torch.int32, device=self.device))

    def submit(self, mid: int, category: int, x: Optional[torch.Tensor] = None, token: int = 0, kv_len: int = 0,
               table: Optional[torch.Tensor] = None, deadline_ns: int = 0, arrival_ns: int = 0, stream: int = 0,
               outs=None, tokens=None) -> int:
        """tokens: a prompt chunk (sequence of token ids) for a decoder; `token` is then ignored."""
        logits, am = outs if outs is not None else self._outs(mid)
        inp = E.Inputs()
        inp.input = x.data_ptr() if x is not None else None
        inp.token, inp.kv_len = int(token), int(kv_len)
        inp.block_table = table.data_ptr() if table is not None else None
        inp.n_blocks = int(table.numel()) if table is not None else 0
        if tokens is not None:
            arr = (E.C.c_int32 * len(tokens))(*[int(t) for t in tokens])     # read by the library during submit only
            inp.tokens, inp.n_tokens = arr, len(tokens)
        inp.deadline_ns, inp.arrival_ns, inp.stream = int(deadline_ns), int(arrival_ns), int(stream)
        inp.out_logits, inp.out_argmax = logits.data_ptr(), am.data_ptr()
        t = self.ctx.epara_submit(mid, category, inp)
        self.pending[t] = (logits, am, x, table)
        return t

    def step(self, now_ns: int = -1) -> E.StepInfo:
        return self.ctx.epara_step(torch.cuda.current_stream(self.device).cuda_stream, now_ns)

    def collect(self, ticket: int):
        """(status, logits tensor, argmax tensor); buffers are released once the status is final."""
        s, _ = self.ctx.epara_collect(ticket)
        if s == E.PENDING:
            return s, None, None
        logits, am, _, _ = self.pending.pop(ticket)
        return s, logits, am

    def collect_wait(self, ticket: int):
        torch.cuda.current_stream(self.device).synchronize()
        return self.collect(ticket)

    def close(self):
        self.ctx.close()
