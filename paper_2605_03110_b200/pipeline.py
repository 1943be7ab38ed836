"""Selection / attention pipelining on two CUDA streams (Section 8.4 of the paper: the selection
of layer l+1 can run while the attention of layer l is computed, which hides its latency).

Host-side plumbing only: streams, events and the order of the library calls.  The selection
chain (full selection at layer 0, a cascade step per later layer) runs on one stream with one
context; its consumer -- the nearest-representative map and the attention on the
representatives of the same layer -- runs on a second stream with a context of its own (the
two calls share no workspace).  Layer l's consumer waits for layer l's selection; the
selection reuses a set buffer only after the consumer that read it has finished.
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import binding as ada


class SelectionAttentionPipeline:
    """layers: list of (T, h, d_h) bf16 tensors; a layer's activations stand in for its Q, K, V."""

    def __init__(self, T: int, h: int, d_h: int, tau: float, device, n_sets: int = 3, flags: int = 0,
                 attn_flags: int = 0):
        self.T, self.h, self.d_h, self.tau = T, h, d_h, tau
        self.flags, self.attn_flags = flags, attn_flags
        idx = device.index if hasattr(device, "index") and device.index is not None else 0
        self.sel = ada.ada_create(1, T, h * d_h, ada.ADA_BF16, device=idx)
        self.con = ada.ada_create(1, T, h * d_h, ada.ADA_BF16, device=idx)
        self.sets = [ada.CascadeOut(1, T, device, want_gamma=False) for _ in range(n_sets)]
        self.near = torch.empty((1, T), dtype=torch.int32, device=device)
        self.s_sel, self.s_att = torch.cuda.Stream(device), torch.cuda.Stream(device)
        self.device = device

    def close(self):
        ada.ada_destroy(self.sel)
        ada.ada_destroy(self.con)

    def _select(self, l: int, X: torch.Tensor, stream):
        cur = self.sets[l % len(self.sets)]
        if l == 0:
            ada.ada_select_full(self.sel, X.view(1, self.T, -1), self.tau, cur.rep_out, cur.rep_out_cnt,
                                want_gamma=False, stream=stream)
        else:
            prev = self.sets[(l - 1) % len(self.sets)]
            ada.ada_cascade_step(self.sel, X.view(1, self.T, -1), self.tau, prev.rep_out, prev.rep_out_cnt,
                                 out=cur, flags=self.flags, stream=stream)
        return cur

    def _consume(self, l: int, X: torch.Tensor, out: torch.Tensor, stream):
        cur = self.sets[l % len(self.sets)]
        lib = ada.lib()
        ada._check(lib.ada_nearest_rep(self.con.h, X.data_ptr(), 1, self.T, self.h * self.d_h, X.stride(0),
                                       ada.ADA_BF16, cur.rep_out.data_ptr(), cur.rep_out_cnt.data_ptr(),
                                       self.near.data_ptr(), None, ada._stream(stream)), "ada_nearest_rep")
        ada.ada_attention_reps(self.con, X, X, X, cur.rep_out[0], cur.rep_out_cnt, nearest_idx=self.near[0],
                               out=out, flags=self.attn_flags, stream=stream)

    def run(self, layers: List[torch.Tensor], outs: List[torch.Tensor], overlap: bool = True,
            stream: Optional[torch.cuda.Stream] = None):
        """Enqueue the whole chain.  overlap=False: everything on one stream, in order."""
        L = len(layers)
        if not overlap:
            st = stream or torch.cuda.current_stream()
            for l in range(L):
                self._select(l, layers[l], st)
                self._consume(l, layers[l], outs[l], st)
            return
        base = stream or torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(base)
        self.s_sel.wait_event(start)
        self.s_att.wait_event(start)
        sel_done = [torch.cuda.Event() for _ in range(L)]
        att_done = [torch.cuda.Event() for _ in range(L)]
        n = len(self.sets)
        for l in range(L):
            # layer l's selection overwrites the buffer layer l - n used: its consumer must be done
            if l >= n:
                self.s_sel.wait_event(att_done[l - n])
            self._select(l, layers[l], self.s_sel)
            sel_done[l].record(self.s_sel)
            self.s_att.wait_event(sel_done[l])
            self._consume(l, layers[l], outs[l], self.s_att)
            att_done[l].record(self.s_att)
        base.wait_stream(self.s_sel)
        base.wait_stream(self.s_att)
