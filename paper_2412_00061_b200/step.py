"""One draft-and-verify step as five C-ABI calls on one stream, with its device buffers.

This is plumbing: it allocates the outputs once, keeps the inputs resident, and enqueues
the calls in order.  No arithmetic of the method happens here.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding
from .synth import StepConfig


def to_device(a: np.ndarray, dtype: str, device) -> torch.Tensor:
    """Host array (values already representable in `dtype`) -> device tensor of that dtype."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.float32:
        return t.to(device=device, dtype=torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()
    return t.to(device=device).contiguous()


class DraftVerifyStep:
    L2_PREFETCH_BYTES = 48 << 20
    def __init__(self, cfg: StepConfig, device="cuda:0", max_draft_rows: int = 0, debug_logits: bool = False):
        self.cfg = cfg
        self.device = torch.device(device)
        self.h = binding.Handle(cfg.B, cfg.H, cfg.V, cfg.T, cfg.k, cfg.beam, cfg.topN, cfg.max_nodes,
                                cfg.Hq, cfg.Hkv, cfg.D,
                                binding.DTYPE_BF16 if cfg.dtype == "bf16" else binding.DTYPE_F32,
                                cfg.score_mode, max_draft_rows, device=device)
        self.M = max_draft_rows or cfg.B
        B, T, k, N, n = cfg.B, cfg.T, cfg.k, cfg.topN, cfg.max_nodes
        W = (n + 63) // 64
        dev, i32, f32 = self.device, torch.int32, torch.float32
        act = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        z = lambda *s, dtype=i32: torch.zeros(*s, dtype=dtype, device=dev)
        self.out: Dict[str, torch.Tensor] = dict(
            topk_id=z(self.M, T, k), topk_lp=z(self.M, T, k, dtype=f32), lse=z(self.M, T, dtype=f32),
            cand_tok=z(B, N, T), cand_len=z(B, N), cand_score=z(B, N, dtype=f32), n_cand=z(B),
            node_tok=z(B, n), parent=z(B, n), depth=z(B, n), pos=z(B, n),
            mask=z(B, n, W, dtype=torch.int64), retrieve=z(B, N, T), n_nodes=z(B),
            O=z(B, n, cfg.Hq, cfg.D, dtype=act),
            argmax=z(B, n), acc_len=z(B), acc_nodes=z(B, T), acc_tok=z(B, T), next_tok=z(B),
            new_kv_len=z(B), next_sel_row=z(B),
        )
        if debug_logits:
            self.out["draft_logits_dbg"] = z(self.M, T, cfg.V + 1, dtype=f32)
            self.out["lm_logits_dbg"] = z(B * n, cfg.V, dtype=f32)
        self.inp: Dict[str, Optional[torch.Tensor]] = {}

    def set_inputs(self, **tensors):
        """x, Wd, blank_bias, row_seq, sel_row, base_tok, kv_len, Q, K, V, hn, Wl (device tensors)."""
        self.inp.update(tensors)
        if "Wl" in tensors and self.cfg.dtype == "bf16":
            # while the small kernels between draft head and LM head run, HBM is idle: let L2
            # fetch the head of the LM-head weights then
            self.h.set_l2_prefetch(tensors["Wl"], self.L2_PREFETCH_BYTES)

    # individual stages ----------------------------------------------------------------
    def draft(self, stream=None):
        i, o = self.inp, self.out
        self.h.draft_logits(i["x"], i["Wd"], i.get("row_seq"), i.get("blank_bias"),
                            o["topk_id"], o["topk_lp"], o["lse"], o.get("draft_logits_dbg"), stream=stream)

    def collapse(self, stream=None):
        i, o = self.inp, self.out
        self.h.topk_collapse(o["topk_id"], o["topk_lp"], i.get("sel_row"),
                             o["cand_tok"], o["cand_len"], o["cand_score"], o["n_cand"], stream=stream)

    def tree(self, stream=None):
        i, o = self.inp, self.out
        self.h.build_tree(i["base_tok"], i["kv_len"], o["cand_tok"], o["cand_len"], o["n_cand"],
                          o["node_tok"], o["parent"], o["depth"], o["pos"], o["mask"], o["retrieve"], o["n_nodes"],
                          stream=stream)

    def attention(self, stream=None):
        i, o = self.inp, self.out
        self.h.tree_attention(i["Q"], i["K"], i["V"], i["kv_len"], o["n_nodes"], o["mask"],
                              1.0 / float(self.cfg.D) ** 0.5, o["O"], stream=stream)

    def verify(self, stream=None):
        i, o = self.inp, self.out
        self.h.verify_accept(i["hn"], i["Wl"], o["node_tok"], o["parent"], o["n_nodes"],
                             o["argmax"], o["acc_len"], o["acc_nodes"], o["acc_tok"], o["next_tok"],
                             o.get("lm_logits_dbg"), stream=stream)

    def commit(self, stream=None):
        """History update (not part of run(): it changes the K/V cache in place)."""
        i, o = self.inp, self.out
        self.h.commit_accepted(i["K"], i["V"], i["kv_len"], o["acc_len"], o["acc_nodes"],
                               o["new_kv_len"], o["next_sel_row"], stream=stream)

    def run(self, stream=None):
        """The whole hot path: five calls back to back on one stream, no host sync."""
        self.draft(stream)
        self.collapse(stream)
        self.tree(stream)
        self.attention(stream)
        self.verify(stream)

    def check_status(self):
        st = self.h.poll_status()
        if st != 0:
            raise binding.CtcsdError("device status %d: %s" % (st, self.h.lib.ctcsd_strerror(st).decode()))

    def host(self, name: str) -> np.ndarray:
        t = self.out[name]
        if t.dtype == torch.bfloat16:
            t = t.float()
        return t.cpu().numpy()
