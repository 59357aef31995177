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
    # Bytes of the LM-head weights that the draft head asks L2 to fetch when its own stream is issued
    # (ctcsd_set_l2_prefetch).  Off: on B200 the step was measured at the same time with 0, 24 and 48 MB
    # and slower beyond (the fetched lines did not shorten the LM head, whose tiles come by TMA).
    L2_PREFETCH_BYTES = 0
    def __init__(self, cfg: StepConfig, device="cuda:0", max_draft_rows: int = 0, debug_logits: bool = False,
                 layout: str = "packed"):
        """layout "packed": collapse first, tree over the collapsed candidates (the default);
        "raw": the paper's own layout (Sec. 3.3) - tree over the most probable raw slot paths,
        removed symbols masked in the attention map."""
        if layout not in ("packed", "raw"):
            raise ValueError("layout must be 'packed' or 'raw'")
        self.layout = layout
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
            argmax=z(B, n),
        )
        if layout == "raw":
            self.out.update(kept=z(B, n), nka=z(B, n))
        # the step's results share one buffer, so that reading them back is a single copy
        names = [("acc_len", (B,)), ("acc_nodes", (B, T)), ("acc_tok", (B, T)), ("next_tok", (B,)),
                 ("new_kv_len", (B,)), ("next_sel_row", (B,))]
        self.result = z(sum(int(np.prod(sh)) for _, sh in names))
        off = 0
        for nm, sh in names:
            cnt = int(np.prod(sh))
            self.out[nm] = self.result[off:off + cnt].view(*sh)
            off += cnt
        self.input_arena = None
        if debug_logits:
            self.out["draft_logits_dbg"] = z(self.M, T, cfg.V + 1, dtype=f32)
            self.out["lm_logits_dbg"] = z(B * n, cfg.V, dtype=f32)
        self.inp: Dict[str, Optional[torch.Tensor]] = {}

    def set_inputs(self, **tensors):
        """x, Wd, blank_bias, row_seq, sel_row, base_tok, kv_len, Q, K, V, hn, Wl (device tensors)."""
        self.inp.update(tensors)
        if "Wl" in tensors and self.cfg.dtype == "bf16" and self.L2_PREFETCH_BYTES > 0:
            self.h.set_l2_prefetch(tensors["Wl"], self.L2_PREFETCH_BYTES)

    PER_STEP_INPUTS = ("x", "base_tok", "kv_len", "Q", "hn")

    def pack_step_inputs(self):
        """Moves the tensors that change every step (hidden state, base token, cache length, tree
        queries, tree-node hidden states) into one device buffer, 256-byte aligned each, so that a
        step's host-to-device traffic is a single copy.  Returns a pinned host mirror of that
        buffer holding the current values; upload() copies a mirror to the device."""
        sizes = []
        for k in self.PER_STEP_INPUTS:
            t = self.inp[k]
            sizes.append((k, t, (t.numel() * t.element_size() + 255) // 256 * 256))
        self.input_arena = torch.empty(sum(sz for _, _, sz in sizes), dtype=torch.uint8, device=self.device)
        off = 0
        for k, t, sz in sizes:
            nbytes = t.numel() * t.element_size()
            view = self.input_arena[off:off + nbytes].view(t.dtype).view(t.shape)
            view.copy_(t)
            self.inp[k] = view
            off += sz
        # x, base_tok and kv_len come first: the draft head and the tree need them; Q and hn are
        # needed only from the attention on
        self.early_bytes = sum(sz for k, _, sz in sizes if k in ("x", "base_tok", "kv_len"))
        torch.cuda.synchronize(self.device)
        return self.input_arena.cpu().pin_memory()

    def upload(self, host_arena: torch.Tensor):
        self.input_arena.copy_(host_arena, non_blocking=True)

    def run_from_host(self, host_arena: torch.Tensor, host_result: torch.Tensor):
        """One step end to end on the current stream: every per-step input is copied from the pinned
        host mirror, the five calls run, the result goes back to pinned host memory.  The copy of
        the tree queries and tree-node hidden states (the bulk of the bytes) runs on a second stream
        beside the draft head, which does not read them, and joins before the attention."""
        cur = torch.cuda.current_stream(self.device)
        if not hasattr(self, "_copy_stream"):
            self._copy_stream = torch.cuda.Stream(device=self.device)
        e = self.early_bytes
        fork, join = torch.cuda.Event(), torch.cuda.Event()
        fork.record(cur)
        self._copy_stream.wait_event(fork)
        with torch.cuda.stream(self._copy_stream):
            self.input_arena[e:].copy_(host_arena[e:], non_blocking=True)
            join.record(self._copy_stream)
        self.input_arena[:e].copy_(host_arena[:e], non_blocking=True)
        self.draft()
        self.collapse()
        self.tree()
        cur.wait_event(join)
        self.attention()
        self.verify()
        self.download(host_result)

    def download(self, host_result: torch.Tensor):
        host_result.copy_(self.result, non_blocking=True)

    # individual stages ----------------------------------------------------------------
    def draft(self, stream=None):
        i, o = self.inp, self.out
        self.h.draft_logits(i["x"], i["Wd"], i.get("row_seq"), i.get("blank_bias"),
                            o["topk_id"], o["topk_lp"], o["lse"], o.get("draft_logits_dbg"), stream=stream)

    def collapse(self, stream=None):
        i, o = self.inp, self.out
        if self.layout == "raw":      # cand_tok / cand_score / n_cand then hold the raw paths
            self.h.select_raw_paths(o["topk_id"], o["topk_lp"], i.get("sel_row"),
                                    o["cand_tok"], o["cand_score"], o["n_cand"], stream=stream)
            return
        self.h.topk_collapse(o["topk_id"], o["topk_lp"], i.get("sel_row"),
                             o["cand_tok"], o["cand_len"], o["cand_score"], o["n_cand"], stream=stream)

    def tree(self, stream=None):
        i, o = self.inp, self.out
        if self.layout == "raw":
            self.h.build_raw_tree(i["base_tok"], i["kv_len"], o["cand_tok"], o["n_cand"],
                                  o["node_tok"], o["parent"], o["depth"], o["pos"], o["mask"], o["retrieve"],
                                  o["n_nodes"], o["kept"], o["nka"], stream=stream)
            return
        self.h.build_tree(i["base_tok"], i["kv_len"], o["cand_tok"], o["cand_len"], o["n_cand"],
                          o["node_tok"], o["parent"], o["depth"], o["pos"], o["mask"], o["retrieve"], o["n_nodes"],
                          stream=stream)

    def attention(self, stream=None):
        i, o = self.inp, self.out
        self.h.tree_attention(i["Q"], i["K"], i["V"], i["kv_len"], o["n_nodes"], o["mask"],
                              1.0 / float(self.cfg.D) ** 0.5, o["O"], stream=stream)

    def verify(self, stream=None):
        i, o = self.inp, self.out
        if self.layout == "raw":
            self.h.verify_accept_raw(i["hn"], i["Wl"], o["node_tok"], o["kept"], o["nka"], o["n_nodes"],
                                     o["argmax"], o["acc_len"], o["acc_nodes"], o["acc_tok"], o["next_tok"],
                                     o.get("lm_logits_dbg"), stream=stream)
            return
        self.h.verify_accept(i["hn"], i["Wl"], o["node_tok"], o["parent"], o["n_nodes"],
                             o["argmax"], o["acc_len"], o["acc_nodes"], o["acc_tok"], o["next_tok"],
                             o.get("lm_logits_dbg"), stream=stream)

    def verify_sampled(self, noise, temperature, stream=None):
        """Sampling acceptance in place of the greedy one (packed layout): out["argmax"] then holds
        the sampled tokens."""
        i, o = self.inp, self.out
        self.h.verify_accept_sampled(i["hn"], i["Wl"], o["node_tok"], o["parent"], o["depth"], o["n_nodes"],
                                     noise, temperature, o["argmax"], o["acc_len"], o["acc_nodes"], o["acc_tok"],
                                     o["next_tok"], o.get("lm_logits_dbg"), stream=stream)

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

    # chained steps ----------------------------------------------------------------------
    CHAIN_RECORDED = ("topk_id", "topk_lp", "cand_tok", "cand_len", "cand_score", "n_cand", "node_tok", "parent",
                      "depth", "pos", "mask", "retrieve", "n_nodes", "O", "argmax", "acc_len", "acc_nodes", "acc_tok",
                      "next_tok", "new_kv_len", "next_sel_row")

    def setup_chain(self, n_steps: int, x0, base_tok0, kv_len0, Qtab, Ktab, Vtab, hntab, record: bool = True):
        """Device-side state of n_steps chained steps (history update after every step, no host work
        in between).  x0 [B,H], base_tok0 [B], kv_len0 [B]: where the chain starts.  The per-step
        tables stand in for the base model: Qtab [S,B,max_nodes,Hq,D] tree-node queries, Ktab/Vtab
        [S,B,Hkv,max_nodes,D] tree-node keys/values, hntab [S,B*max_nodes,H] tree-node hidden states.
        K, V (the cache, updated in place), Wd, Wl, blank_bias come from set_inputs()."""
        cfg, dev = self.cfg, self.device
        self.chain = dict(n=n_steps, x0=x0, base_tok0=base_tok0, kv_len0=kv_len0, Qtab=Qtab, Ktab=Ktab, Vtab=Vtab,
                          hntab=hntab, kv_len=kv_len0.clone(), kv_before=None, rec=None,
                          node_off=torch.arange(cfg.max_nodes, device=dev, dtype=torch.int64))
        if record:
            self.chain["rec"] = {k: torch.zeros((n_steps,) + tuple(self.out[k].shape), dtype=self.out[k].dtype,
                                                device=dev) for k in self.CHAIN_RECORDED if k in self.out}
            self.chain["kv_before"] = torch.zeros(n_steps, cfg.B, dtype=torch.int32, device=dev)
            if self.layout == "raw":
                for k in ("kept", "nka"):
                    self.chain["rec"][k] = torch.zeros((n_steps,) + tuple(self.out[k].shape), dtype=torch.int32,
                                                       device=dev)

    def write_tree_kv(self, s: int):
        """Stand-in for the base model's key/value projection of step s: node j's key and value go
        to cache row kv_len[b]+j (device-side indices, no host work)."""
        c, cfg = self.chain, self.cfg
        rows = c["kv_len"].to(torch.int64)[:, None] + c["node_off"][None, :]                    # [B,n]
        idx = rows[:, None, :, None].expand(cfg.B, cfg.Hkv, cfg.max_nodes, cfg.D)
        self.inp["K"].scatter_(2, idx, c["Ktab"][s])
        self.inp["V"].scatter_(2, idx, c["Vtab"][s])

    def chain_head(self, s: int):
        """Step s of the chain up to the token tree: draft head, candidates, tree."""
        c, i, o = self.chain, self.inp, self.out
        i["kv_len"] = c["kv_len"]
        i["sel_row"] = None
        if s == 0:
            i["base_tok"] = c["base_tok0"]
            self.h.draft_logits(c["x0"], i["Wd"], None, i.get("blank_bias"), o["topk_id"], o["topk_lp"], o["lse"])
        else:
            i["base_tok"] = o["next_tok"]              # the previous step's bonus token is this step's root
            self.h.draft_logits_rows(c["hntab"][s - 1], o["next_sel_row"], i["Wd"], None, i.get("blank_bias"),
                                     o["topk_id"], o["topk_lp"], o["lse"])
        self.collapse()
        self.tree()

    def chain_tail(self, s: int):
        """The rest of step s: the base model's stand-in writes the tree's keys/values, then tree
        attention, LM head + acceptance, and the history update."""
        c, i, o = self.chain, self.inp, self.out
        self.write_tree_kv(s)
        i["Q"] = c["Qtab"][s]
        i["hn"] = c["hntab"][s]
        self.attention()
        self.verify()
        if c["kv_before"] is not None:
            c["kv_before"][s].copy_(c["kv_len"])
        # the new length overwrites the old one in place; the next step drafts from out["next_sel_row"]
        self.h.commit_accepted(i["K"], i["V"], c["kv_len"], o["acc_len"], o["acc_nodes"], c["kv_len"],
                               o["next_sel_row"])
        if c["rec"] is not None:
            o["new_kv_len"].copy_(c["kv_len"])
            for k, buf in c["rec"].items():
                buf[s].copy_(o[k])

    def run_chain(self):
        """All steps of the chain back to back on the current stream: per step the five calls and
        the history update, the next step reading its drafting row, root token and cache length
        from what the previous one left on the device."""
        c = self.chain
        c["kv_len"].copy_(c["kv_len0"])
        for s in range(c["n"]):
            self.chain_head(s)
            self.chain_tail(s)

    def plant_chain_hidden(self, seed: int, Wl_host: np.ndarray):
        """Fills the chain's table of tree-node hidden states so that the base model agrees with the
        drafts at the configured rate.  The hidden states of step s depend on the tree of step s,
        which depends on what earlier steps accepted, so this walks the chain once with a host
        round trip per step (set-up only; run_chain() then needs none)."""
        from . import synth
        c, cfg = self.chain, self.cfg
        c["kv_len"].copy_(c["kv_len0"])
        for s in range(c["n"]):
            self.chain_head(s)
            self.check_status()
            parent = self.host("parent")
            if self.layout == "raw":
                parent = np.where(self.host("kept") != 0, self.host("nka"), -1)
            hn, _ = synth.gen_node_hidden(cfg, synth.chain_step_seed(seed, s), Wl_host, self.host("node_tok"),
                                          parent, self.host("n_nodes"))
            c["hntab"][s].copy_(to_device(hn, cfg.dtype, self.device))
            self.chain_tail(s)
        self.check_status()

    def check_status(self):
        st = self.h.poll_status()
        if st != 0:
            raise binding.CtcsdError("device status %d: %s" % (st, self.h.lib.ctcsd_strerror(st).decode()))

    def host(self, name: str) -> np.ndarray:
        t = self.out[name]
        if t.dtype == torch.bfloat16:
            t = t.float()
        return t.cpu().numpy()
