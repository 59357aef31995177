"""Shared machinery of the GPU parity tests: run the CUDA path through the C ABI on seeded
inputs and compare every stage with the CPU oracle.

Two comparisons per stage:
  * definition mode - the oracle starts from the raw inputs in fp64; floats must agree within
    the stated tolerances;
  * stage-fed mode  - the oracle is given the CUDA path's own output of the previous stage
    (e.g. its fp32 logits), and every integer output must then match bit for bit.
"""
from __future__ import annotations

import math
from typing import Optional

import numpy as np
import torch

from oracle import ctcsd_oracle as orc
from paper_2412_00061_b200 import synth
from paper_2412_00061_b200.step import DraftVerifyStep, to_device

TAU = 1e-9          # score gaps below this make the candidate order a tie (fp64 on both sides)


def tolerances(dtype: str):
    # max-abs error on logits / attention outputs, relative error on log-probs
    return (2e-2, 1e-4) if dtype == "bf16" else (2e-4, 1e-4)


def make_inputs(cfg, seed, M=None, force_repeats=False, row_seq=None, sel_row=None):
    x, Wd, bb = synth.gen_draft(cfg, seed, M=M, force_repeats=force_repeats)
    base_tok, kv_len = synth.gen_base(cfg, seed)
    Q, K, V = synth.gen_attention(cfg, seed)
    Wl = synth.gen_lm_head(cfg, seed)
    return dict(x=x, Wd=Wd, blank_bias=bb, base_tok=base_tok, kv_len=kv_len, Q=Q, K=K, V=V, Wl=Wl,
                row_seq=row_seq, sel_row=sel_row)


def check_topk(z_gpu, ids_gpu, lp_gpu, lse_gpu, k, rel):
    """Stage-fed check of S2/S3: selection must be exact w.r.t. the kernel's own logits."""
    ids_o, lp_o = orc.topk_slots(z_gpu.astype(np.float64), k)
    lse_o, _ = orc.log_softmax_slots(z_gpu.astype(np.float64))
    np.testing.assert_array_equal(ids_gpu, ids_o)
    np.testing.assert_allclose(lse_gpu, lse_o, rtol=rel, atol=1e-6)
    np.testing.assert_allclose(lp_gpu, lp_o, rtol=rel, atol=1e-6)


def check_candidates(cfg, topk_id, topk_lp, sel_row, got, require_certified=False):
    """Stage-fed check of S4-S7 against the oracle fed the CUDA path's top-k lists."""
    cand_tok, cand_len, cand_score, n_cand = got
    st = {}
    o_tok, o_len, o_score, o_n = orc.topk_collapse(
        topk_id.astype(np.int64), topk_lp.astype(np.float64), blank=cfg.V, T=cfg.T, N=cfg.topN,
        beam=cfg.beam, score_mode=cfg.score_mode, sel_row=sel_row, B=cfg.B, stats=st)
    certified = True
    for b in range(cfg.B):
        if st["margin"][b] > TAU:
            np.testing.assert_array_equal(cand_tok[b], o_tok[b])
            np.testing.assert_array_equal(cand_len[b], o_len[b])
            assert n_cand[b] == o_n[b]
            n = int(o_n[b])
            np.testing.assert_allclose(cand_score[b, :n], o_score[b, :n], rtol=1e-5, atol=1e-6)
            assert np.all(np.isneginf(cand_score[b, n:]))
        else:
            # several orders are correct: accept any that is valid within TAU
            certified = False
            assert cfg.beam == 0, "beam cut inside a tie: pick another seed"
            r = b if sel_row is None else int(sel_row[b])
            exact = orc.enumerate_candidates(topk_id[r].astype(np.int64), topk_lp[r].astype(np.float64),
                                             cfg.V, cfg.score_mode)
            exact = {y: s for y, s in exact.items() if len(y) > 0}
            n = int(n_cand[b])
            assert n == min(cfg.topN, len(exact))
            kept = []
            for c in range(n):
                y = tuple(int(v) for v in cand_tok[b, c, :cand_len[b, c]])
                assert y in exact and y not in kept
                assert abs(exact[y] - cand_score[b, c]) <= 1e-5 * max(1.0, abs(exact[y]))
                kept.append(y)
            sc = [exact[y] for y in kept]
            assert all(sc[i] >= sc[i + 1] - TAU for i in range(n - 1))
            assert all(s <= min(sc) + TAU for y, s in exact.items() if y not in kept)
    if require_certified:
        assert certified, "headline seeds must be free of score ties"
    return certified


def run_parity(cfg, seed=0, M=None, force_repeats=False, row_seq=None, sel_row=None, device="cuda:0",
               require_certified=False, attention_rows: Optional[int] = None, lm_rows: Optional[int] = None,
               draft_rows=None):
    """Runs the five calls on the GPU and checks every output against the oracle.
    attention_rows / lm_rows / draft_rows bound the work of the definition-mode oracle at
    large shapes by sampling (sequence, head) pairs / node rows / draft rows."""
    logit_tol, rel = tolerances(cfg.dtype)
    inp = make_inputs(cfg, seed, M, force_repeats, row_seq, sel_row)
    Mrows = inp["x"].shape[0]
    step = DraftVerifyStep(cfg, device=device, max_draft_rows=Mrows, debug_logits=True)
    dev = step.device
    i32 = lambda a: None if a is None else torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    step.set_inputs(
        x=to_device(inp["x"], cfg.dtype, dev), Wd=to_device(inp["Wd"], cfg.dtype, dev),
        blank_bias=torch.from_numpy(inp["blank_bias"]).to(dev), row_seq=i32(row_seq), sel_row=i32(sel_row),
        base_tok=i32(inp["base_tok"]), kv_len=i32(inp["kv_len"]),
        Q=to_device(inp["Q"], cfg.dtype, dev), K=to_device(inp["K"], cfg.dtype, dev),
        V=to_device(inp["V"], cfg.dtype, dev), Wl=to_device(inp["Wl"], cfg.dtype, dev))

    # ---- S1-S3 --------------------------------------------------------------------------
    step.draft()
    step.check_status()
    z_gpu = step.host("draft_logits_dbg")
    rows = list(range(Mrows)) if draft_rows is None else list(draft_rows)
    rs = np.arange(Mrows) if row_seq is None else np.asarray(row_seq)
    z_def = orc.draft_logits(inp["x"][rows], inp["Wd"], inp["blank_bias"], rs[rows])
    assert np.max(np.abs(z_gpu[rows] - z_def)) <= logit_tol
    check_topk(z_gpu, step.host("topk_id"), step.host("topk_lp"), step.host("lse"), cfg.k, rel)

    # ---- S4-S7 --------------------------------------------------------------------------
    step.collapse()
    step.check_status()
    got = (step.host("cand_tok"), step.host("cand_len"), step.host("cand_score"), step.host("n_cand"))
    certified = check_candidates(cfg, step.host("topk_id"), step.host("topk_lp"), sel_row, got, require_certified)

    # ---- S8 -----------------------------------------------------------------------------
    step.tree()
    step.check_status()
    o_tree = orc.build_tree(inp["base_tok"], inp["kv_len"], got[0].astype(np.int64), got[1].astype(np.int64),
                            got[3].astype(np.int64), cfg.max_nodes)
    names = ["node_tok", "parent", "depth", "pos", "mask", "retrieve", "n_nodes"]
    for name, want in zip(names, o_tree):
        have = step.host(name)
        if name == "mask":
            have = have.view(np.uint64)
        np.testing.assert_array_equal(have, want, err_msg=name)
    node_tok, parent, depth, pos, mask, retrieve, n_nodes = o_tree

    # ---- S9 -----------------------------------------------------------------------------
    step.attention()
    step.check_status()
    O_gpu = step.host("O")
    if attention_rows is None:
        O_def = orc.tree_attention(inp["Q"], inp["K"], inp["V"], inp["kv_len"], n_nodes, mask, 1.0 / math.sqrt(cfg.D))
        assert np.max(np.abs(O_gpu - O_def)) <= logit_tol
    else:
        rng = np.random.default_rng(seed + 77)
        for _ in range(attention_rows):                 # sampled (sequence, head) pairs, all nodes each
            b = int(rng.integers(0, cfg.B))
            h = int(rng.integers(0, cfg.Hq))
            g = h // (cfg.Hq // cfg.Hkv)
            one = orc.tree_attention(inp["Q"][b:b + 1, :, h:h + 1], inp["K"][b:b + 1, g:g + 1],
                                     inp["V"][b:b + 1, g:g + 1], inp["kv_len"][b:b + 1], n_nodes[b:b + 1],
                                     mask[b:b + 1], 1.0 / math.sqrt(cfg.D))
            assert np.max(np.abs(O_gpu[b, :, h] - one[0, :, 0])) <= logit_tol
        dead = [(b, i) for b in range(cfg.B) for i in range(int(n_nodes[b]), cfg.max_nodes)]
        for b, i in dead[:64]:
            assert np.all(O_gpu[b, i] == 0)

    # ---- S10-S11 ------------------------------------------------------------------------
    hn, target = synth.gen_node_hidden(cfg, seed, inp["Wl"], node_tok, parent, n_nodes)
    step.set_inputs(hn=to_device(hn, cfg.dtype, dev))
    step.verify()
    step.check_status()
    y_gpu = step.host("lm_logits_dbg")
    live = [b * cfg.max_nodes + i for b in range(cfg.B) for i in range(int(n_nodes[b]))]
    rows = live
    if lm_rows is not None and len(live) > lm_rows:
        rows = [live[j] for j in np.random.default_rng(seed + 5).choice(len(live), lm_rows, replace=False)]
    y_def, am_def = orc.lm_head_argmax(hn[rows], inp["Wl"])
    assert np.max(np.abs(y_gpu[rows] - y_def)) <= logit_tol
    am_gpu = step.host("argmax")
    np.testing.assert_array_equal(am_gpu.reshape(-1), orc.argmax_rows(y_gpu))           # stage-fed, all rows
    np.testing.assert_array_equal(am_gpu.reshape(-1)[rows], am_def)                      # definition mode
    np.testing.assert_array_equal(am_gpu.reshape(-1)[live], target.reshape(-1)[live])    # the planted targets
    acc = orc.greedy_accept(node_tok, parent, n_nodes, am_gpu.astype(np.int64), cfg.T)
    for name, want in zip(["acc_len", "acc_nodes", "acc_tok", "next_tok"], acc):
        np.testing.assert_array_equal(step.host(name), want, err_msg=name)
    assert np.all(acc[0] <= np.array([depth[b, :n_nodes[b]].max() for b in range(cfg.B)]))
    assert np.all(acc[0] <= cfg.T)

    # ---- the whole step again in one go: same integers (determinism, no stale state) -------
    before = {k: step.host(k).copy() for k in ["topk_id", "cand_tok", "node_tok", "mask", "argmax", "acc_len", "acc_tok", "next_tok"]}
    step.run()
    step.check_status()
    for k, v in before.items():
        np.testing.assert_array_equal(step.host(k), v, err_msg="rerun " + k)
    return dict(certified=certified, acc_len=acc[0], n_nodes=n_nodes, step=step)


def run_parity_raw(cfg, seed=0, force_repeats=False, device="cuda:0", attention_rows: Optional[int] = None,
                   lm_rows: Optional[int] = None):
    """The paper's raw-tree layout (Sec. 3.3) through the C ABI against the oracle: raw-path
    selection, raw tree with the transform's mask, attention under that mask, acceptance over
    the kept nodes.  Integer outputs are compared bit for bit (the oracle is fed the CUDA path's
    previous-stage output); path scores are float64 sums of the same float32 terms in the same
    order on both sides, so even the order of equal scores must agree."""
    logit_tol, rel = tolerances(cfg.dtype)
    inp = make_inputs(cfg, seed, None, force_repeats, None, None)
    step = DraftVerifyStep(cfg, device=device, debug_logits=True, layout="raw")
    dev = step.device
    i32 = lambda a: None if a is None else torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    step.set_inputs(
        x=to_device(inp["x"], cfg.dtype, dev), Wd=to_device(inp["Wd"], cfg.dtype, dev),
        blank_bias=torch.from_numpy(inp["blank_bias"]).to(dev), row_seq=None, sel_row=None,
        base_tok=i32(inp["base_tok"]), kv_len=i32(inp["kv_len"]),
        Q=to_device(inp["Q"], cfg.dtype, dev), K=to_device(inp["K"], cfg.dtype, dev),
        V=to_device(inp["V"], cfg.dtype, dev), Wl=to_device(inp["Wl"], cfg.dtype, dev))
    step.draft()
    step.check_status()
    check_topk(step.host("draft_logits_dbg"), step.host("topk_id"), step.host("topk_lp"), step.host("lse"), cfg.k, rel)

    # ---- raw-path selection -----------------------------------------------------------------
    step.collapse()
    step.check_status()
    tid, tlp = step.host("topk_id").astype(np.int64), step.host("topk_lp").astype(np.float64)
    raw_tok, raw_score, n_raw = step.host("cand_tok"), step.host("cand_score"), step.host("n_cand")
    for b in range(cfg.B):
        want_tok, want_score = orc.select_raw_paths(tid[b], tlp[b], cfg.topN)
        n = want_tok.shape[0]
        assert n_raw[b] == n == min(cfg.topN, cfg.k ** cfg.T)
        np.testing.assert_array_equal(raw_tok[b, :n], want_tok)
        np.testing.assert_allclose(raw_score[b, :n], want_score, rtol=1e-6, atol=1e-6)
        assert np.all(raw_tok[b, n:] == -1) and np.all(np.isneginf(raw_score[b, n:]))

    # ---- raw tree ---------------------------------------------------------------------------
    step.tree()
    step.check_status()
    o_tree = orc.build_raw_tree(inp["base_tok"], inp["kv_len"], raw_tok.astype(np.int64), n_raw.astype(np.int64),
                                cfg.V, cfg.max_nodes)
    names = ["node_tok", "parent", "depth", "pos", "mask", "retrieve", "n_nodes", "kept", "nka"]
    for name, want in zip(names, o_tree):
        have = step.host(name)
        if name == "mask":
            have = have.view(np.uint64)
        np.testing.assert_array_equal(have, want, err_msg=name)
    node_tok, parent, depth, pos, mask, retrieve, n_nodes, kept, nka = o_tree

    # ---- attention under the transform's mask -------------------------------------------------
    step.attention()
    step.check_status()
    O_gpu = step.host("O")
    if attention_rows is None:
        O_def = orc.tree_attention(inp["Q"], inp["K"], inp["V"], inp["kv_len"], n_nodes, mask, 1.0 / math.sqrt(cfg.D))
        assert np.max(np.abs(O_gpu - O_def)) <= logit_tol
    else:
        rng = np.random.default_rng(seed + 77)
        for _ in range(attention_rows):
            b = int(rng.integers(0, cfg.B))
            h = int(rng.integers(0, cfg.Hq))
            g = h // (cfg.Hq // cfg.Hkv)
            one = orc.tree_attention(inp["Q"][b:b + 1, :, h:h + 1], inp["K"][b:b + 1, g:g + 1],
                                     inp["V"][b:b + 1, g:g + 1], inp["kv_len"][b:b + 1], n_nodes[b:b + 1],
                                     mask[b:b + 1], 1.0 / math.sqrt(cfg.D))
            assert np.max(np.abs(O_gpu[b, :, h] - one[0, :, 0])) <= logit_tol

    # ---- LM head + acceptance over the kept nodes -----------------------------------------------
    follows = np.where(kept != 0, nka, -1)          # who a node may follow; removed nodes follow nobody
    hn, target = synth.gen_node_hidden(cfg, seed, inp["Wl"], node_tok, follows, n_nodes)
    step.set_inputs(hn=to_device(hn, cfg.dtype, dev))
    step.verify()
    step.check_status()
    y_gpu = step.host("lm_logits_dbg")
    live = [b * cfg.max_nodes + i for b in range(cfg.B) for i in range(int(n_nodes[b]))]
    rows = live
    if lm_rows is not None and len(live) > lm_rows:
        rows = [live[j] for j in np.random.default_rng(seed + 5).choice(len(live), lm_rows, replace=False)]
    y_def, am_def = orc.lm_head_argmax(hn[rows], inp["Wl"])
    assert np.max(np.abs(y_gpu[rows] - y_def)) <= logit_tol
    am_gpu = step.host("argmax")
    np.testing.assert_array_equal(am_gpu.reshape(-1), orc.argmax_rows(y_gpu))
    np.testing.assert_array_equal(am_gpu.reshape(-1)[live], target.reshape(-1)[live])
    acc = orc.raw_accept(node_tok, kept, nka, n_nodes, am_gpu.astype(np.int64), cfg.T)
    for name, want in zip(["acc_len", "acc_nodes", "acc_tok", "next_tok"], acc):
        np.testing.assert_array_equal(step.host(name), want, err_msg=name)
    # accepted nodes are kept, their positions are consecutive after the root's
    for b in range(cfg.B):
        for l in range(int(acc[0][b])):
            d = int(acc[1][b, l])
            assert kept[b, d] == 1 and pos[b, d] == inp["kv_len"][b] + l + 1

    before = {k: step.host(k).copy() for k in ["cand_tok", "node_tok", "mask", "kept", "nka", "argmax", "acc_len", "acc_tok", "next_tok"]}
    step.run()
    step.check_status()
    for k, v in before.items():
        np.testing.assert_array_equal(step.host(k), v, err_msg="rerun " + k)
    return dict(acc_len=acc[0], n_nodes=n_nodes, kept=kept, step=step)
