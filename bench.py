#!/usr/bin/env python
"""Benchmark of the draft-and-verify step (the five C-ABI calls back to back on one stream).

Default workload: the Vicuna-7B-shaped step (batch 1, hidden 4096, vocab 32000 + blank, T=5,
top-k 4, top-N 16, <= 64-node tree, 32 heads x 128 over 1024 cached tokens, bf16).  One
"step" is one pass S1..S11 over synthetic, seeded inputs that are resident in HBM.  With
N > 1 GPUs every rank runs its own replica of the step on its own sequences (the path is
independent per sequence: no collective on the data path), so the aggregate is N x.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import datetime
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")


def ncu_traffic(workload: str, kernel: str):
    """DRAM bytes (read + write) of one launch of `kernel` on `workload`, as counted by ncu and
    recorded in profiles/traffic.json by paper_2412_00061_b200/ncu_traffic.py, or None when no
    record exists or a source file of the kernel has changed since the counters were taken (the
    record carries the files' SHA-256)."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(workload, {}).get(kernel)
    except (OSError, ValueError):
        return None
    if not rec:
        return None
    for rel, want in rec.get("source_sha256", {}).items():
        try:
            with open(os.path.join(ROOT, rel), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != want:
                    return None
        except OSError:
            return None
    return rec.get("traffic_bytes")


METRIC = "draft+verify steps/s at 7B shape (batch 1, 64-node tree)"
UNIT = "steps/s"


def algorithmic_bytes(cfg, mean_kv_len, n_live):
    """Bytes the method must move per step: every draft-head and LM-head weight once, every
    live key/value row once (activations, lists and tree arrays are < 0.1 %)."""
    esz = 2 if cfg.dtype == "bf16" else 4
    draft = cfg.T * (cfg.V + 1) * cfg.H * esz
    lm = cfg.V * cfg.H * esz
    kv = 2 * cfg.B * cfg.Hkv * (mean_kv_len + n_live) * cfg.D * esz
    return draft, lm, kv


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run.
    It is started before the warm-up (nvidia-smi needs a moment to come up); only samples whose
    timestamp falls inside a window opened with begin() and closed with end() are kept."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 10):
        self.windows = []
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", str(period_ms)],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def begin(self):
        self._t0 = datetime.datetime.now()

    def end(self):
        self.windows.append((self._t0, datetime.datetime.now()))

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        clocks, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                clk, cmx = float(parts[1]), float(parts[2])
            except ValueError:
                continue
            if not any(a <= ts <= b for a, b in self.windows):
                continue
            clocks.append(clk)
            mx = cmx
            for nme, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        self.f.close()
        os.unlink(self.f.name)
        if clocks:
            out["sm_mhz"] = float(np.median(clocks))
            out["sm_max_mhz"] = mx
            out["reasons"] = sorted(reasons)
            out["samples"] = len(clocks)
        return out


def oracle_step(cfg, inp, layout="packed"):
    """One pass of the CPU oracle over the step (definition mode, fp64).  Returns nothing:
    it is only timed."""
    import math

    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200 import synth
    z = orc.draft_logits(inp["x"], inp["Wd"], inp["blank_bias"])
    ids, lps = orc.topk_slots(z, cfg.k)
    if layout == "raw":
        raw = [orc.select_raw_paths(ids[b], lps[b], cfg.topN)[0] for b in range(cfg.B)]
        n_raw = np.array([r.shape[0] for r in raw])
        tree = orc.build_raw_tree(inp["base_tok"], inp["kv_len"], np.stack(raw), n_raw, cfg.V, cfg.max_nodes)
        node_tok, parent, depth, pos, mask, retrieve, n_nodes, kept, nka = tree
        orc.tree_attention(inp["Q"], inp["K"], inp["V"], inp["kv_len"], n_nodes, mask, 1.0 / math.sqrt(cfg.D))
        if "hn" not in inp:
            inp["hn"], _ = synth.gen_node_hidden(cfg, 0, inp["Wl"], node_tok, np.where(kept != 0, nka, -1), n_nodes)
        _, am = orc.lm_head_argmax(inp["hn"], inp["Wl"])
        orc.raw_accept(node_tok, kept, nka, n_nodes, am.reshape(cfg.B, cfg.max_nodes), cfg.T)
        return
    ctok, clen, cscore, nc = orc.topk_collapse(ids, lps, cfg.V, cfg.T, cfg.topN, cfg.beam, cfg.score_mode)
    tree = orc.build_tree(inp["base_tok"], inp["kv_len"], ctok, clen, nc, cfg.max_nodes)
    node_tok, parent, depth, pos, mask, retrieve, n_nodes = tree
    orc.tree_attention(inp["Q"], inp["K"], inp["V"], inp["kv_len"], n_nodes, mask, 1.0 / math.sqrt(cfg.D))
    if "hn" not in inp:
        inp["hn"], _ = synth.gen_node_hidden(cfg, 0, inp["Wl"], node_tok, parent, n_nodes)
    _, am = orc.lm_head_argmax(inp["hn"], inp["Wl"])
    orc.greedy_accept(node_tok, parent, n_nodes, am.reshape(cfg.B, cfg.max_nodes), cfg.T)


def host_inputs(cfg, seed, force_repeats=False):
    from paper_2412_00061_b200 import synth
    x, Wd, bb = synth.gen_draft(cfg, seed, force_repeats=force_repeats)
    base_tok, kv_len = synth.gen_base(cfg, seed)
    Q, K, V = synth.gen_attention(cfg, seed)
    Wl = synth.gen_lm_head(cfg, seed)
    return dict(x=x, Wd=Wd, blank_bias=bb, base_tok=base_tok, kv_len=kv_len, Q=Q, K=K, V=V, Wl=Wl)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle(cfg, inp, steps, warmup, layout="packed"):
    for _ in range(warmup):
        oracle_step(cfg, inp, layout=layout)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(cfg, inp, layout=layout)
    return (time.perf_counter() - t0) / steps


def run_reference(args):
    """The CPU oracle as it stands, timed on the host cores.  Each step is one full pass of
    the oracle over the same workload (about two seconds at the 7B shape)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2412_00061_b200 import synth
    cfg = workload_config(args)
    inp = host_inputs(cfg, 0, args.force_repeats)
    steps = max(1, min(args.steps, 20))
    warmup = max(1, min(args.warmup, 2))
    sec = time_oracle(cfg, inp, steps, warmup, args.layout)
    val = 1.0 / sec
    cores = blas_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "layout": args.layout, "sample": "whole step, all stages"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "%d full steps of the fp64 oracle (numpy, BLAS threads = cores)" % steps},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_name(cfg):
    return ("%s: B=%d H=%d V=%d+blank T=%d k=%d %s topN=%d nodes<=%d heads=%d/%d x%d kv=%d..%d %s"
            % (cfg.name, cfg.B, cfg.H, cfg.V, cfg.T, cfg.k,
               "enumerate" if cfg.beam == 0 else "beam=%d" % cfg.beam, cfg.topN, cfg.max_nodes,
               cfg.Hq, cfg.Hkv, cfg.D, cfg.kv_lo, cfg.kv_hi, cfg.dtype))


def workload_config(args):
    from paper_2412_00061_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.blank_bias is not None:
        cfg = cfg.replace(blank_bias=(float(args.blank_bias),))
    return cfg


def stage_times_us(step, torch, repeats=20, replays=10):
    """Device time of each call of the step on its own: `repeats` back-to-back launches of the
    call in a CUDA graph, replayed `replays` times (the weights exceed L2, so every launch
    streams from HBM)."""
    out = {}
    side = torch.cuda.Stream(device=step.device)
    for name, fn in (("draft_logits", step.draft), ("topk_collapse", step.collapse), ("build_tree", step.tree),
                     ("tree_attention", step.attention), ("verify_accept", step.verify), ("whole_step", step.run)):
        with torch.cuda.stream(side):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for _ in range(repeats):
                    fn()
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(replays):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / (repeats * replays)
    return out


def roofline_times_us(cfg, mean_kv, n_live, hbm_gbs, tensor_tflops):
    """Per heavy call: the slower of (algorithmic bytes / measured copy bandwidth) and
    (flops / measured bf16 matmul rate); the step's roofline time is their sum."""
    draft_b, lm_b, kv_b = algorithmic_bytes(cfg, mean_kv, n_live)
    M_lm = cfg.B * n_live               # rows the LM head must serve: the live tree nodes
    fl = {"draft_logits": 2.0 * cfg.B * cfg.T * (cfg.V + 1) * cfg.H,
          "verify_accept": 2.0 * M_lm * cfg.V * cfg.H,
          "tree_attention": 4.0 * cfg.B * cfg.Hq * n_live * (mean_kv + n_live) * cfg.D}
    by = {"draft_logits": draft_b, "verify_accept": lm_b, "tree_attention": kv_b}
    out = {k: max(by[k] / (hbm_gbs * 1e9), fl[k] / (tensor_tflops * 1e12)) * 1e6 for k in by}
    out["whole_step"] = sum(out.values())
    return out


def chain_tokens_per_s(args, cfg, step, inp, seed, torch, to_device, synth):
    """--chain n: n chained steps (five calls + history update each, the next step starting from
    what the previous one left on the device) captured in one CUDA graph and replayed; tokens/s =
    emitted tokens (accepted drafts + one bonus token per step and sequence) over device time."""
    n, dev = args.chain, step.device
    big = synth.chain_cache_config(cfg, n)
    _, K, V = synth.gen_attention(big, seed)
    Qtab, Ktab, Vtab = synth.gen_chain_tables(cfg, seed, n)
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    K0, V0 = to_device(K, cfg.dtype, dev), to_device(V, cfg.dtype, dev)
    step.set_inputs(K=K0.clone(), V=V0.clone())
    act = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    hntab = torch.zeros(n, cfg.B * cfg.max_nodes, cfg.H, dtype=act, device=dev)
    step.setup_chain(n, to_device(inp["x"], cfg.dtype, dev), i32(inp["base_tok"]), i32(inp["kv_len"]),
                     to_device(Qtab, cfg.dtype, dev), to_device(Ktab, cfg.dtype, dev), to_device(Vtab, cfg.dtype, dev),
                     hntab, record=True)
    step.plant_chain_hidden(seed, inp["Wl"])
    side = torch.cuda.Stream(device=dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step.run_chain()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            step.run_chain()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    reps = max(1, min(50, args.steps // n))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    step.check_status()
    acc = step.chain["rec"]["acc_len"].cpu().numpy()            # [n, B]
    tokens = int(acc.sum()) + n * cfg.B
    sec = e0.elapsed_time(e1) * 1e-3 / reps
    return {"steps": n, "replays": reps, "tokens_per_s": tokens / sec, "tokens_per_step": tokens / (n * cfg.B),
            "us_per_step": sec * 1e6 / n, "includes": "torch scatter standing in for the base model's K/V write of the tree rows"}


def draft_module_time(args, cfg, step, seed, torch, to_device, synth):
    """--draft-module: the paper's attention draft module (one decoder layer before the draft head,
    Sec. 3.1) at the workload's shape with a LLaMA-style MLP width, timed alone (20 calls per CUDA
    graph).  Reports its time, the weight bytes it streams and its share of (layer + step), the
    figure the paper gives for its own drafter (Sec. 4.3)."""
    dev = step.device
    I = {4096: 11008, 5120: 13824, 8192: 28672}.get(cfg.H, (cfg.H * 8 // 3 + 255) // 256 * 256)
    R = cfg.T + 1
    w, F_new, n_new, kv_len, Kd, Vd = synth.gen_draft_layer(cfg, seed, I, R, cfg.kv_lo, cfg.kv_hi)
    td = lambda a: to_device(a, cfg.dtype, dev)
    f32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float32)).to(dev)
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    dl = step.h.make_draft_layer(f32(w["g1"]), td(w["Wqkv"]), td(w["Wo"]), f32(w["g2"]), td(w["Wgu"]), td(w["Wdn"]), R=R)
    act = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    args_d = (dl, td(F_new), i32(n_new), i32(kv_len), td(Kd), td(Vd), torch.zeros(cfg.B, cfg.H, dtype=act, device=dev),
              torch.zeros(cfg.B, dtype=torch.int32, device=dev))
    fn = lambda: step.h.draft_module(*args_d)
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(20):
                fn()
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
    step.check_status()
    us = e0.elapsed_time(e1) * 1e3 / 200
    esz = 2 if cfg.dtype == "bf16" else 4
    wbytes = esz * (((cfg.Hq + 2 * cfg.Hkv) * cfg.D + cfg.Hq * cfg.D) * cfg.H + 3 * I * cfg.H)
    return {"us": us, "mlp_width": I, "new_rows": R, "weight_bytes": wbytes, "GBps": wbytes / us / 1e3}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2412_00061_b200 import binding, build, replicas, synth
    from paper_2412_00061_b200.step import DraftVerifyStep, to_device

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    build.build()
    binding.load_library()

    cfg = workload_config(args)
    seed = replicas.rank_seed(0, rank)             # every rank drafts for its own sequences
    inp = host_inputs(cfg, seed, args.force_repeats)
    step = DraftVerifyStep(cfg, device=str(dev), layout=args.layout)
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    step.set_inputs(x=to_device(inp["x"], cfg.dtype, dev), Wd=to_device(inp["Wd"], cfg.dtype, dev),
                    blank_bias=torch.from_numpy(inp["blank_bias"]).to(dev),
                    base_tok=i32(inp["base_tok"]), kv_len=i32(inp["kv_len"]),
                    Q=to_device(inp["Q"], cfg.dtype, dev), K=to_device(inp["K"], cfg.dtype, dev),
                    V=to_device(inp["V"], cfg.dtype, dev), Wl=to_device(inp["Wl"], cfg.dtype, dev))
    # tree-node hidden states need the tree: build it once on the GPU, outside the timed loop
    step.draft(); step.collapse(); step.tree()
    step.check_status()
    node_tok, parent, n_nodes = step.host("node_tok"), step.host("parent"), step.host("n_nodes")
    if args.layout == "raw":      # a kept node follows its nearest kept ancestor; removed nodes follow nobody
        parent = np.where(step.host("kept") != 0, step.host("nka"), -1)
    hn, _ = synth.gen_node_hidden(cfg, seed, inp["Wl"], node_tok, parent, n_nodes)
    inp["hn"] = hn
    step.set_inputs(hn=to_device(hn, cfg.dtype, dev))
    # how much the inputs exercise the CTC transform: distinct candidates out of k^T slot paths
    n_cand = step.host("n_cand")
    cand_len = step.host("cand_len") if args.layout == "packed" else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K, Wm = args.steps, max(3, args.warmup)
    sampler = ClockSampler(local, args.clock_period_ms) if rank == 0 else None
    for _ in range(Wm):
        step.run()
    step.check_status()

    # ---- device-timed region: inputs resident in HBM -----------------------------------
    # The five calls of a step are captured once into a CUDA graph of S steps and replayed
    # K / S times (the library only enqueues kernels on the caller's stream, so it captures
    # like any stream work).  Events recorded inside the graph bracket every draft-head launch;
    # after the last replay they hold that replay's S launch times.
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_beg, t_end = ev(), ev()
    use_graph = not args.no_graph
    S = 1
    if use_graph:                 # at least two replays per timed region when K allows it
        S = max(d for d in range(1, 21) if K % d == 0 and (d <= K // 2 or K < 2))
    d_beg = [torch.cuda.Event(enable_timing=True, external=use_graph) for _ in range(S if use_graph else K)]
    d_end = [torch.cuda.Event(enable_timing=True, external=use_graph) for _ in range(S if use_graph else K)]

    def timed_steps(count, off=0, events=True):
        for i in range(count):
            if events:
                d_beg[off + i].record()
            step.draft()
            if events:
                d_end[off + i].record()
            step.collapse()
            step.tree()
            step.attention()
            step.verify()

    launches0 = step.h.launch_count
    step.run()
    launches_per_step = step.h.launch_count - launches0
    # Two graphs of S steps: one plain, one with an event pair around every draft-head launch.
    # An event node between two kernels keeps the second from starting its prologue under the
    # first one's tail, so only the last replay of the timed region carries the events.
    graph = graph_plain = None
    side = torch.cuda.Stream(device=dev)
    if use_graph:
        graph = torch.cuda.CUDAGraph()
        graph_plain = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                timed_steps(S)
            with torch.cuda.graph(graph_plain, stream=side):
                timed_steps(S, events=False)
        for _ in range(2):
            graph.replay()
            graph_plain.replay()
    # Settling run: untimed replays for about half a second with the clock sampler's window open,
    # so that the record around a timed region of a few milliseconds is never empty and shows the
    # clocks the GPU runs this very load at.  The timed region follows without a pause.
    barrier()
    if sampler:
        sampler.begin()
    if use_graph:
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 0.5:
            for _ in range(10):
                graph_plain.replay()
            torch.cuda.synchronize()
    barrier()
    t_beg.record()
    if use_graph:
        for _ in range(K // S - 1):
            graph_plain.replay()
        graph.replay()
    else:
        timed_steps(K)
    t_end.record()
    barrier()
    launches = launches_per_step * K
    step.check_status()
    ms = t_beg.elapsed_time(t_end)
    draft_ms = float(np.mean([a.elapsed_time(b) for a, b in zip(d_beg, d_end)]))

    # ---- end to end: per-step inputs come from pinned host memory, results go back ------
    # the per-step inputs (x, base token, cache length, tree queries, tree-node hidden states) sit in
    # one device buffer and the results in another: one copy each way per step
    h_in = step.pack_step_inputs()
    h_out = torch.empty_like(step.result, device="cpu").pin_memory()
    h2d = h_in.numel() * h_in.element_size()
    d2h = h_out.numel() * h_out.element_size()
    # two host mirrors each way: while the GPU works on one step the host already hands over the
    # next (steps are independent batches), and reads a step's result once its event has passed
    h_ins = [h_in, h_in.clone().pin_memory()]
    h_outs = [h_out, torch.empty_like(h_out).pin_memory()]

    graphs = [None, None]
    if use_graph:
        torch.cuda.synchronize()
        # one graph per step and mirror: the copy in from pinned memory, the calls, the copy out
        for b in range(2):
            graphs[b] = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graphs[b], stream=side):
                    step.run_from_host(h_ins[b], h_outs[b])
        torch.cuda.synchronize()
    done = [torch.cuda.Event(), torch.cuda.Event()]
    seen = [0]

    def e2e_steps(count, in_flight):
        """`count` steps; the host waits for step i's result before it enqueues step i + in_flight."""
        for i in range(count):
            b = i % in_flight
            if i >= in_flight:
                done[b].synchronize()
                seen[0] += int(h_outs[b].view(-1)[0].item() >= 0)     # the host reads the result
            if graphs[b] is not None:
                graphs[b].replay()
            else:
                step.run_from_host(h_ins[b], h_outs[b])
            done[b].record()
        torch.cuda.synchronize()

    e2e_ms = {}
    for in_flight in (1, 2):
        e2e_steps(3, in_flight)
        barrier()
        e_beg, e_end = ev(), ev()
        e_beg.record()
        e2e_steps(K, in_flight)
        e_end.record()
        torch.cuda.synchronize()
        e2e_ms[in_flight] = e_beg.elapsed_time(e_end)
    barrier()
    if sampler:
        sampler.end()
    clocks = sampler.stop() if sampler else None
    ms, e2e_ms, e2e1_ms, draft_ms = replicas.max_over_ranks([ms, e2e_ms[2], e2e_ms[1], draft_ms])
    launches = replicas.sum_over_ranks(launches)

    if rank == 0:
        peak, peak_kind = load_peaks()
        mean_kv = float(np.mean(inp["kv_len"]))
        n_live = float(np.mean(n_nodes))
        draft_b, lm_b, kv_b = algorithmic_bytes(cfg, mean_kv, n_live)
        achieved = draft_b / (draft_ms * 1e-3) / 1e9
        step_bytes = draft_b + lm_b + kv_b
        value = world * K / (ms * 1e-3)
        paths = cfg.k ** cfg.T
        config = {"workload": workload_name(cfg), "layout": args.layout, "l2": "inputs larger than L2 (weights %.0f MB)" % (
            (draft_b + lm_b) / 1e6), "parallelism": "replicas x%d" % world,
            "launch": ("CUDA graph of %d steps, replayed %d times; the last replay carries an event pair around "
                       "each draft-head launch" % (S, K // S)) if use_graph
            else "direct launches",
            "tree_nodes": n_live, "step_bytes": step_bytes,
            "step_hbm_frac_of_%s_peak" % peak_kind: step_bytes / (ms / K * 1e-3) / 1e9 / peak,
            "inputs": {"force_repeats": bool(args.force_repeats), "blank_bias": [float(v) for v in cfg.blank_bias],
                       "slot_paths": paths, "candidates_kept": [int(v) for v in n_cand[:8]]}}
        if cand_len is not None:
            config["inputs"]["kept_candidates_shorter_than_T"] = int((cand_len[cand_len > 0] < cfg.T).sum())
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
            "config": config,
            "clocks": clocks,
            "e2e": {"value": world * K / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps_in_flight": 2,
                    "value_one_step_in_flight": world * K / (e2e1_ms * 1e-3)},
            "gpu_launches": launches,
            "roofline": {"kernel": "gemv_stream_kernel (draft head)", "bound": "hbm", "achieved": achieved,
                         "peak": peak, "peak_source": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": ncu_traffic(cfg.name, "gemv_stream_kernel")},
        }
        if args.stage_times:
            st = stage_times_us(step, torch)
            tens = 1400.0
            try:
                with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                    tens = float(json.load(f)["bf16_tflops_sustained"])
            except (OSError, ValueError, KeyError):
                pass
            rf = roofline_times_us(cfg, mean_kv, n_live, peak, tens)
            line["stages_us"] = {k: round(v, 2) for k, v in st.items()}
            line["stages_roofline_us"] = {k: round(v, 2) for k, v in rf.items()}
            line["stages_frac"] = {k: round(rf[k] / st[k], 3) for k in rf}
        if args.draft_module and world == 1:
            dm = draft_module_time(args, cfg, step, seed, torch, to_device, synth)
            dm["share_of_layer_plus_step"] = dm["us"] / (dm["us"] + ms / K * 1e3)
            dm["frac_of_%s_hbm_peak" % peak_kind] = dm["GBps"] / peak
            line["draft_module"] = dm
        if args.chain > 0 and world == 1:
            line["chain"] = chain_tokens_per_s(args, cfg, step, inp, seed, torch, to_device, synth)
        if world == 1 and not args.no_cpu_baseline:
            n_or = 10
            sec = time_oracle(cfg, inp, n_or, 1, args.layout)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                    "sample": "%d full steps of the fp64 oracle on the same inputs" % n_or}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(args) -> int:
    """`--gpus N` without a launcher: start N ranks of this script, one per GPU, the way
    `python -m torch.distributed.run` would be asked to (rendezvous on 127.0.0.1)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2", choices=["c1", "c2", "c3", "c4", "c5", "c6"])
    ap.add_argument("--layout", default="packed", choices=["packed", "raw"],
                    help="packed: collapse, then tree (headline); raw: the paper's raw-path tree with masked removed symbols")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--clock-period-ms", type=int, default=10, help="period of the nvidia-smi clock sampler")
    ap.add_argument("--no-graph", action="store_true", help="enqueue every call directly instead of replaying a CUDA graph")
    ap.add_argument("--force-repeats", action="store_true",
                    help="draft weights that make neighbouring slots favour the same tokens, so that repeats and merges occur")
    ap.add_argument("--blank-bias", type=float, default=None, help="blank-logit bias for every sequence (default: the workload's)")
    ap.add_argument("--stage-times", action="store_true", help="add per-call device times and their roofline times to the line")
    ap.add_argument("--draft-module", action="store_true",
                    help="also time the paper's attention draft module (one decoder layer before the draft head)")
    ap.add_argument("--chain", type=int, default=0, help="also time N chained steps (history update after each); adds tokens/s")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
