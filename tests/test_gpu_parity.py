"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, stage by stage.

Tolerances (written out here as the acceptance bar): integer outputs bit-exact when the oracle
is fed the CUDA path's previous-stage output; logits and attention outputs within 2e-2 max-abs
for bf16 inputs with fp32 accumulation (2e-4 for fp32 inputs); fp32 log-probabilities within
1e-4 relative."""
import numpy as np
import pytest

from paper_2412_00061_b200 import synth

pytestmark = pytest.mark.gpu

C = synth.CONFIGS

# scaled-down instances of the five workloads: several tiles, ragged tails, odd V+1
SMALL = {
    "c2s": C["c2"].replace(name="c2s", H=520, V=2999, Hq=8, Hkv=8, kv_lo=200, kv_hi=200),
    "c3s": C["c3"].replace(name="c3s", B=3, H=512, V=1777, Hq=4, Hkv=4, kv_lo=70, kv_hi=300, beam=16),
    "c4s": C["c4"].replace(name="c4s", B=2, H=640, V=2500, Hq=4, Hkv=4, kv_lo=333, kv_hi=333),
    "c5s": C["c5"].replace(name="c5s", B=5, H=1024, V=1200, Hq=8, Hkv=2, kv_lo=100, kv_hi=500),
    "c1d64": C["c1"].replace(name="c1d64", B=2, H=264, V=777, kv_lo=1, kv_hi=90, dtype="bf16"),
}


def _run(cfg, **kw):
    from tests.parity_util import run_parity
    return run_parity(cfg, **kw)


def test_c1_tiny_fp32_full():
    r = _run(C["c1"], seed=0, require_certified=True)
    assert r["n_nodes"][0] >= 2


@pytest.mark.parametrize("name", sorted(SMALL))
@pytest.mark.parametrize("seed", [0, 1])
def test_small_shapes(name, seed):
    _run(SMALL[name], seed=seed)


def test_forced_repeats_make_real_duplicates():
    r = _run(SMALL["c2s"], seed=3, force_repeats=True)
    assert r["n_nodes"][0] >= 2


def test_many_draft_rows_with_row_and_sel_maps():
    # draft head on 11 rows (three passes of the row-blocked kernel), 3 sequences pick rows 9, 0, 4
    cfg = SMALL["c3s"]
    row_seq = np.array([0, 1, 2, 0, 1, 2, 0, 1, 2, 0, 1], dtype=np.int32)
    sel_row = np.array([9, 0, 4], dtype=np.int32)
    _run(cfg, seed=2, M=11, row_seq=row_seq, sel_row=sel_row)


def test_draft_head_on_every_tree_row_uses_several_row_tiles():
    # the "draft head on all tree rows" variant: 5 sequences x 64 tree rows = 320 draft rows (three
    # 128-row tiles of the tensor-core path), each sequence drafting from one of its own rows
    cfg = SMALL["c5s"]
    M = cfg.B * cfg.max_nodes
    row_seq = (np.arange(M) // cfg.max_nodes).astype(np.int32)
    sel_row = np.array([b * cfg.max_nodes + (7 * b + 3) % cfg.max_nodes for b in range(cfg.B)], dtype=np.int32)
    _run(cfg, seed=1, M=M, row_seq=row_seq, sel_row=sel_row, draft_rows=[0, 127, 128, 200, 319])


def test_c5_draft_head_on_all_2048_tree_rows_full_size():
    """The 70B-shaped workload with the draft head run on every tree row (32 sequences x 64 rows =
    2048 rows, sixteen 128-row tiles of the tensor-core path against 3.1 GB of weights).  The
    logits of sampled rows are compared with the oracle (definition mode) and their top-k and
    log-sum-exp with the oracle fed those logits (bit-exact ids)."""
    import torch
    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200.step import DraftVerifyStep, to_device
    from tests.parity_util import check_topk, tolerances
    cfg = C["c5"]
    M = cfg.B * cfg.max_nodes
    x, Wd, bb = synth.gen_draft(cfg, 3, M=M)
    row_seq = (np.arange(M) // cfg.max_nodes).astype(np.int32)
    step = DraftVerifyStep(cfg, device="cuda:0", max_draft_rows=M, debug_logits=True)
    dev = step.device
    step.set_inputs(x=to_device(x, cfg.dtype, dev), Wd=to_device(Wd, cfg.dtype, dev),
                    blank_bias=torch.from_numpy(bb).to(dev), row_seq=torch.from_numpy(row_seq).to(dev))
    step.draft()
    step.check_status()
    rows = [0, 127, 128, 1000, 2047]
    idx = torch.tensor(rows, device=dev)
    z_gpu = step.out["draft_logits_dbg"][idx].cpu().numpy()
    logit_tol, rel = tolerances(cfg.dtype)
    z_def = orc.draft_logits(x[rows], Wd, bb, row_seq[rows])
    assert np.max(np.abs(z_gpu - z_def)) <= logit_tol
    check_topk(z_gpu, step.out["topk_id"][idx].cpu().numpy(), step.out["topk_lp"][idx].cpu().numpy(),
               step.out["lse"][idx].cpu().numpy(), cfg.k, rel)


def test_enumeration_limits_and_max_score_mode():
    # 4096 paths (T=6, k=4) enumerated exhaustively; best-alignment scoring variant
    _run(C["c1"].replace(name="enum4096", T=6, k=4, topN=64, max_nodes=128), seed=0)
    _run(C["c1"].replace(name="maxmode", score_mode=1), seed=0)
    # k = V + 1: the lists hold the whole distribution (tiny vocabulary)
    _run(C["c1"].replace(name="tinyV", V=4, k=5, T=3, H=64), seed=0)


def test_only_blank_paths_leave_just_the_root():
    # a huge blank bias with k = 1 makes every slot pick the blank: no candidate, tree = root
    cfg = C["c1"].replace(name="allblank", k=1, blank_bias=(50.0,))
    r = _run(cfg, seed=0)
    assert r["n_nodes"][0] == 1 and r["acc_len"][0] == 0


def test_c2_full_size_sampled():
    """The headline workload at full size.  The definition-mode oracle checks one draft row in
    full, sampled LM-head rows and sampled attention (sequence, head) pairs; all integer stages are
    compared in full.  Then the step is rerun the way the benchmark launches it (no debug dumps, a CUDA
    graph of three steps replayed twice) and must give the same results bit for bit."""
    from tests.parity_util import check_benchmark_launch_configuration
    r = _run(C["c2"], seed=0, require_certified=True, attention_rows=4, lm_rows=8)
    assert 2 <= r["n_nodes"][0] <= 64
    check_benchmark_launch_configuration(r)


def test_c2_raw_layout_and_c3_in_the_benchmark_launch_configuration():
    from tests.parity_util import check_benchmark_launch_configuration, run_parity_raw
    check_benchmark_launch_configuration(run_parity_raw(C["c2"], seed=0, attention_rows=2, lm_rows=8))
    check_benchmark_launch_configuration(_run(C["c3"], seed=1, attention_rows=2, lm_rows=6, draft_rows=[0]))
    check_benchmark_launch_configuration(_run(SMALL["c5s"], seed=2))


def test_attention_is_reproducible_while_the_lm_head_streams_beside_it():
    """Attention and LM head alternating inside one CUDA graph: under programmatic dependent launch
    the LM head of one pair streams its weights while the last attention CTAs of the same pair still
    run, which slows their K/V loads and shifts the relative timing of the warps inside them.  The
    attention output must not depend on that: every replay must reproduce, bit for bit, the output of
    the stand-alone call that the oracle has checked.  (An earlier version whose softmax warps
    shared one P-ready barrier between consecutive tiles failed exactly here.)"""
    import torch
    r = _run(C["c3"], seed=1, attention_rows=3, lm_rows=6, draft_rows=[0])
    step = r["step"]
    want = step.out["O"].clone()
    side = torch.cuda.Stream(device=step.device)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step.attention(); step.verify()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            for _ in range(4):
                step.attention()
                step.verify()
    for _ in range(6):
        step.out["O"].zero_()
        g.replay()
        step.check_status()
        assert torch.equal(step.out["O"], want)


@pytest.mark.parametrize("name", ["c3", "c4", "c5", "c6"])
def test_batched_workloads_full_size_sampled(name):
    """The batched workloads at full size (prefix beam, ragged KV lengths, 128-node trees, GQA):
    all integer stages are compared in full; the definition-mode oracle checks one draft row,
    sampled LM-head rows and sampled attention (sequence, head) pairs."""
    cfg = C[name]
    r = _run(cfg, seed=0, attention_rows=3, lm_rows=6, draft_rows=[cfg.B - 1])
    assert all(2 <= n <= cfg.max_nodes for n in r["n_nodes"])


@pytest.mark.parametrize("name", ["c2s", "c3s", "c5s", "c1d64"])
def test_history_update_moves_the_accepted_rows(name):
    """ctcsd_commit_accepted against the oracle: the K/V caches must match byte for byte, the new
    lengths and the next drafting rows exactly (steps that run on the updated cache: the chain tests)."""
    import torch
    from oracle import ctcsd_oracle as orc
    cfg = SMALL[name]
    r = _run(cfg, seed=4)
    step = r["step"]
    K0, V0 = step.inp["K"].float().cpu().numpy(), step.inp["V"].float().cpu().numpy()
    kv_len = step.inp["kv_len"].cpu().numpy()
    acc_len, acc_nodes = step.host("acc_len"), step.host("acc_nodes")
    K1, V1, new_len, sel = orc.commit_accepted(K0, V0, kv_len, acc_len, acc_nodes, cfg.max_nodes)
    step.commit()
    step.check_status()
    assert np.array_equal(step.inp["K"].float().cpu().numpy(), K1)
    assert np.array_equal(step.inp["V"].float().cpu().numpy(), V1)
    np.testing.assert_array_equal(step.host("new_kv_len"), new_len)
    np.testing.assert_array_equal(step.host("next_sel_row"), sel)
    assert acc_len.max() >= 1, "pick a seed where something is accepted"
    # a path that would leave the cache is refused on the device and changes nothing
    bad_len = torch.full_like(step.inp["kv_len"], step.inp["K"].shape[2])
    step.h.commit_accepted(step.inp["K"], step.inp["V"], bad_len, step.out["acc_len"], step.out["acc_nodes"],
                           step.out["new_kv_len"], step.out["next_sel_row"])
    assert step.h.poll_status() == -1
    assert np.array_equal(step.inp["K"].float().cpu().numpy(), K1)


def test_history_update_may_write_the_new_length_over_the_old_one():
    """out_kv_len is the same array as kv_len, on a shape with more (sequence, kv head) CTAs than the
    GPU holds at once (48 x 32 = 1536): a CTA that starts late must still see the old length."""
    import torch
    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200 import binding
    from paper_2412_00061_b200.step import to_device
    cfg = C["c3"].replace(name="alias", B=48, H=64, V=100, Hq=32, Hkv=32, D=64, kv_lo=3, kv_hi=60, max_nodes=32, T=6)
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(21)
    _, K, V = synth.gen_attention(cfg, 21)
    _, kv_len = synth.gen_base(cfg, 21)
    acc_len = rng.integers(0, cfg.T + 1, size=cfg.B).astype(np.int32)
    acc_nodes = np.full((cfg.B, cfg.T), -1, dtype=np.int32)
    for b in range(cfg.B):                       # strictly increasing node ids, node_l >= l + 1
        acc_nodes[b, :acc_len[b]] = np.sort(rng.choice(np.arange(1, cfg.max_nodes), size=acc_len[b], replace=False))
    K1, V1, new_len, sel = orc.commit_accepted(K, V, kv_len, acc_len, acc_nodes, cfg.max_nodes)
    h = binding.Handle(cfg.B, cfg.H, cfg.V, cfg.T, cfg.k, cfg.beam, cfg.topN, cfg.max_nodes, cfg.Hq, cfg.Hkv, cfg.D,
                       binding.DTYPE_BF16)
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    Kd, Vd, len_d = to_device(K, "bf16", dev), to_device(V, "bf16", dev), i32(kv_len)
    sel_d = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    h.commit_accepted(Kd, Vd, len_d, i32(acc_len), i32(acc_nodes), len_d, sel_d)
    assert h.poll_status() == 0
    assert np.array_equal(Kd.float().cpu().numpy(), K1) and np.array_equal(Vd.float().cpu().numpy(), V1)
    np.testing.assert_array_equal(len_d.cpu().numpy(), new_len)
    np.testing.assert_array_equal(sel_d.cpu().numpy(), sel)
    # and once more on the result (the per-sequence tickets were left at zero)
    K2, V2, new_len2, _ = orc.commit_accepted(K1, V1, new_len, acc_len, acc_nodes, cfg.max_nodes)
    h.commit_accepted(Kd, Vd, len_d, i32(acc_len), i32(acc_nodes), len_d, sel_d)
    assert h.poll_status() == 0
    assert np.array_equal(Kd.float().cpu().numpy(), K2)
    np.testing.assert_array_equal(len_d.cpu().numpy(), new_len2)
    h.close()


@pytest.mark.parametrize("name", ["c2s", "c3s", "c5s", "c1d64"])
def test_chained_steps_without_host_work(name):
    """Five steps in a row, each followed by the history update, the next one taking its root token,
    cache length and drafting row from the device: every step's integers against the oracle fed the
    GPU's previous stage, the final K/V cache byte for byte, and the oracle's own chain from the raw
    inputs wherever none of its decisions was a near-tie."""
    from tests.parity_util import run_chain_parity
    r = run_chain_parity(SMALL[name], seed=4, n_steps=5)
    assert r["tokens"] > 5 * SMALL[name].B, "pick a seed where draft tokens are accepted"


def test_chained_steps_fp32_and_inside_a_cuda_graph():
    from tests.parity_util import run_chain_parity
    cfg = C["c1"].replace(name="c1chain", B=2, kv_lo=5, kv_hi=90)
    run_chain_parity(cfg, seed=1, n_steps=4)
    r = run_chain_parity(SMALL["c3s"], seed=6, n_steps=4, graph=True)
    assert r["tokens"] > 4 * SMALL["c3s"].B


@pytest.mark.parametrize("name", ["c2s", "c5s", "c1d64", "c1fp32"])
def test_sampling_acceptance(name):
    """ctcsd_verify_accept_sampled after a checked step: the sampled token of every node against the
    oracle fed the kernel's own logits (same float32 fused multiply-add, so bit-exact wherever the two
    best perturbed logits are not within rounding of each other), against the oracle from the raw
    inputs in float64 wherever that margin is comfortable, and the acceptance walk over the sampled
    tokens bit for bit.  Three temperatures; a tiny one must reproduce the greedy result."""
    import torch
    from oracle import ctcsd_oracle as orc
    cfg = SMALL[name] if name in SMALL else C["c1"].replace(name="c1fp32", B=2, kv_lo=3, kv_hi=60)
    r = _run(cfg, seed=5)
    step = r["step"]
    dev = step.device
    greedy = {k: step.host(k).copy() for k in ("argmax", "acc_len", "acc_nodes", "acc_tok", "next_tok")}
    node_tok, parent, depth, n_nodes = (step.host(k).astype(np.int64) for k in ("node_tok", "parent", "depth", "n_nodes"))
    noise = synth.gen_gumbel_noise(cfg, 5)
    noise_d = torch.from_numpy(noise).to(dev)
    hn = step.inp["hn"].float().cpu().numpy()
    Wl = step.inp["Wl"].float().cpu().numpy()
    y_def, _ = orc.lm_head_argmax(hn, Wl)
    y_def = y_def.reshape(cfg.B, cfg.max_nodes, cfg.V)
    accepted = []
    for temperature in (1.0, 0.05, 1e-6):
        inv_t = float(np.float32(1.0) / np.float32(temperature))
        step.verify_sampled(noise_d, temperature)
        step.check_status()
        y_gpu = step.host("lm_logits_dbg").reshape(cfg.B, cfg.max_nodes, cfg.V)
        x_gpu = step.host("argmax").astype(np.int64)
        want = orc.sample_accept(node_tok, parent, n_nodes, depth, y_gpu, noise, inv_t, cfg.T, fp32=True)
        for b in range(cfg.B):
            for i in range(int(n_nodes[b])):
                z = (y_gpu[b, i].astype(np.float64) * np.float64(np.float32(inv_t)) + noise[b, depth[b, i]]).astype(np.float32)
                top2 = np.sort(z)[-2:]
                if top2[1] - top2[0] > 4 * np.spacing(np.float32(abs(top2[1]))):     # not a rounding-level tie
                    assert x_gpu[b, i] == want[0][b, i], (temperature, b, i)
                zd = y_def[b, i] * inv_t + noise[b, depth[b, i]]
                t2 = np.sort(zd)[-2:]
                if t2[1] - t2[0] > 2 * 2e-2 * inv_t + 1e-3:                          # beyond the logit tolerance
                    assert x_gpu[b, i] == int(np.argmax(zd)), ("definition mode", temperature, b, i)
        acc = orc.greedy_accept(node_tok, parent, n_nodes, x_gpu, cfg.T)                 # the walk over the kernel's draws
        for nm, w in zip(["acc_len", "acc_nodes", "acc_tok", "next_tok"], acc):
            np.testing.assert_array_equal(step.host(nm), w, err_msg=nm)
        accepted.append(int(acc[0].sum()))
    for k, v in greedy.items():                                                      # temperature 1e-6: the greedy result
        live = np.arange(cfg.max_nodes)[None, :] < n_nodes[:, None]
        if k == "argmax":
            np.testing.assert_array_equal(step.host(k)[live], v[live])
        else:
            np.testing.assert_array_equal(step.host(k), v, err_msg=k)
    assert accepted[2] == int(greedy["acc_len"].sum())


DM = {
    # (workload, MLP width I, new rows R, positions already cached)
    "dm_mha": (C["c2"].replace(name="dm_mha", H=512, V=999, Hq=4, Hkv=4, D=128), 1368, 6, (100, 300)),
    "dm_gqa": (C["c5"].replace(name="dm_gqa", B=3, H=768, V=999, Hq=12, Hkv=4, D=64), 2048, 7, (0, 200)),
    "dm_fp32": (C["c1"].replace(name="dm_fp32", B=2, H=256, V=999, Hq=4, Hkv=2, D=64), 688, 5, (3, 90)),
    "dm_long_inner": (C["c2"].replace(name="dm_long_inner", B=3, H=256, V=999, Hq=2, Hkv=2, D=128), 11008, 3, (10, 50)),
    # the 7B shape: hidden 4096, 32 heads x 128, MLP width 11008, six new rows on top of ~1000 cached positions
    "dm_7b": (C["c2"].replace(name="dm_7b", V=999), 11008, 6, (900, 1024)),
}


@pytest.mark.parametrize("name", sorted(DM))
def test_attention_draft_module(name):
    """ctcsd_draft_module against the oracle's layer.  The CUDA path keeps the four activation vectors
    that feed a projection (and the cached keys/values) in the run dtype; the oracle, float64 otherwise,
    can round the same vectors (its `store` argument).  Tolerance, derived for bf16: every rounded vector
    carries a relative error of 2^-9 / sqrt(3) r.m.s. into a projection of up to 11008 terms with
    weights of 0.02 r.m.s.; chained through the layer that is 6.5e-3 r.m.s. on an output of 2.4 r.m.s.
    at the 7B shape (the float64 oracle with and without `store` differ by exactly that: 6.5e-3 r.m.s.,
    2.4e-2 maximum over 4096 outputs), and two implementations that round at the same places still
    differ by as much, because a 1e-3 difference in the attention output (P is bf16 inside the kernel)
    moves many values across a rounding boundary.  Hence: r.m.s. error <= 1.2e-2 and maximum <= 6e-2
    against both oracles (float32: 6e-4).  The appended key/value rows pass through one projection only
    and keep the 2e-2 bound; every other cache row must be untouched, the new lengths exact; then the
    draft head runs on the layer's output and its top-k lists are checked against the oracle fed its logits."""
    import torch
    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200 import binding
    from paper_2412_00061_b200.step import to_device
    from tests.parity_util import check_topk, tolerances
    cfg, I, R, (lo, hi) = DM[name]
    seed = 8
    dev = torch.device("cuda:0")
    w, F_new, n_new, kv_len, Kd, Vd = synth.gen_draft_layer(cfg, seed, I, R, lo, hi)
    store = synth.round_bf16 if cfg.dtype == "bf16" else None
    want_F, want_K, want_V, want_len = orc.draft_module(F_new, n_new, kv_len, Kd, Vd, w, cfg.Hq, cfg.Hkv, cfg.D, store=store)
    exact_F = orc.draft_module(F_new, n_new, kv_len, Kd, Vd, w, cfg.Hq, cfg.Hkv, cfg.D)[0]
    h = binding.Handle(cfg.B, cfg.H, cfg.V, cfg.T, cfg.k, cfg.beam, cfg.topN, cfg.max_nodes, cfg.Hq, cfg.Hkv, cfg.D,
                       binding.DTYPE_BF16 if cfg.dtype == "bf16" else binding.DTYPE_F32)
    td = lambda a: to_device(a, cfg.dtype, dev)
    f32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float32)).to(dev)
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    dl = h.make_draft_layer(f32(w["g1"]), td(w["Wqkv"]), td(w["Wo"]), f32(w["g2"]), td(w["Wgu"]), td(w["Wdn"]), R=R)
    Kd_d, Vd_d = td(Kd), td(Vd)
    act = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    out_F = torch.zeros(cfg.B, cfg.H, dtype=act, device=dev)
    out_dbg = torch.zeros(cfg.B, cfg.H, dtype=torch.float32, device=dev)
    out_len = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    for rep in range(2):                                   # twice: the workspace carries nothing over
        Kd_d.copy_(td(Kd)); Vd_d.copy_(td(Vd))
        h.draft_module(dl, td(F_new), i32(n_new), i32(kv_len), Kd_d, Vd_d, out_F, out_len, out_dbg)
        assert h.poll_status() == 0
        logit_tol, rel = tolerances(cfg.dtype)
        for ref_F in (want_F, exact_F):
            err = out_dbg.cpu().numpy() - ref_F
            assert np.max(np.abs(err)) <= 3 * logit_tol
            assert np.sqrt(np.mean(err ** 2)) <= 0.6 * logit_tol
        got_F = out_F.float().cpu().numpy()
        ulp = 2.0 ** -8 if cfg.dtype == "bf16" else 0.0
        assert np.all(np.abs(got_F - want_F) <= 3 * logit_tol + ulp * np.abs(want_F))
        np.testing.assert_array_equal(out_len.cpu().numpy(), want_len)
        gK, gV = Kd_d.float().cpu().numpy(), Vd_d.float().cpu().numpy()
        for b in range(cfg.B):
            L, r = int(kv_len[b]), int(n_new[b])
            assert np.array_equal(gK[b, :, :L], Kd[b, :, :L]) and np.array_equal(gK[b, :, L + r:], Kd[b, :, L + r:])
            assert np.array_equal(gV[b, :, :L], Vd[b, :, :L]) and np.array_equal(gV[b, :, L + r:], Vd[b, :, L + r:])
            assert np.all(np.abs(gK[b, :, L:L + r] - want_K[b, :, L:L + r]) <= logit_tol + ulp * np.abs(want_K[b, :, L:L + r]))
            assert np.all(np.abs(gV[b, :, L:L + r] - want_V[b, :, L:L + r]) <= logit_tol + ulp * np.abs(want_V[b, :, L:L + r]))
    # the per-place projection on the layer's output
    x, Wd, bb = synth.gen_draft(cfg, seed)
    topk_id = torch.zeros(cfg.B, cfg.T, cfg.k, dtype=torch.int32, device=dev)
    topk_lp = torch.zeros(cfg.B, cfg.T, cfg.k, dtype=torch.float32, device=dev)
    lse = torch.zeros(cfg.B, cfg.T, dtype=torch.float32, device=dev)
    zdbg = torch.zeros(cfg.B, cfg.T, cfg.V + 1, dtype=torch.float32, device=dev)
    h.draft_logits(out_F, td(Wd), None, torch.from_numpy(bb).to(dev), topk_id, topk_lp, lse, zdbg)
    assert h.poll_status() == 0
    z_def = orc.draft_logits(got_F, Wd, bb)
    assert np.max(np.abs(zdbg.cpu().numpy() - z_def)) <= logit_tol
    check_topk(zdbg.cpu().numpy(), topk_id.cpu().numpy(), topk_lp.cpu().numpy(), lse.cpu().numpy(), cfg.k, rel)
    # a sequence whose new rows would leave the cache is reported and its cache left alone
    bad_len = i32(np.full(cfg.B, Kd.shape[2], dtype=np.int32))
    Kd_d.copy_(td(Kd))
    h.draft_module(dl, td(F_new), i32(n_new), bad_len, Kd_d, Vd_d, out_F, out_len)
    assert h.poll_status() == -1
    assert np.array_equal(Kd_d.float().cpu().numpy(), Kd)
    h.close()


BIG = {
    # trees above 128 nodes: three and four mask words, two LM-head row tiles per sequence
    "big_enum": C["c2"].replace(name="big_enum", H=520, V=2999, Hq=8, Hkv=8, kv_lo=200, kv_hi=200,
                                T=6, k=4, topN=64, max_nodes=256),
    "big_beam_gqa": C["c5"].replace(name="big_beam_gqa", B=3, H=512, V=1500, Hq=8, Hkv=2, kv_lo=90, kv_hi=400,
                                    T=8, k=5, beam=128, topN=64, max_nodes=200),
    "big_fp32": C["c1"].replace(name="big_fp32", B=2, H=264, V=777, kv_lo=1, kv_hi=90, T=6, k=4, topN=64,
                                max_nodes=200),
}


def test_attention_fallback_when_heads_per_kv_head_do_not_divide_the_row_tile():
    """Three query heads per kv head: the tensor-core kernel's 128-row tile cannot hold whole
    nodes, so the warp-level kernel runs; once with a small tree, once above 128 nodes."""
    small = C["c5"].replace(name="gqa3", B=2, H=512, V=1500, Hq=6, Hkv=2, kv_lo=60, kv_hi=300, beam=16)
    _run(small, seed=1)
    big = BIG["big_beam_gqa"].replace(name="gqa3_big", Hq=6, Hkv=2, D=64)
    r = _run(big, seed=2)
    assert max(r["n_nodes"]) > 128


@pytest.mark.parametrize("name", sorted(BIG))
def test_trees_above_128_nodes(name):
    cfg = BIG[name]
    r = _run(cfg, seed=2)
    assert max(r["n_nodes"]) > 128, "the tree must reach past the first two mask words"


@pytest.mark.parametrize("name", ["big_enum", "big_fp32"])
def test_raw_layout_on_a_tree_above_128_nodes(name):
    from tests.parity_util import run_parity_raw
    r = run_parity_raw(BIG[name], seed=2)
    assert max(r["n_nodes"]) > 128


def test_empty_prefix_and_every_limit_at_once():
    """kv_len = 0 (the tree attends to nothing but itself) on both attention kernels' dtypes, and a
    configuration that sits on every documented maximum at once: T = 8 slots, k = 8 symbols per
    slot (T*k = 64), beam 128, 64 candidates, 256 tree nodes."""
    for base in ("c2s", "c1d64"):
        _run(SMALL[base].replace(name=base + "_kv0", kv_lo=0, kv_hi=0), seed=2)
    _run(C["c1"].replace(name="c1_kv0", kv_lo=0, kv_hi=0), seed=2)
    top = C["c4"].replace(name="limits", B=2, H=512, V=1500, Hq=8, Hkv=4, kv_lo=50, kv_hi=700,
                          T=8, k=8, beam=128, topN=64, max_nodes=256)
    r = _run(top, seed=1)
    assert max(r["n_nodes"]) > 128


@pytest.mark.parametrize("grp", [1, 4])
def test_attention_when_later_keys_score_far_higher(grp):
    """Keys whose scores grow from tile to tile by far more than the slack the kernel allows between
    the row maximum and the exponent's reference: every tile then moves the reference and rescales
    the output accumulated so far (with uniform random keys that path would never run)."""
    import math
    import torch
    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200.step import DraftVerifyStep, to_device
    cfg = C["c2"].replace(name="grow", H=256, V=999, Hq=8, Hkv=8 // grp, kv_lo=3000, kv_hi=3000)
    x, Wd, bb = synth.gen_draft(cfg, 7)
    base_tok, kv_len = synth.gen_base(cfg, 7)
    Q, K, V = synth.gen_attention(cfg, 7)
    ramp = 1.0 + 3.0 * (np.arange(cfg.Lcap) // 128).astype(np.float32)          # tile t: keys x (1 + 3t)
    K = synth.to_dtype(K * ramp[None, None, :, None], cfg.dtype)
    step = DraftVerifyStep(cfg, device="cuda:0")
    dev = step.device
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    step.set_inputs(x=to_device(x, cfg.dtype, dev), Wd=to_device(Wd, cfg.dtype, dev),
                    blank_bias=torch.from_numpy(bb).to(dev), base_tok=i32(base_tok), kv_len=i32(kv_len),
                    Q=to_device(Q, cfg.dtype, dev), K=to_device(K, cfg.dtype, dev), V=to_device(V, cfg.dtype, dev))
    step.draft(); step.collapse(); step.tree(); step.attention()
    step.check_status()
    n_nodes, mask = step.host("n_nodes"), step.host("mask").view(np.uint64)
    want = orc.tree_attention(Q, K, V, kv_len, n_nodes, mask, 1.0 / math.sqrt(cfg.D))
    assert np.max(np.abs(step.host("O") - want)) <= 2e-2


RAW = {
    # the raw trie of N paths of T symbols has up to 1 + N*T nodes
    "c2raw": C["c2"].replace(name="c2raw", H=520, V=2999, Hq=8, Hkv=8, kv_lo=200, kv_hi=200, max_nodes=96),
    "c3raw": C["c3"].replace(name="c3raw", B=3, H=512, V=1777, Hq=4, Hkv=4, kv_lo=70, kv_hi=300, beam=0,
                             T=4, k=4, topN=24, max_nodes=128),
    "c5raw_cut": C["c5"].replace(name="c5raw_cut", B=5, H=1024, V=1200, Hq=8, Hkv=2, kv_lo=100, kv_hi=500,
                                 beam=0, T=5, k=3, topN=32, max_nodes=64),      # node budget cuts the trie
    "c1raw": C["c1"].replace(name="c1raw", B=2, H=264, V=777, kv_lo=1, kv_hi=90),   # fp32 path
}


@pytest.mark.parametrize("name", sorted(RAW))
@pytest.mark.parametrize("seed", [3, 5])
def test_raw_tree_layout(name, seed):
    """The paper's own verification layout (Sec. 3.3): raw paths, removed symbols masked."""
    from tests.parity_util import run_parity_raw
    cfg = RAW[name]
    r = run_parity_raw(cfg, seed=seed, force_repeats=(seed == 5))
    live = sum(int(n) for n in r["n_nodes"])
    removed = live - int(r["kept"].sum())
    assert removed > 0, "the inputs must exercise the transform (blanks or repeats in the raw paths)"


@pytest.mark.parametrize("name", ["c2raw", "c5raw_cut"])
def test_chained_steps_raw_layout(name):
    from tests.parity_util import run_chain_parity
    r = run_chain_parity(RAW[name], seed=3, n_steps=4, layout="raw")
    assert r["tokens"] > 4 * RAW[name].B


def test_raw_tree_layout_c2_full_size_and_history_update():
    """Headline shape, raw layout, sampled attention / LM-head rows; then the history update
    moves the accepted (kept) nodes' rows exactly as the oracle does."""
    from oracle import ctcsd_oracle as orc
    from tests.parity_util import run_parity_raw
    cfg = C["c2"].replace(name="c2rawfull", max_nodes=96)
    r = run_parity_raw(cfg, seed=1, attention_rows=4, lm_rows=24)
    step = r["step"]
    K0, V0 = step.inp["K"].float().cpu().numpy(), step.inp["V"].float().cpu().numpy()
    kv_len = step.inp["kv_len"].cpu().numpy()
    acc_len, acc_nodes = step.host("acc_len"), step.host("acc_nodes")
    K1, V1, new_len, sel = orc.commit_accepted(K0, V0, kv_len, acc_len, acc_nodes, cfg.max_nodes)
    step.commit()
    step.check_status()
    assert np.array_equal(step.inp["K"].float().cpu().numpy(), K1)
    assert np.array_equal(step.inp["V"].float().cpu().numpy(), V1)
    np.testing.assert_array_equal(step.host("new_kv_len"), new_len)
    np.testing.assert_array_equal(step.host("next_sel_row"), sel)


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """Failure detection without a fault: a bounded device-side wait on a barrier that nothing
    signals gives up, the status word says CTCSD_ERR_TIMEOUT, polling clears it, and the same
    handle then runs a full step that matches the oracle."""
    r = _run(C["c1"], seed=1)
    step = r["step"]
    before = {k: step.host(k).copy() for k in ("cand_tok", "node_tok", "argmax", "acc_len")}
    step.h.selftest_timeout()
    assert step.h.poll_status() == -5
    assert step.h.poll_status() == 0
    step.run()
    step.check_status()
    for k, v in before.items():
        np.testing.assert_array_equal(step.host(k), v)


def _random_slot_lists(rng, M, T, k, V, pool):
    """Per-slot lists as S3 would hand them over (k distinct ids, log-probabilities descending), drawn
    from a small pool of tokens plus the blank so that blanks, repeats and merges are the rule."""
    ids = np.zeros((M, T, k), dtype=np.int32)
    lp = np.zeros((M, T, k), dtype=np.float32)
    symbols = np.array(list(range(pool)) + [V])
    for m in range(M):
        for t in range(T):
            pick = rng.choice(symbols, size=k, replace=False)
            z = np.sort(rng.normal(0.0, 2.0, size=k))[::-1]
            ids[m, t] = pick
            lp[m, t] = (z - np.log(np.sum(np.exp(z))) - rng.uniform(0.0, 0.5)).astype(np.float32)
    return ids, lp


@pytest.mark.parametrize("pattern", [(1, 64, 17, 64, 1), (1, 1, 1, 1, 1), (64, 64, 64, 64, 64), (3, 2, 64, 1, 40)])
def test_lm_head_serves_live_rows_only(pattern):
    """More than 128 tree rows: the LM head packs the rows of used nodes and computes nothing else.  After
    a checked step the node counts are cut to a pattern (a prefix of a tree is a tree), the rows of
    nodes that are now unused are filled with large values that would win any arg-max, and the call
    is repeated: arg-max of every live row and the acceptance against the oracle, -1 for unused rows."""
    import torch
    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200.step import to_device
    cfg = SMALL["c5s"]
    r = _run(cfg, seed=9)
    step = r["step"]
    dev = step.device
    n0 = step.host("n_nodes").astype(np.int64)
    n_new = np.minimum(n0, np.array(pattern, dtype=np.int64))
    node_tok, parent = step.host("node_tok").astype(np.int64), step.host("parent").astype(np.int64)
    hn = step.inp["hn"].float().cpu().numpy().copy()
    Wl = step.inp["Wl"].float().cpu().numpy()
    for b in range(cfg.B):
        hn[b * cfg.max_nodes + int(n_new[b]):(b + 1) * cfg.max_nodes] = 50.0      # must never be looked at
    step.set_inputs(hn=to_device(hn, cfg.dtype, dev))
    step.out["n_nodes"].copy_(torch.from_numpy(n_new.astype(np.int32)).to(dev))
    step.out["argmax"].fill_(-7)
    step.verify()
    step.check_status()
    am = step.host("argmax").astype(np.int64)
    live = [b * cfg.max_nodes + i for b in range(cfg.B) for i in range(int(n_new[b]))]
    dead = sorted(set(range(cfg.B * cfg.max_nodes)) - set(live))
    _, am_def = orc.lm_head_argmax(hn[live].astype(np.float64), Wl.astype(np.float64))
    np.testing.assert_array_equal(am.reshape(-1)[live], am_def)
    assert np.all(am.reshape(-1)[dead] == -1)
    acc = orc.greedy_accept(node_tok, parent, n_new, am, cfg.T)
    for name, want in zip(["acc_len", "acc_nodes", "acc_tok", "next_tok"], acc):
        np.testing.assert_array_equal(step.host(name), want, err_msg=name)


@pytest.mark.parametrize("mode", ["beam", "enumerate"])
def test_random_slot_lists_through_collapse_and_tree(mode):
    """S4-S8 on many small random shapes (slots, list length, beam, candidates kept, tree budget all
    drawn at random; a token pool of k + 1 or k + 2 symbols, so nearly every path has blanks or
    repeats and most candidates have several alignments), fed straight into the candidate call."""
    import torch
    from tests import parity_util
    from paper_2412_00061_b200.step import DraftVerifyStep
    rng = np.random.default_rng(20241200 + (mode == "beam"))
    done = 0
    for case in range(60):
        T = int(rng.integers(1, 9))
        k = int(rng.integers(1, 9))
        if mode == "enumerate":
            while k ** T > 4096:
                k -= 1
        beam = int(rng.choice([1, 2, 3, 5, 8, 16, 33, 64, 128])) if mode == "beam" else 0
        N = int(rng.integers(1, 65))
        B = int(rng.integers(1, 5))
        M = B + int(rng.integers(0, 3))
        n_max = int(rng.choice([8, 33, 64, 128, 200, 256]))
        V = 40
        cfg = C["c1"].replace(name="rnd", B=B, T=T, k=k, beam=beam, topN=N, max_nodes=n_max, V=V,
                              score_mode=int(rng.integers(0, 2)) if mode == "enumerate" else 0)
        ids, lp = _random_slot_lists(rng, M, T, k, V, pool=min(k + int(rng.integers(0, 2)), V))
        sel = rng.permutation(M)[:B].astype(np.int32)
        st = {}
        parity_util.orc.topk_collapse(ids.astype(np.int64), lp.astype(np.float64), blank=V, T=T, N=N, beam=beam,
                                      score_mode=cfg.score_mode, sel_row=sel, B=B, stats=st)
        if beam > 0 and min(st["margin"]) <= parity_util.TAU:
            continue                                    # the beam cut falls inside a tie: several answers are right
        step = DraftVerifyStep(cfg, device="cuda:0", max_draft_rows=M)
        dev = step.device
        step.out["topk_id"].copy_(torch.from_numpy(ids).to(dev))
        step.out["topk_lp"].copy_(torch.from_numpy(lp).to(dev))
        base_tok, kv_len = parity_util.synth.gen_base(cfg, case)
        step.set_inputs(sel_row=torch.from_numpy(sel).to(dev), base_tok=torch.from_numpy(base_tok.astype(np.int32)).to(dev),
                        kv_len=torch.from_numpy(kv_len.astype(np.int32)).to(dev))
        step.collapse()
        step.tree()
        step.check_status()
        got = (step.host("cand_tok"), step.host("cand_len"), step.host("cand_score"), step.host("n_cand"))
        parity_util.check_candidates(cfg, ids, lp, sel, got)
        want = parity_util.orc.build_tree(base_tok, kv_len, got[0].astype(np.int64), got[1].astype(np.int64),
                                          got[3].astype(np.int64), n_max)
        for name, w in zip(["node_tok", "parent", "depth", "pos", "mask", "retrieve", "n_nodes"], want):
            have = step.host(name)
            if name == "mask":
                have = have.view(np.uint64)
            np.testing.assert_array_equal(have, w, err_msg="case %d %s" % (case, name))
        done += 1
    assert done >= 45


@pytest.mark.parametrize("layout", ["packed", "raw"])
def test_a_draft_row_out_of_range_leaves_the_root_alone(layout):
    """sel_row pointing outside the draft rows: the call that makes the candidates reports the
    error and gives that sequence none, the tree is the root alone (what the oracle builds
    from zero candidates), and the handle runs a correct step afterwards."""
    import torch
    from paper_2412_00061_b200 import binding
    from tests import parity_util
    r = (_run(C["c1"], seed=2) if layout == "packed" else parity_util.run_parity_raw(C["c1"], seed=2))
    step, cfg = r["step"], C["c1"]
    good = {k: step.host(k).copy() for k in ("node_tok", "parent", "mask", "n_nodes", "acc_len")}
    step.set_inputs(sel_row=torch.full((cfg.B,), 10 ** 6, dtype=torch.int32, device=step.device))
    step.collapse()
    step.tree()
    with pytest.raises(binding.CtcsdError):
        step.check_status()
    assert (step.host("n_cand") == 0).all() and (step.host("n_nodes") == 1).all()
    base_tok, kv_len = parity_util.synth.gen_base(cfg, 2)
    zero = np.zeros((cfg.B, cfg.topN), dtype=np.int64)
    want = parity_util.orc.build_tree(base_tok, kv_len, np.full((cfg.B, cfg.topN, cfg.T), -1, dtype=np.int64), zero,
                                      np.zeros(cfg.B, dtype=np.int64), cfg.max_nodes)
    for name, w in zip(["node_tok", "parent", "depth", "pos"], want):
        np.testing.assert_array_equal(step.host(name), w, err_msg=name)
    step.set_inputs(sel_row=torch.arange(cfg.B, dtype=torch.int32, device=step.device))
    step.run()
    step.check_status()
    for k, v in good.items():
        np.testing.assert_array_equal(step.host(k), v, err_msg=k)


def test_invalid_arguments_are_rejected_on_the_host():
    import ctypes
    from paper_2412_00061_b200 import binding
    lib = binding.load_library()
    bad = binding.CConfig(1, 250, 100, 4, 3, 0, 8, 32, 4, 4, 64, 0, 0, 0)     # H not a multiple of 8
    n = ctypes.c_size_t(0)
    assert lib.ctcsd_workspace_bytes(ctypes.byref(bad), ctypes.byref(n)) == -1
    too_many = binding.CConfig(1, 256, 100, 7, 4, 0, 8, 32, 4, 4, 64, 0, 0, 0)  # 4^7 paths > 4096
    assert lib.ctcsd_workspace_bytes(ctypes.byref(too_many), ctypes.byref(n)) == -1
    h = ctypes.c_void_p()
    ok = binding.CConfig(1, 256, 100, 4, 3, 0, 8, 32, 4, 4, 64, 0, 0, 0)
    assert lib.ctcsd_create(ctypes.byref(h), ctypes.byref(ok), None, 0) == -3   # no workspace
    with pytest.raises(binding.CtcsdError):
        import torch
        hd = binding.Handle(1, 256, 100, 4, 3, 0, 8, 32, 4, 4, 64, 0)
        x = torch.zeros(1, 256, device="cuda")
        hd.draft_logits(x, x, None, None, x, x, x)          # wrong sizes and dtypes
