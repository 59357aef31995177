"""The no-allocation tree-attention entry point against the CPU oracle and the regular entry point.

ctcsd_tree_attention_static serves callers that are not allowed to allocate device memory
when they run (an operator inside a runtime that owns the memory plan, a process whose
allocator is frozen after start-up): its scratch is a fixed array inside the library.  It must
give the same result as ctcsd_tree_attention, call after call, although every call reuses the
same scratch with the previous call's contents still in it.  This file is named so that pytest
collects it last."""
import ctypes

import numpy as np
import pytest

from paper_2412_00061_b200 import synth

pytestmark = pytest.mark.gpu


def _tree_inputs(cfg, seed, dev):
    import torch
    from oracle import ctcsd_oracle as orc
    from paper_2412_00061_b200.step import to_device
    rng = np.random.default_rng(seed)
    # a random ranked candidate list -> a tree through the oracle (test infrastructure)
    cand_tok = np.full((cfg.B, cfg.topN, cfg.T), -1, dtype=np.int64)
    cand_len = np.zeros((cfg.B, cfg.topN), dtype=np.int64)
    for b in range(cfg.B):
        for c in range(cfg.topN):
            l = int(rng.integers(1, cfg.T + 1))
            cand_len[b, c] = l
            cand_tok[b, c, :l] = rng.integers(0, 4, size=l)
    n_cand = np.full(cfg.B, cfg.topN, dtype=np.int64)
    base_tok, kv_len = synth.gen_base(cfg, seed)
    tree = orc.build_tree(base_tok, kv_len, cand_tok, cand_len, n_cand, cfg.max_nodes)
    mask, n_nodes = tree[4], tree[6]
    Q, K, V = synth.gen_attention(cfg, seed)
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).to(dev)
    return dict(Q=to_device(Q, "bf16", dev), K=to_device(K, "bf16", dev), V=to_device(V, "bf16", dev),
                kv_len=i32(kv_len), n_nodes=i32(n_nodes),
                mask=torch.from_numpy(mask.view(np.int64).copy()).to(dev))


def _host(t):
    return t.float().cpu().numpy()


def _oracle_attention(cfg, t):
    from oracle import ctcsd_oracle as orc
    return orc.tree_attention(_host(t["Q"]), _host(t["K"]), _host(t["V"]), t["kv_len"].cpu().numpy(),
                              t["n_nodes"].cpu().numpy(), t["mask"].cpu().numpy().view(np.uint64),
                              1.0 / float(cfg.D) ** 0.5)


def test_static_entry_point_matches_the_oracle_and_the_regular_one_twice_in_a_row():
    import torch
    from paper_2412_00061_b200 import binding
    dev = torch.device("cuda:0")
    base = synth.CONFIGS["c3"].replace(B=3, H=64, V=100, Hq=8, Hkv=4, kv_lo=70, kv_hi=700)
    # two different problems back to back: the second call finds the first call's partials in the scratch
    for seed, cfg in [(0, base), (1, base.replace(B=2, Hq=4, Hkv=4, kv_lo=5, kv_hi=130, D=64, max_nodes=32))]:
        t = _tree_inputs(cfg, seed, dev)
        want = _oracle_attention(cfg, t)
        h = binding.Handle(cfg.B, cfg.H, cfg.V, cfg.T, cfg.k, cfg.beam, cfg.topN, cfg.max_nodes, cfg.Hq, cfg.Hkv,
                           cfg.D, binding.DTYPE_BF16)
        scale = 1.0 / float(cfg.D) ** 0.5
        O_ref = torch.zeros(cfg.B, cfg.max_nodes, cfg.Hq, cfg.D, dtype=torch.bfloat16, device=dev)
        h.tree_attention(t["Q"], t["K"], t["V"], t["kv_len"], t["n_nodes"], t["mask"], scale, O_ref)
        assert h.poll_status() == 0
        status = torch.full((2,), 7, dtype=torch.int32, device=dev)
        for call in range(2):
            O = torch.full_like(O_ref, float("nan"))
            binding.tree_attention_static(t["Q"], t["K"], t["V"], t["kv_len"], t["n_nodes"], t["mask"], scale, O,
                                          out_status=status)
            torch.cuda.synchronize()
            assert status.tolist() == [0, 0]
            assert np.max(np.abs(_host(O) - want)) <= 2e-2, (seed, call)           # against the CPU oracle
            err = (O.float() - O_ref.float()).abs().max().item()                    # and against the handle path
            assert err <= 2e-2, (seed, call, err)
        h.close()


def test_static_entry_point_with_fewer_splits_than_it_would_like():
    """6 sequences x 8 heads x 128 nodes x 130 floats = 3.2 MB of partials per KV split; the sixteen
    splits that twelve (sequence, kv head) units would get need 51 MB, so the call has to settle for
    the ten that fit into the 32 MiB array.  Same result as the oracle and as the handle path."""
    import torch
    from paper_2412_00061_b200 import binding
    dev = torch.device("cuda:0")
    cfg = synth.CONFIGS["c4"].replace(B=6, H=64, V=100, Hq=8, Hkv=2, kv_lo=300, kv_hi=900, T=8, topN=32,
                                      max_nodes=128)
    assert 16 * cfg.B * cfg.Hq * cfg.max_nodes * (cfg.D + 2) * 4 > 32 << 20
    t = _tree_inputs(cfg, 5, dev)
    want = _oracle_attention(cfg, t)
    scale = 1.0 / float(cfg.D) ** 0.5
    status = torch.full((2,), 7, dtype=torch.int32, device=dev)
    for call in range(2):
        O = torch.full((cfg.B, cfg.max_nodes, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device=dev)
        binding.tree_attention_static(t["Q"], t["K"], t["V"], t["kv_len"], t["n_nodes"], t["mask"], scale, O,
                                      out_status=status)
        torch.cuda.synchronize()
        assert status.tolist() == [0, 0]
        assert np.max(np.abs(_host(O) - want)) <= 2e-2, call


def test_a_length_beyond_the_cache_is_recorded_and_reads_nothing():
    """kv_len[1] = Lcap + 1 cannot be served.  The library is told a cache capacity smaller than the
    buffers really are, so that even a kernel that ignored the check would stay inside the
    allocation.  Both entry points must record CTCSD_ERR_INVALID_ARG with the sequence index, write
    zero rows for that sequence and the right rows for the others.  Three query heads per kv head:
    the handle path runs the same warp-level kernel as the static one."""
    import torch
    from paper_2412_00061_b200 import binding
    lib = binding.load_library()
    dev = torch.device("cuda:0")
    cfg = synth.CONFIGS["c3"].replace(B=3, H=64, V=100, Hq=6, Hkv=2, kv_lo=40, kv_hi=100, D=64, max_nodes=32)
    t = _tree_inputs(cfg, 9, dev)
    Lcap = cfg.Lcap
    big = lambda a: torch.cat([a.reshape(-1), torch.zeros(a.numel(), dtype=a.dtype, device=dev)])   # twice the room
    K, V = big(t["K"]), big(t["V"])
    kv_bad = t["kv_len"].clone()
    kv_bad[1] = Lcap + 1
    good = _oracle_attention(cfg, t)
    scale = 1.0 / float(cfg.D) ** 0.5
    vp = ctypes.c_void_p
    stream = vp(torch.cuda.current_stream().cuda_stream)
    for path in ("static", "handle"):
        O = torch.full((cfg.B, cfg.max_nodes, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device=dev)
        if path == "static":
            status = torch.full((2,), 7, dtype=torch.int32, device=dev)
            rc = lib.ctcsd_tree_attention_static(stream, cfg.B, cfg.max_nodes, cfg.Hq, cfg.Hkv, cfg.D,
                                                 vp(t["Q"].data_ptr()), vp(K.data_ptr()), vp(V.data_ptr()), Lcap,
                                                 vp(kv_bad.data_ptr()), vp(t["n_nodes"].data_ptr()),
                                                 vp(t["mask"].data_ptr()), scale, vp(O.data_ptr()), vp(status.data_ptr()))
            assert rc == 0
            torch.cuda.synchronize()
            assert status.tolist() == [-1, 1]
        else:
            h = binding.Handle(cfg.B, cfg.H, cfg.V, cfg.T, cfg.k, cfg.beam, cfg.topN, cfg.max_nodes, cfg.Hq, cfg.Hkv,
                               cfg.D, binding.DTYPE_BF16)
            rc = lib.ctcsd_tree_attention(h._h, stream, vp(t["Q"].data_ptr()), vp(K.data_ptr()), vp(V.data_ptr()), Lcap,
                                          vp(kv_bad.data_ptr()), vp(t["n_nodes"].data_ptr()), vp(t["mask"].data_ptr()),
                                          scale, vp(O.data_ptr()))
            assert rc == 0
            assert h.poll_status() == -1
            assert h.poll_status() == 0
            h.close()
        got = _host(O)
        assert np.all(got[1] == 0)
        for b in (0, 2):
            assert np.max(np.abs(got[b] - good[b])) <= 2e-2, (path, b)


def test_static_entry_point_rejects_what_does_not_fit():
    import torch
    from paper_2412_00061_b200 import binding
    lib = binding.load_library()
    dev = torch.device("cuda:0")
    one = torch.zeros(16, dtype=torch.int64, device=dev)
    p = ctypes.c_void_p(one.data_ptr())
    # 64 sequences x 64 heads x 128 nodes x 130 floats = 272 MB of partials per split: beyond the 32 MiB array.
    # The size check comes before anything is launched, so the dummy pointers are never used.
    rc = lib.ctcsd_tree_attention_static(None, 64, 128, 64, 8, 128, p, p, p, 4096, p, p, p, 1.0, p, None)
    assert rc == -7
    assert b"scratch" in lib.ctcsd_strerror(rc)
    assert lib.ctcsd_tree_attention_static(None, 1, 64, 8, 3, 128, p, p, p, 4096, p, p, p, 1.0, p, None) == -1
