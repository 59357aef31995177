"""The no-allocation tree-attention entry point against the regular one.

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


def test_static_entry_point_matches_the_regular_one_twice_in_a_row():
    import torch
    from paper_2412_00061_b200 import binding
    dev = torch.device("cuda:0")
    base = synth.CONFIGS["c3"].replace(B=3, H=64, V=100, Hq=8, Hkv=4, kv_lo=70, kv_hi=700)
    # two different problems back to back: the second call finds the first call's partials in the scratch
    for seed, cfg in [(0, base), (1, base.replace(B=2, Hq=4, Hkv=4, kv_lo=5, kv_hi=130, D=64, max_nodes=32))]:
        t = _tree_inputs(cfg, seed, dev)
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
            err = (O.float() - O_ref.float()).abs().max().item()
            assert err <= 2e-2, (seed, call, err)
        h.close()


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
