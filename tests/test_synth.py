"""The shared input generators: determinism, shapes, and exact dtype rounding."""
import numpy as np
import torch

from paper_2412_00061_b200 import synth


def test_round_bf16_matches_library_rounding():
    rng = np.random.default_rng(0)
    a = (rng.normal(size=100000) * 10.0 ** rng.integers(-6, 6, size=100000)).astype(np.float32)
    got = synth.round_bf16(a)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(got, want)


def test_generators_are_seeded_and_shaped():
    cfg = synth.CONFIGS["c1"]
    x, Wd, bb = synth.gen_draft(cfg, seed=0)
    x2, Wd2, _ = synth.gen_draft(cfg, seed=0)
    x3, _, _ = synth.gen_draft(cfg, seed=1)
    assert x.shape == (1, 256) and Wd.shape == (4, 1001, 256) and bb.tolist() == [1.0]
    np.testing.assert_array_equal(x, x2)
    np.testing.assert_array_equal(Wd, Wd2)
    assert not np.array_equal(x, x3)
    assert abs(float(Wd.std()) - 0.02) < 1e-3
    base_tok, kv_len = synth.gen_base(synth.CONFIGS["c3"], seed=0)
    assert base_tok.shape == (8,) and kv_len.min() >= 512 and kv_len.max() <= 2048
    small = synth.CONFIGS["c3"].replace(H=64, V=100, kv_lo=5, kv_hi=9, Hq=4, Hkv=2, D=16)
    Q, K, V = synth.gen_attention(small, seed=0)
    assert Q.shape == (8, 64, 4, 16) and K.shape == V.shape == (8, 2, small.Lcap, 16)
    assert small.Lcap % 64 == 0 and small.Lcap >= 9 + 64
    assert set(synth.gen_draft(small, seed=0)[2].tolist()) == {0.0, 1.0, 2.0}
    np.testing.assert_array_equal(K, synth.round_bf16(K))      # already bf16-representable
