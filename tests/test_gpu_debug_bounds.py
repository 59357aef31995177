"""The debug-bounds build of the library (-DCTCSD_DEBUG_BOUNDS: every kernel checks the index of
its stores into the callers' arrays and its internal lists, records a failed check in the device
status word and skips the store) on small shapes of every code path: the status word must stay
clean and the results must be the ones the oracle checks in the regular build."""
import numpy as np
import pytest

from paper_2412_00061_b200 import synth

pytestmark = pytest.mark.gpu

C = synth.CONFIGS
SHAPES = {
    "enum_bf16": C["c2"].replace(name="enum_bf16", H=520, V=2999, Hq=8, Hkv=8, kv_lo=200, kv_hi=200),
    "beam_ragged": C["c3"].replace(name="beam_ragged", B=3, H=512, V=1777, Hq=4, Hkv=4, kv_lo=70, kv_hi=300, beam=16),
    "beam_gqa": C["c5"].replace(name="beam_gqa", B=5, H=1024, V=1200, Hq=8, Hkv=2, kv_lo=100, kv_hi=500),
    "fp32": C["c1"],
    "limits": C["c4"].replace(name="limits", B=2, H=512, V=1500, Hq=8, Hkv=4, kv_lo=50, kv_hi=700, T=8, k=8, beam=128,
                              topN=64, max_nodes=256),
}


@pytest.fixture()
def debug_library():
    from paper_2412_00061_b200 import binding, build
    lib = binding.use_library(build.build(debug_bounds=True))
    assert lib.ctcsd_debug_bounds_enabled() == 1
    yield lib
    assert binding.use_library(None).ctcsd_debug_bounds_enabled() == 0


@pytest.mark.parametrize("name", sorted(SHAPES))
def test_small_shapes_under_the_debug_bounds_build(name, debug_library):
    from tests.parity_util import run_parity, run_parity_raw
    r = run_parity(SHAPES[name], seed=1)          # every stage against the oracle; check_status() after each call
    assert r["step"].h.lib.ctcsd_debug_bounds_enabled() == 1
    if SHAPES[name].beam == 0:
        run_parity_raw(SHAPES[name], seed=1)
