"""CPU-side checks of the C ABI: the library loads, exports every declared symbol,
and its integer host logic (mask generators) is bit-exact against the oracle's own."""
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2507_20030_b200 import build, binding
    build.build()
    return binding.load()


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(faedkv_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2507_20030_b200 import binding
    declared = _declared_symbols()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert declared == set(binding.EXPORTS)


@pytest.mark.parametrize("P,M", [(256, 32), (2048, 256), (32768, 4096), (16384, 2048), (4096, 128),
                                 (131072, 8192), (1000, 64), (250, 48)])
def test_mixed_mask_bit_exact_vs_oracle(lib, oracle, P, M):
    from paper_2507_20030_b200 import binding
    for layer in (0, 1, 7, 31):
        for seed in (20030100, 20030400, 5):
            a = binding.mask_mixed(P, M, layer, seed)
            b = oracle.mask_mixed(P, M, layer, seed)
            assert a.dtype == b.dtype == np.uint8 and a.tobytes() == b.tobytes()


@pytest.mark.parametrize("P,M", [(64, 0), (64, 1), (64, 33), (63, 32), (2048, 256)])
def test_lowpass_mask_bit_exact_vs_oracle(lib, oracle, P, M):
    from paper_2507_20030_b200 import binding
    assert binding.mask_lowpass(P, M).tobytes() == oracle.mask_lowpass(P, M).tobytes()


def test_mask_generators_reject_bad_requests(lib):
    from paper_2507_20030_b200 import binding
    with pytest.raises(binding.FaedkvError):
        binding.mask_lowpass(64, 34)
    with pytest.raises(binding.FaedkvError):
        binding.mask_mixed(256, 30, 0, 1)       # not a multiple of 16
    with pytest.raises(binding.FaedkvError):
        binding.mask_mixed(64, 64, 0, 1)        # more chunks than exist below P/2


def test_create_rejects_bad_configs_before_touching_cuda(lib):
    import ctypes
    from paper_2507_20030_b200 import binding
    h = ctypes.c_void_p()
    good = dict(n_layers=1, n_kv_heads=8, n_q_heads=32, head_dim=128, n_dft=2048, max_batch=1,
                kv_dtype=binding.F32, prefill_mode=0, twiddle_terms=0, decode_mode=0)
    for key, bad, code in [("head_dim", 64, -4), ("n_dft", 1, -1), ("n_q_heads", 12, -4),
                           ("n_q_heads", 128, -4), ("kv_dtype", 7, -1), ("max_batch", 0, -1),
                           ("twiddle_terms", 3, -1), ("n_layers", 0, -1), ("decode_mode", 5, -1),
                           ("n_defer", -1, -1), ("n_defer", 129, -1), ("n_sink", 2000, -1)]:
        cfg = binding.Config(**{**good, key: bad})
        assert lib.faedkv_create(ctypes.byref(cfg), ctypes.byref(h)) == code, key
        assert not h.value
    assert lib.faedkv_create(None, ctypes.byref(h)) == -1
    lib.faedkv_destroy(None)  # allowed


def test_selection_tooling_matches_the_oracle_bit_for_bit(lib, oracle):
    """Chunk ranges, ablation bins / gains and the greedy keep-mask: host-only integer logic, identical to
    the oracle's independent Python restatement."""
    import numpy as np
    from paper_2507_20030_b200 import binding
    rng = np.random.default_rng(3)
    for P, C in [(64, 22), (2048, 22), (100, 7), (32768, 22)]:
        for c in range(C):
            assert binding.chunk_range(P, C, c) == oracle.chunk_range(P, C, c)
        for c in (0, 1, C // 2, C - 1):
            lo, hi = oracle.chunk_range(P, C, c)
            m, g = binding.ablation_bins(P, lo, hi)
            om, og = oracle.ablation_bins(P, lo, hi)
            assert m.tobytes() == om.tobytes() and g.tobytes() == og.tobytes()
        for ratio in (0.05, 0.094, 0.125, 0.25, 1.0):
            delta = np.round(rng.standard_normal(C), 1)             # rounded: ties occur
            m, n = binding.mask_from_scores(P, C, delta, ratio)
            om, on = oracle.mask_from_scores(P, C, delta, ratio)
            assert n == on and m.tobytes() == om.tobytes(), (P, C, ratio)
    with pytest.raises(binding.FaedkvError):
        binding.chunk_range(64, 22, 22)
    with pytest.raises(binding.FaedkvError):
        binding.ablation_bins(64, 10, 10)
