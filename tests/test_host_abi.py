"""CPU-only checks of the C-ABI library: it builds, loads, exports every declared symbol, and
its host-side helpers agree with what the paper fixes.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2602_02599_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding._lib()


def test_every_declared_symbol_is_exported(lib):
    header = "".join(open(os.path.join(ROOT, "include", f)).read() for f in sorted(os.listdir(os.path.join(ROOT, "include"))))
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rap_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_retained_counts_follow_table13_and_workloads(lib):
    gold = os.path.join(ROOT, "tests", "golden", "table13_retained_fraction.txt")
    for line in open(gold):
        if line.strip() and not line.startswith("#"):
            rho, frac = line.split()
            P, _ = binding.rap_retained_counts(float(rho), 128)
            assert abs(P / 64 - float(frac)) < 5.1e-4
    for w in synth.CONFIGS.values():
        assert binding.rap_retained_counts(w.rho, w.head_dim) == (w.n_pairs, w.n_vch)
    P, dv = ctypes.c_int32(), ctypes.c_int32()
    for rho, D in [(0.0, 128), (1.5, 128), (0.5, 127), (float("nan"), 128)]:
        assert lib.rap_retained_counts(rho, D, ctypes.byref(P), ctypes.byref(dv)) == binding.RAP_EINVAL
    assert lib.rap_retained_counts(0.5, 128, None, ctypes.byref(dv)) == binding.RAP_EINVAL


def test_cache_offset_is_dense_row_major(lib):
    H, cap, W = 8, 32832, 90
    assert binding.rap_cache_elem_offset(H, cap, W, 0, 0, 0, 0) == 0
    assert binding.rap_cache_elem_offset(H, cap, W, 0, 0, 1, 0) == W
    assert binding.rap_cache_elem_offset(H, cap, W, 0, 1, 0, 0) == cap * W
    assert binding.rap_cache_elem_offset(H, cap, W, 31, 7, cap - 1, W - 1) == 32 * H * cap * W - 1   # > 2^31
    # a tile of 8 rows starts on a 16-byte boundary for every row width (bf16)
    for W in (90, 116, 115, 102, 64, 128):
        assert (binding.rap_cache_elem_offset(H, cap, W, 3, 5, 64, 0) * 2) % 16 == 0


def test_status_strings_and_bad_descriptions(lib):
    for s in range(10):
        assert lib.rap_status_string(s).decode().startswith("RAP_")
    good = dict(n_layers=1, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, rope_theta=10000.0, pairing=0,
                dtype=0, max_batch=1, max_rows=1)
    for key, val in [("n_layers", 0), ("head_dim", 63), ("n_q_heads", 5), ("rope_theta", 1.0), ("pairing", 2),
                     ("dtype", 7), ("max_batch", 0), ("hidden", 255), ("n_q_heads", 18)]:
        d = dict(good)
        d[key] = val
        desc = binding.rap_model_desc(**d)
        ctx = ctypes.c_void_p()
        assert lib.rap_create(ctypes.byref(desc), ctypes.byref(ctx)) == binding.RAP_EINVAL, key
        assert not ctx
    assert lib.rap_create(None, None) == binding.RAP_EINVAL
    assert lib.rap_destroy(None) == binding.RAP_EINVAL


def test_create_without_a_gpu_reports_cuda_error(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.RapError) as e:
        binding.RapContext(1, 256, 4, 2, 64, 10000.0, 0, 0, 1)
    assert e.value.status == binding.RAP_ECUDA


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/librap_b200.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding._lib()


def test_budget_alloc_matches_the_oracle(lib):
    """rap_budget_alloc (host C++) against the oracle's Algorithm 2 on seeded scores, with clipping cases."""
    import numpy as np
    from oracle import rap_oracle as O
    rng = np.random.default_rng(9)
    for L, H, D, rho, spread in [(32, 8, 128, 0.7, 1.0), (28, 8, 128, 0.9, 3.0), (48, 8, 128, 0.5, 0.3), (4, 1, 64, 0.5, 50.0),
                                 (6, 2, 16, 0.2, 8.0)]:
        sc = rng.lognormal(0, 1, (L, H, D // 2)) * np.exp(rng.normal(0, np.log1p(spread), L))[:, None, None]
        got_p, got_v = binding.rap_budget_alloc(sc, rho, D)
        want_p, want_v = O.budget_alloc(sc, rho, D)
        assert np.array_equal(got_p, want_p) and np.array_equal(got_v, want_v), (L, rho)
    n = np.zeros(2, dtype=np.int32)
    bad = np.ones((2, 1, 8))
    assert lib.rap_budget_alloc(2, 1, 16, binding._ptr(bad), 0.0, binding._ptr(n), binding._ptr(n)) == binding.RAP_EINVAL
    assert lib.rap_budget_alloc(2, 1, 15, binding._ptr(bad), 0.5, binding._ptr(n), binding._ptr(n)) == binding.RAP_EINVAL


def test_every_named_workload_has_both_shape_specialised_scans():
    """The build instantiates the tensor-core scan (and the FP32-pipe scan behind it) for the head shape of every
    bf16 workload the benchmark and the sweep name, so none of them can end up on a slower generic tier."""
    from paper_2602_02599_b200 import build, synth
    mma, fp32 = set(build.mma_shapes()), set(build.scan_shapes())
    for name, w in synth.CONFIGS.items():
        if w.dtype != "bf16":
            continue
        shape = (w.n_q_heads // w.n_kv_heads, w.n_pairs, w.n_vch)
        assert shape in mma, (name, shape)
        assert shape in fp32, (name, shape)
    # layer-adaptive budgets (d_v' = 2P) of the shaped models all have the tensor-core form
    for G in (3, 4, 5):
        for P in range(16, 65):
            assert (G, P, 2 * P) in mma
