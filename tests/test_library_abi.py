"""The C-ABI library builds for sm_100a, loads, and exports every symbol include/rtopk.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rtopk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rtopk_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_named_entry_points():
    names = _declared_symbols()
    for must in ("rtopk_sparsify", "rtopk_aggregate", "rtopk_step"):
        assert must in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2005_10761_b200 import build, binding
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    declared = _declared_symbols()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in rtopk.h but not exported"
    # the binding covers the same set, under the same names
    assert sorted(binding.EXPORTS) == declared
    loaded = binding.load_library()
    assert loaded.rtopk_version() >= 100
    assert loaded.rtopk_status_string(0) == b"ok"
    assert b"invalid" in loaded.rtopk_status_string(1)


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2005_10761_b200 import RTopK
    with pytest.raises(RuntimeError):
        RTopK(d_max=16, W_max=1, r_max=4, k_max=2)


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2005_10761_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "oracle/" not in src, f


def test_warmup_sizes_host_function_matches_the_oracle():
    """rtopk_warmup_sizes is host-only arithmetic: callable without a GPU.  The contract is one formula in
    binary64, k = max(1, min(d, floor(d * initial * pow(final / initial, t / T)))) for t < T, evaluated in
    that order with the C library's pow, and r = min(d, n k): integer outputs, so both sides must agree
    exactly."""
    import oracle
    import paper_2005_10761_b200 as rt
    d, n = 1 << 20, 8
    for t in range(7):
        assert rt.warmup_sizes(d, n, 0.25, 1.0 / 1024, 4, t) == oracle.warmup_sizes(d, n, 0.25, 1.0 / 1024, 4, t)
    for (dd, nn, hi, lo, T) in [(11_173_962, 5, 0.3, 0.001, 50), (25_557_032, 16, 1.0, 0.001, 97),
                                (1 << 28, 32, 0.25, 0.0001, 1000), (1000, 3, 0.5, 0.01, 7)]:
        for t in range(0, T + 20, max(1, T // 40)):
            assert rt.warmup_sizes(dd, nn, hi, lo, T, t) == oracle.warmup_sizes(dd, nn, hi, lo, T, t), (dd, t)
    import pytest
    with pytest.raises(rt.RTopKError):
        rt.warmup_sizes(100, 4, 0.001, 0.01, 5, 0)


def test_workload_recipes_scale_by_length_and_by_rows():
    """The seeded input recipes: another length keeps the ratios r / d and k / r (floor, at least 1), another
    row count keeps everything else; the per-tensor workload is tied to its tensor sizes, so only its rows
    may change."""
    from paper_2005_10761_b200 import workloads as wl
    cfgs = wl.configs()
    c3 = cfgs["c3_f32"]
    s = wl.scaled(c3, d=1_000_000, W=3)
    assert (s.d, s.W, s.r, s.k) == (1_000_000, 3, c3.r * 1_000_000 // c3.d, c3.k * 1_000_000 // c3.d)
    assert wl.scaled(c3, d=10).r == 1 and wl.scaled(c3, d=10).k == 1
    c4 = cfgs["c4"]
    one = wl.scaled(c4, d=c4.d, W=1, name="c4_W1")
    assert one.W == 1 and one.name == "c4_W1"
    assert (one.seg_off, one.seg_r, one.seg_k, one.d) == (c4.seg_off, c4.seg_r, c4.seg_k, c4.d)
    with pytest.raises(AssertionError):
        wl.scaled(c4, d=c4.d // 2)
