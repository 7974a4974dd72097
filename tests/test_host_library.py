"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its
host-side logic (status strings, workspace sizing, argument validation) works without a GPU."""
import ctypes as C
import os
import re

import pytest

import paper_2501_17116_b200 as fp4
from paper_2501_17116_b200 import build as fp4_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fp4_build.build()
    return fp4.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "fp4_linear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fp4_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_three_named_entry_points():
    names = _declared_functions()
    for required in ("fp4_quantize", "fp4_linear_fwd", "fp4_linear_bwd"):
        assert required in names


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert len(names) >= 8
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in the header but not exported"
    assert sorted(fp4.EXPORTS) == names       # the binding covers the whole header


def test_status_strings(lib):
    assert lib.fp4_status_string(0) == b"ok"
    seen = {lib.fp4_status_string(-c) for c in range(1, 9)}
    assert len(seen) == 8 and b"unknown status" not in seen
    assert lib.fp4_status_string(-99) == b"unknown status"


def test_workspace_sizes_are_monotone_and_cover_the_fp32_result(lib):
    small = lib.fp4_workspace_bytes(256, 1024, 1024)
    big = lib.fp4_workspace_bytes(4096, 2048, 5504)
    assert 0 < small < big
    assert big >= 4096 * 5504 * 4 + 4096 * 5504            # fp32 result + both dY code tensors
    assert lib.fp4_workspace_bytes(0, 128, 128) == 0
    assert lib.fp4_step_host_workspace_bytes(256, 1024, 1024, 0.99) > small


def test_null_and_shape_validation_needs_no_gpu(lib):
    q = fp4.binding.fp4_qtensor()
    dummy = C.c_void_p(256)
    assert lib.fp4_quantize(None, None, dummy, 128, 128, 0, 1.0, None, C.byref(q), dummy) == -1
    assert lib.fp4_gemm(None, None, dummy, dummy, 128, 128, 128, None, None, dummy, 1, 0, dummy) == -1
    assert lib.fp4_destroy(None) == -1
    assert lib.fp4_profile_enable(None, 1) == -1
    assert lib.fp4_launch_count(None) == -1


def test_create_without_a_gpu_returns_an_error_code(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = C.c_void_p()
    assert lib.fp4_create(C.byref(h), 0, 1024) == -6
    assert not h.value


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        fp4.load_library(str(tmp_path / "libfp4linear.so"))


def test_tail_capacity_matches_the_header_rule():
    assert fp4.tail_capacity(256, 1024, 0.99) == 2 * 2621
    assert fp4.tail_capacity(128, 128, 1.0) == 0


def test_sparse_capacity_is_the_librarys_rule(lib):
    """Two tails of n_tail = round((1 - alpha) n) entries (Section 3.2 as read here); per token two
    tails of round((1 - alpha) cols) entries in every row."""
    cap = lib.fp4_sparse_capacity
    assert cap(256, 1024, 0.99, fp4.FP4_QUANTILE_SIGNED) == 2 * 2621            # n_tail of the first configuration
    assert cap(256, 1024, 0.99, fp4.FP4_QUANTILE_ABS) == 2 * 2621
    assert cap(256, 1024, 0.99, fp4.FP4_QUANTILE_TOKEN) == 2 * 256 * 10
    assert cap(16384, 13824, 0.99, fp4.FP4_QUANTILE_SIGNED) == 2 * 2264924       # the largest activation of the workloads
    assert cap(128, 128, 1.0, fp4.FP4_QUANTILE_SIGNED) == 0
    assert cap(128, 128, 0.4, fp4.FP4_QUANTILE_SIGNED) == -1
    assert cap(128, 128, 0.99, 7) == -1
    assert cap(0, 128, 0.99, fp4.FP4_QUANTILE_SIGNED) == -1


def test_debug_switches_validate_their_arguments(lib):
    assert lib.fp4_debug_set(None, 1, 1000) == -1


def test_l2_probe_validates_its_arguments(lib):
    dummy = C.c_void_p(4096)
    assert lib.fp4_l2_read_probe(None, None, 1 << 20, 1, 1, dummy) == -1
    assert lib.fp4_l2_read_probe(None, dummy, 1000, 1, 1, dummy) == -7           # not a multiple of 32 KB
    assert lib.fp4_l2_read_probe(None, dummy, 1 << 20, 0, 1, dummy) == -7
    assert lib.fp4_l2_read_probe(None, C.c_void_p(4100), 1 << 20, 1, 1, dummy) == -7   # misaligned
