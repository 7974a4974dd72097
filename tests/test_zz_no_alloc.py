"""The allocation-free threshold entry point against the regular quantiser.

Some callers are not allowed to allocate device memory (they run inside a pool-only framework or
a real-time loop) and so cannot own a context with its cudaMalloc'ed workspace.  For them the
library offers fp4_quantile_thresholds_static, whose scratch is a fixed array in the library
image.  That array is shared by all calls and keeps the previous call's contents, so the check
is made on two calls in a row with different inputs: the second one only passes if the first
one's histogram was cleared.
"""
import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def test_static_thresholds_equal_the_quantisers_on_two_calls_in_a_row(lib):
    cfg = WL.CONFIGS[0]
    x1 = _dev(WL.activations(cfg, 1024, seed=0))                     # 256 x 1024, alpha 0.99
    x2 = _dev(WL.activations(WL.CONFIGS[1], 2048, seed=3, M=512))    # other shape and distribution
    ctx = lib.Context(0, 256 << 20)
    want1 = lib.fp4_quantize(ctx, x1, 0, alpha=0.99).thresholds
    want2 = lib.fp4_quantize(ctx, x2, 0, alpha=0.999).thresholds
    out = torch.empty(2, dtype=torch.float32, device="cuda")
    got1 = lib.fp4_quantile_thresholds_static(x1, 0.99, out=out).clone()
    got2 = lib.fp4_quantile_thresholds_static(x2, 0.999, out=out).clone()
    torch.cuda.synchronize()
    # thresholds are order statistics of BF16 data: the tolerance of the threshold tests is "bit exact"
    assert torch.equal(got1, want1)
    assert torch.equal(got2, want2)
    assert got1[0] < 0 < got1[1]
    ctx.close()


def test_static_thresholds_equal_the_oracles(lib):
    """The same call against the CPU oracle's order statistics, on two calls in a row, the second
    at the largest row count the fixed scratch takes."""
    out = torch.empty(2, dtype=torch.float32, device="cuda")
    a1 = WL.activations(WL.CONFIGS[0], 1024, seed=5)                               # 256 x 1024
    a2 = WL.activations(WL.CONFIGS[1], 128, seed=6, M=lib.binding.FP4_STATIC_MAX_ROWS)   # 65536 x 128
    for bits, alpha in ((a1, 0.99), (a2, 0.999), (a1, 0.97)):
        got = lib.fp4_quantile_thresholds_static(_dev(bits), alpha, out=out).cpu().numpy()
        lo, hi, _ = O.quantile_thresholds(O.bf16_bits_to_f64(bits), alpha)
        assert (float(got[0]), float(got[1])) == (float(lo), float(hi))


def test_static_entry_rejects_what_its_fixed_scratch_cannot_hold(lib):
    raw = lib.load_library()
    x = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty(2, dtype=torch.float32, device="cuda")
    too_many_rows = lib.binding.FP4_STATIC_MAX_ROWS + 128
    rc = raw.fp4_quantile_thresholds_static(None, x.data_ptr(), too_many_rows, 128, 0.99, out.data_ptr())
    assert rc == -9
    assert b"fixed scratch" in raw.fp4_status_string(rc)
    assert raw.fp4_quantile_thresholds_static(None, x.data_ptr(), 100, 128, 0.99, out.data_ptr()) == -2
    assert raw.fp4_quantile_thresholds_static(None, x.data_ptr(), 128, 128, 1.0, out.data_ptr()) == -3
