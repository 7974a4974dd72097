"""Randomised differential test of the whole layer against the oracle.

Seeded draws over shapes (multiples of 128, ragged against every tile size), clamp fractions,
activation distributions, number of outlier channels, GEMM kind and DGE setting.  Every draw checks
what the fixed cases check: saved operands bit for bit, the three outputs within the bar stated in
test_gpu_linear.py.  The draws are fixed by the seed, so a failure reproduces; FP4_RANDOM_DRAWS in
the environment sets how many are made (default 16), FP4_RANDOM_SEED moves the generators to
another sequence of cases (default 0), FP4_RANDOM_BIG_DRAWS and FP4_RANDOM_HOST_SEQUENCES set the
number of many-tile layers and of further host-step sequences; FP4_TEST_NO_OVERLAP=1 runs them with the library's side
streams switched off.
"""
import os

import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL
from test_gpu_linear import _dev, _saved_matches, assert_bf16_rounding, assert_close_f32, fp32_sum_floor, tail_floor

pytestmark = pytest.mark.gpu
SEED_SHIFT = 100003 * int(os.environ.get("FP4_RANDOM_SEED", "0"))


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0, 1 << 30)
    if os.environ.get("FP4_TEST_NO_OVERLAP"):          # the same draws with every kernel on one stream
        c.set_overlap(False)
    yield c
    c.close()


def _fp8_floor(terms, contraction):
    """Allowance for a GEMM with an E4M3 operand: its products are not on one binary scale, so the
    tensor cores' fp32 accumulation (rounding toward zero, one addition per 32 contraction columns)
    is no longer exact: at most 2 * 2^-23 of the running sum per instruction, bounded here against
    the sum of the magnitudes of the products.  GEMMs of E2M1 operands alone are exact: no floor."""
    return 2.0 * -(-contraction // 32) * 2.0 ** -23 * terms


def _draws(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        M = int(rng.choice([128, 256, 384, 512, 1024]))
        K = int(rng.choice([128, 256, 384, 640, 1152]))
        N = int(rng.choice([128, 256, 384, 512, 640]))
        alpha = float(rng.choice([1.0, 0.9999, 0.999, 0.99, 0.97, 0.9]))
        dist = str(rng.choice(["normal", "student_t3", "laplace"]))
        hot = int(rng.choice([0, 2, 9, 40]))
        kind = int(rng.integers(0, 2))
        dge = bool(rng.integers(0, 2))
        # FP8 settings need the byte-container kind; an E4M3 activation is not clamped
        fp8 = str(rng.choice(["none", "none", "w8", "a8", "dy8", "w8+dy8", "dy5", "w8+dy5", "a5"])) if kind == 1 else "none"
        if fp8 in ("a8", "a5"):
            alpha = 1.0
        out.append((i, M, K, N, alpha, dist, hot, kind, dge, fp8))
    return out


@pytest.mark.parametrize("i,M,K,N,alpha,dist,hot,kind,dge,fp8",
                         _draws(int(os.environ.get("FP4_RANDOM_DRAWS", "16")), seed=2501 + SEED_SHIFT))
def test_random_layer_matches_oracle(lib, ctx, i, M, K, N, alpha, dist, hot, kind, dge, fp8):
    _layer_case(lib, ctx, 1000 + i, M, K, N, alpha, dist, hot, kind, dge, fp8, out_f32=True)


def _many_tile_draws(n, seed):
    """Shapes whose GEMMs have more 128 x 240 tiles than the GPU has SMs (forward 176-234, and with the
    large K the backward's two problems as well), so that CTAs walk several tiles and both
    accumulator buffers; every other draw stores BF16 outputs."""
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        M = int(rng.choice([2048, 2304]))
        K = int(rng.choice([256, 640, 2560]))
        N = int(rng.choice([2560, 2944, 3072]))
        alpha = float(rng.choice([1.0, 0.999, 0.99, 0.97]))
        dist = str(rng.choice(["normal", "student_t3", "laplace"]))
        hot = int(rng.choice([0, 9, 40]))
        kind = int(rng.integers(0, 2))
        dge = bool(rng.integers(0, 2))
        out.append((i, M, K, N, alpha, dist, hot, kind, dge, i % 2 == 0))
    return out


@pytest.mark.parametrize("i,M,K,N,alpha,dist,hot,kind,dge,out_f32",
                         _many_tile_draws(int(os.environ.get("FP4_RANDOM_BIG_DRAWS", "3")), seed=4099 + SEED_SHIFT))
def test_random_layer_with_more_tiles_than_sms(lib, i, M, K, N, alpha, dist, hot, kind, dge, out_f32):
    c = lib.Context(0, int(lib.load_library().fp4_workspace_bytes(M, K, N)))
    try:
        _layer_case(lib, c, 700000 + i, M, K, N, alpha, dist, hot, kind, dge, "none", out_f32=out_f32)
    finally:
        c.close()


def _degenerate(bits_list, rng):
    """Zero rows and columns, rows on scales 2^-20 .. 2^20 and a few huge values in one column of each
    of the three tensors: vectors whose absmax is 0, de-scales far from 1, residuals near and beyond
    what the dense tail's FP16 operands hold."""
    out = []
    for bits in bits_list:
        x = O.bf16_bits_to_f64(bits).astype(np.float32)
        r, c = x.shape
        if rng.random() < 0.7:
            x[rng.integers(0, r, size=int(rng.integers(1, 4)))] = 0.0
        if rng.random() < 0.7:
            x[:, rng.integers(0, c, size=int(rng.integers(1, 4)))] = 0.0
        if rng.random() < 0.5:
            x *= np.exp2(rng.integers(-20, 21, size=(r, 1))).astype(np.float32)
        if rng.random() < 0.5:
            rows = rng.integers(0, r, size=int(rng.integers(1, 6)))
            x[rows, int(rng.integers(0, c))] *= np.float32(10.0 ** rng.integers(3, 9))
        out.append(WL.to_bf16_bits(x))
    return out


@pytest.mark.parametrize("i,M,K,N,alpha,dist,hot,kind,dge,fp8",
                         _draws(int(os.environ.get("FP4_RANDOM_DRAWS", "16")), seed=9973 + SEED_SHIFT))
def test_random_layer_with_degenerate_vectors(lib, ctx, i, M, K, N, alpha, dist, hot, kind, dge, fp8):
    _layer_case(lib, ctx, 300000 + i, M, K, N, alpha, dist, hot, kind, dge, fp8, out_f32=True,
                mutate=np.random.default_rng(77000 + i + SEED_SHIFT))


@pytest.mark.parametrize("i,M,K,N,alpha,dist,hot,kind,dge,fp8",
                         _draws(int(os.environ.get("FP4_RANDOM_DRAWS", "16")), seed=31337 + SEED_SHIFT))
def test_random_layer_in_the_other_quantile_modes(lib, i, M, K, N, alpha, dist, hot, kind, dge, fp8):
    """The two variants of the clamp (one threshold on |x|; thresholds per token) through the whole
    layer, forward and backward, FP8 settings and dense tail included where the draw has them."""
    if alpha >= 1.0:
        alpha = 0.99
        if fp8 in ("a8", "a5"):
            fp8 = "none"
    quantile = "abs" if i % 2 == 0 else "token"
    c = lib.Context(0, 1 << 30)
    c.set_quantile_mode(lib.FP4_QUANTILE_ABS if quantile == "abs" else lib.FP4_QUANTILE_TOKEN)
    try:
        _layer_case(lib, c, 500000 + i, M, K, N, alpha, dist, hot, kind, dge, fp8, out_f32=True, quantile=quantile)
    finally:
        c.close()


def _layer_case(lib, ctx, case_seed, M, K, N, alpha, dist, hot, kind, dge, fp8, out_f32, mutate=None,
                quantile="signed"):
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=case_seed + SEED_SHIFT, alpha_outliers=hot, dist=dist)
    if mutate is not None:
        a_bits, w_bits, dy_bits = _degenerate([a_bits, w_bits, dy_bits], mutate)
    fmt_a = {"a8": "e4m3", "a5": "e5m2"}.get(fp8, "e2m1")
    fmt_w = "e4m3" if "w8" in fp8 else "e2m1"
    fmt_dy = "e4m3" if "dy8" in fp8 else ("e5m2" if "dy5" in fp8 else "e2m1")
    code = {"e2m1": lib.FP4_FORMAT_E2M1, "e4m3": lib.FP4_FORMAT_E4M3, "e5m2": lib.FP4_FORMAT_E5M2}
    f = O.linear_fwd(a_bits, w_bits, alpha, fmt_a=fmt_a, fmt_w=fmt_w, quantile=quantile)
    b = O.linear_bwd(dy_bits, w_bits, f, dge_on=dge, fmt_dy=fmt_dy)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    ctx.status.zero_()
    y32, sa, sw = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind, out_f32=out_f32, fmt_a=code[fmt_a],
                                     fmt_w=code[fmt_w])
    da32, dw32 = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind, out_f32=out_f32, dge_on=dge,
                                    dy_fmt=code[fmt_dy])
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    if fp8 in ("none", "dy8", "dy5"):
        _saved_matches(sa, sw, f)
    else:
        np.testing.assert_array_equal(sa.amax.cpu().numpy(), f.qa.amax)
        np.testing.assert_array_equal(sw.amax.cpu().numpy(), f.qw.amax)
        np.testing.assert_array_equal(sa.codes.cpu().numpy(), f.qa.packed() if fmt_a == "e2m1" else f.qa.codes)
        np.testing.assert_array_equal(sw.codes_t.cpu().numpy(),
                                      f.qw.packed_t() if fmt_w == "e2m1" else np.ascontiguousarray(f.qw.codes.T))
    if alpha < 1.0 and quantile == "token":
        from test_gpu_quantize import _check_token_mode
        _check_token_mode(sa, f.qa)
    elif alpha < 1.0:
        th = sa.thresholds.cpu().numpy()
        assert (float(th[0]), float(th[1])) == (f.qa.lo, f.qa.hi)
        assert int(sa.nnz.item()) == int(np.count_nonzero(f.qa.residual))
    # heavy residuals with enough tokens may send hot columns through the GEMM's dense tail
    floor_y = tail_floor(f, w_bits) if (alpha <= 0.995 and M >= 512) else 0.0
    floor_da = floor_dw = 0.0
    va, vw = np.abs(f.qa.values()), np.abs(f.qw.values())
    vg1, vg2 = np.abs(b.qg_dgrad.values()), np.abs(b.qg_wgrad.values())
    d64 = lambda q: q.descale.astype(np.float64)
    if fmt_a != "e2m1" or fmt_w != "e2m1":
        floor_y = floor_y + _fp8_floor((va @ vw) * d64(f.qa)[:, None] * d64(f.qw)[None, :], K)
    if fmt_dy != "e2m1" or fmt_w != "e2m1":
        floor_da = _fp8_floor((vg1 @ vw.T) * d64(b.qg_dgrad)[:, None], N)
    if fmt_a != "e2m1" or fmt_dy != "e2m1":
        floor_dw = _fp8_floor((va.T @ vg2) * d64(b.qg_wgrad)[None, :] * b.dge, M)
    if alpha < 1.0:
        # fp32 accumulation of the per-entry compensation (matters only where its terms cancel)
        floor_y = floor_y + fp32_sum_floor(f.qa.residual, np.abs(O.bf16_bits_to_f64(w_bits)))
        floor_dw = floor_dw + fp32_sum_floor(f.qa.residual, np.abs(O.bf16_bits_to_f64(dy_bits)), transpose=True) * np.abs(b.dge)
    if not out_f32:
        assert_bf16_rounding(y32, f.y, "Y", f.y_fp4, f.y_comp, floor_y)
        assert_bf16_rounding(da32, b.da, "dA", None, None, floor_da)
        assert_bf16_rounding(dw32, b.dw, "dW", b.s_fp4 * b.dge, b.s_comp * b.dge, floor_dw)
        return
    assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y", floor_y)
    assert_close_f32(da32.cpu().numpy(), b.da, b.da, None, "dA", floor_da)
    assert_close_f32(dw32.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, "dW", floor_dw)


def _quantizer_draws(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        rows = int(rng.choice([128, 256, 512, 1024]))
        cols = int(rng.choice([128, 384, 640, 1152, 2048]))
        alpha = float(rng.choice([0.9999, 0.999, 0.99, 0.97, 0.9]))
        spread = int(rng.choice([0, 4, 20, 60]))           # binades over which the rows' scales are spread
        zeros = float(rng.choice([0.0, 0.01, 0.5]))        # fraction of exact zeros
        out.append((i, rows, cols, alpha, spread, zeros))
    return out


@pytest.mark.parametrize("i,rows,cols,alpha,spread,zeros",
                         _quantizer_draws(int(os.environ.get("FP4_RANDOM_DRAWS", "16")), seed=1711 + SEED_SHIFT))
def test_random_clamping_quantizer_is_bit_exact(lib, ctx, i, rows, cols, alpha, spread, zeros):
    """Thresholds, codes in both layouts, amax and the sparse residual on tensors whose rows live on
    scales spread over many binades (values outside the histogram kernel's window, subnormals),
    with ties and exact zeros of both signs."""
    from test_gpu_quantize import _check_dense, _check_sparse, _check_token_mode
    rng = np.random.default_rng(5000 + i + SEED_SHIFT)
    a = rng.standard_normal((rows, cols)).astype(np.float32)
    if spread:
        a *= np.exp2(rng.integers(-spread, spread + 1, size=(rows, 1))).astype(np.float32)
    if i % 3 == 0:
        a = np.round(a * 4) / 4                            # many ties
    if zeros:
        mask = rng.random(a.shape) < zeros
        a[mask] = np.where(rng.random(int(mask.sum())) < 0.5, 0.0, -0.0).astype(np.float32)
    bits = WL.to_bf16_bits(a)
    # every fourth draw each: the one-threshold variant, thresholds per token
    quantile = {1: "abs", 2: "token"}.get(i % 4, "signed")
    ctx.status.zero_()
    ctx.set_quantile_mode({"abs": lib.FP4_QUANTILE_ABS, "token": lib.FP4_QUANTILE_TOKEN,
                           "signed": lib.FP4_QUANTILE_SIGNED}[quantile])
    try:
        q = lib.fp4_quantize(ctx, _dev(bits), 0, alpha=alpha)
        torch.cuda.synchronize()
    finally:
        ctx.set_quantile_mode(lib.FP4_QUANTILE_SIGNED)
    assert ctx.read_status() == 0
    ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha, quantile=quantile)
    if quantile == "token":
        _check_token_mode(q, ref)
        return
    _check_sparse(q, ref)
    _check_dense(q, ref)


@pytest.mark.parametrize("seed", [7, 8] + [100 + SEED_SHIFT + j for j in range(int(os.environ.get("FP4_RANDOM_HOST_SEQUENCES", "0")))])
def test_random_sequence_of_host_steps(lib, seed):
    """Twenty host-buffer steps of random shapes issued back to back on a workspace that fits the
    pipelined layout for some of them only: every output equals the device-resident path's, bit for
    bit, whatever mix of pipelined and single-stream calls the sequence produces."""
    from test_gpu_step_host import ALPHA, _device_reference, _inputs
    rng = np.random.default_rng(seed)
    shapes = [(128, 128, 128), (256, 256, 384), (128, 512, 128), (384, 128, 640), (512, 384, 256)]
    seq = [shapes[int(rng.integers(0, len(shapes)))] for _ in range(20)]
    needs = sorted(int(lib.load_library().fp4_step_host_workspace_bytes(M, K, N, ALPHA)) for M, K, N in shapes)
    ctx = lib.Context(0, needs[len(needs) // 2] if seed % 2 else needs[-1])
    cases, outs = [], []
    for i, (M, K, N) in enumerate(seq):
        hA, hW, hG = _inputs(200 + i, M, K, N)
        hY = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        hdA = torch.empty((M, K), dtype=torch.bfloat16).pin_memory()
        hdW = torch.empty((K, N), dtype=torch.bfloat16).pin_memory()
        try:
            lib.fp4_linear_step_host(ctx, hA, hW, hG, ALPHA, hY, hdA, hdW, read_status=False)
        except Exception:
            continue                                   # a shape the smaller workspace cannot hold at all
        cases.append(((M, K, N), (hA, hW, hG)))
        outs.append((hY, hdA, hdW))
    torch.cuda.synchronize()
    assert len(cases) >= 5
    for ((M, K, N), (hA, hW, hG)), got in zip(cases, outs):
        want = _device_reference(lib, M, K, N, hA, hW, hG)
        for g, w, name in zip(got, want, ("Y", "dA", "dW")):
            assert torch.equal(g.view(torch.int16), w.view(torch.int16)), (M, K, N, name)
    ctx.close()
