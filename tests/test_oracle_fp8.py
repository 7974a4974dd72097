"""Pins of the oracle's E4M3 operands (the W4A8 / W8A4 settings of Section 4.3 and the FP8 reading
of the backward's dY): the format, the rounding, the scaling, and the mixed-format layer against
brute force with exact rationals."""
from fractions import Fraction

import numpy as np
import pytest

from conftest import golden_lines
from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

FINITE = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


def test_decode_matches_the_format_definition():
    for ln in golden_lines("e4m3_spot_values.txt"):
        code, val = ln.split()
        assert O.e4m3_decode(np.array([int(code, 16)], dtype=np.uint8))[0] == float(val)
    v = O.e4m3_decode(np.arange(256, dtype=np.uint8))
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF]) and np.isfinite(np.delete(v, [0x7F, 0xFF])).all()
    pos = v[:0x7F]
    assert (np.diff(pos) > 0).all()                        # codes order like their values
    np.testing.assert_array_equal(v[0x80:0xFF], -pos)       # sign-magnitude
    assert pos.max() == 448.0 and pos[1] == 2.0 ** -9
    # every value is (integer) * 2^-9 with an integer below 2^18: what makes mixed sums exact
    assert (pos * 512 == np.rint(pos * 512)).all()


def test_quantize_is_nearest_with_ties_to_even_and_saturates():
    grid = O.e4m3_decode(FINITE[FINITE < 0x80])            # non-negative values, ascending
    rng = np.random.default_rng(0)
    mids = (grid[:-1] + grid[1:]) / 2                       # every tie of the format
    probes = np.concatenate([grid, mids, np.nextafter(mids.astype(np.float32), np.float32(np.inf)).astype(np.float64),
                             np.nextafter(mids.astype(np.float32), np.float32(0)).astype(np.float64),
                             rng.uniform(0, 448, 20000), rng.uniform(0, 0.05, 5000)])
    probes = probes.astype(np.float32)
    for sign in (1.0, -1.0):
        v = (sign * probes).astype(np.float32)
        codes = O.e4m3_quantize(v)
        got = np.abs(O.e4m3_decode(codes))
        a = np.abs(v.astype(np.float64))
        dist = np.abs(a[:, None] - grid[None, :])
        best = dist.min(axis=1)
        assert (np.abs(got - a) == best).all()              # a nearest value
        tie = (dist == best[:, None]).sum(axis=1) == 2
        assert ((codes[tie] & 1) == 0).all()                # of two nearest, the even mantissa
        assert ((codes >> 7) == (1 if sign < 0 else 0)).all()   # the input's sign, zero included
    big = np.array([449, 464, 470, 480, 1e6, 3e38], dtype=np.float32)
    np.testing.assert_array_equal(O.e4m3_quantize(big), np.full(6, 0x7E, dtype=np.uint8))
    np.testing.assert_array_equal(O.e4m3_quantize(-big), np.full(6, 0xFE, dtype=np.uint8))


def test_quantize_is_the_identity_on_the_grid():
    v = O.e4m3_decode(FINITE).astype(np.float32)
    np.testing.assert_array_equal(O.e4m3_quantize(v), FINITE)


@pytest.mark.parametrize("axis", [0, 1])
def test_absmax_scaling_to_448(axis):
    rng = np.random.default_rng(3 + axis)
    x = O.bf16_bits_to_f64(WL.to_bf16_bits(rng.standard_normal((24, 40)).astype(np.float32)))
    q = O.absmax_quantize(x, axis, fmt="e4m3")
    vals = q.values()
    where = np.abs(x) == np.abs(x).max(axis=1 - axis, keepdims=True)
    assert (np.abs(vals[where]) == 448.0).all()             # the absmax element sits on MAX
    assert np.abs(q.scaled).max() <= 448.0 * (1 + 2.0 ** -22)
    # de-quantised values stay within half a grid step of the scaled input
    step = np.where(np.abs(vals) >= 2.0 ** -6, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(vals), 1e-30))) - 3), 2.0 ** -9)
    assert (np.abs(vals - q.scaled.astype(np.float64)) <= step / 2 * (1 + 1e-12)).all()
    g, d = O.absmax_scales(q.amax, 448.0)
    np.testing.assert_array_equal(g, (np.float32(448) / q.amax).astype(np.float32))
    np.testing.assert_array_equal(d, (q.amax / np.float32(448)).astype(np.float32))


def _frac_matrix(a):
    return [[Fraction(float(v)) for v in row] for row in a]


@pytest.mark.parametrize("fmt_a,fmt_w,fmt_dy", [("e4m3", "e2m1", "e2m1"), ("e2m1", "e4m3", "e2m1"),
                                                ("e2m1", "e2m1", "e4m3"), ("e4m3", "e2m1", "e4m3")])
def test_mixed_layer_against_exact_rationals(fmt_a, fmt_w, fmt_dy):
    """Forward and backward of a tiny layer recomputed from the stored codes and scales with
    exact rational arithmetic, element by element."""
    M, K, N = 4, 6, 5
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=11, alpha_outliers=1)
    alpha = 0.9 if fmt_a == "e2m1" else 1.0
    f = O.linear_fwd(a_bits, w_bits, alpha, fmt_a=fmt_a, fmt_w=fmt_w)
    b = O.linear_bwd(dy_bits, w_bits, f, fmt_dy=fmt_dy)
    va, vw = _frac_matrix(f.qa.values()), _frac_matrix(f.qw.values())
    da_, dw_ = [Fraction(float(x)) for x in f.qa.descale], [Fraction(float(x)) for x in f.qw.descale]
    res, w = _frac_matrix(f.qa.residual), _frac_matrix(O.bf16_bits_to_f64(w_bits))
    dy = _frac_matrix(O.bf16_bits_to_f64(dy_bits))
    for m in range(M):
        for n in range(N):
            y = sum(va[m][k] * vw[k][n] for k in range(K)) * da_[m] * dw_[n] + sum(res[m][k] * w[k][n] for k in range(K))
            assert abs(Fraction(float(f.y[m, n])) - y) <= abs(y) * Fraction(1, 10 ** 12) + Fraction(1, 10 ** 300)
    g1, g2 = _frac_matrix(b.qg_dgrad.values()), _frac_matrix(b.qg_wgrad.values())
    d1, d2 = [Fraction(float(x)) for x in b.qg_dgrad.descale], [Fraction(float(x)) for x in b.qg_wgrad.descale]
    for m in range(M):
        for k in range(K):
            want = sum(g1[m][n] * vw[k][n] for n in range(N)) * d1[m]
            assert abs(Fraction(float(b.da[m, k])) - want) <= abs(want) * Fraction(1, 10 ** 12) + Fraction(1, 10 ** 300)
    for k in range(K):
        for n in range(N):
            want = sum(va[m][k] * g2[m][n] for m in range(M)) * d2[n] + sum(res[m][k] * dy[m][n] for m in range(M))
            assert abs(Fraction(float(b.s[k, n])) - want) <= abs(want) * Fraction(1, 10 ** 12) + Fraction(1, 10 ** 300)
    if fmt_w != "e2m1":
        assert (b.dge == 1.0).all()                         # straight-through for an 8-bit weight
    else:
        np.testing.assert_array_equal(b.dge, O.dge_fprime(f.qw.scaled.astype(np.float64)))
    assert b.qg_dgrad.fmt == fmt_dy and b.qg_wgrad.fmt == fmt_dy and f.qa.fmt == fmt_a and f.qw.fmt == fmt_w


def test_fp8_operands_reduce_to_the_plain_product_on_representable_inputs():
    """Tensors whose scaled entries lie on the E4M3 grid are quantised without error, so the
    layer must return the plain matrix product (a case with a textbook answer)."""
    rng = np.random.default_rng(5)
    M, K, N = 8, 16, 8
    grid = O.e4m3_decode(FINITE[(FINITE < 0x7F) & (FINITE >= 0x20)])      # normal values, >= 2^-3
    a = rng.choice(grid, (M, K)) * rng.choice([-1.0, 1.0], (M, K)) / 256.0
    w = rng.choice(grid, (K, N)) * rng.choice([-1.0, 1.0], (K, N)) / 256.0
    a[:, 0] = 448.0 / 256.0                                  # every row's absmax: gamma = 256 exactly
    w[0, :] = 448.0 / 256.0                                  # every column's absmax
    a_bits, w_bits = WL.to_bf16_bits(a.astype(np.float32)), WL.to_bf16_bits(w.astype(np.float32))
    np.testing.assert_array_equal(O.bf16_bits_to_f64(a_bits), a)          # E4M3 values are BF16 values
    f = O.linear_fwd(a_bits, w_bits, 1.0, fmt_a="e4m3", fmt_w="e4m3")
    np.testing.assert_array_equal(f.qa.values() / 256.0, a)
    np.testing.assert_allclose(f.y, a @ w, rtol=1e-15, atol=0)


def test_activation_clamping_is_refused_for_fp8_activations():
    a_bits, w_bits, _ = WL.small_case(4, 8, 4, seed=1)
    with pytest.raises(ValueError):
        O.linear_fwd(a_bits, w_bits, 0.99, fmt_a="e4m3")


# ---------------------------------------------------------------------------------------------
# E5M2, the other FP8 variant Section 2 names
# ---------------------------------------------------------------------------------------------
FINITE_E5M2 = np.array([c for c in range(256) if ((c >> 2) & 0x1F) != 0x1F], dtype=np.uint8)


def test_e5m2_decode_matches_the_format_definition():
    for ln in golden_lines("e5m2_spot_values.txt"):
        code, val = ln.split()
        assert O.e5m2_decode(np.array([int(code, 16)], dtype=np.uint8))[0] == float(val)
    v = O.e5m2_decode(np.arange(256, dtype=np.uint8))
    assert v[0x7C] == np.inf and v[0xFC] == -np.inf and np.isnan(v[[0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF]]).all()
    pos = v[:0x7C]
    assert (np.diff(pos) > 0).all()                        # codes order like their values
    np.testing.assert_array_equal(v[0x80:0xFC], -pos)       # sign-magnitude
    assert pos.max() == 57344.0 and pos[1] == 2.0 ** -16
    assert (pos * 65536 == np.rint(pos * 65536)).all()     # every value is an integer multiple of 2^-16


def test_e5m2_quantize_is_nearest_with_ties_to_even_and_saturates():
    grid = O.e5m2_decode(FINITE_E5M2[FINITE_E5M2 < 0x80])  # non-negative values, ascending
    rng = np.random.default_rng(1)
    mids = (grid[:-1] + grid[1:]) / 2                       # every tie of the format
    probes = np.concatenate([grid, mids, np.nextafter(mids.astype(np.float32), np.float32(np.inf)).astype(np.float64),
                             np.nextafter(mids.astype(np.float32), np.float32(0)).astype(np.float64),
                             rng.uniform(0, 57344, 20000), rng.uniform(0, 0.001, 5000)])
    probes = probes.astype(np.float32)
    for sign in (1.0, -1.0):
        v = (sign * probes).astype(np.float32)
        codes = O.e5m2_quantize(v)
        got = np.abs(O.e5m2_decode(codes))
        a = np.abs(v.astype(np.float64))
        dist = np.abs(a[:, None] - grid[None, :])
        best = dist.min(axis=1)
        assert (np.abs(got - a) == best).all()              # a nearest value
        tie = (dist == best[:, None]).sum(axis=1) == 2
        assert ((codes[tie] & 1) == 0).all()                # of two nearest, the even mantissa
        assert ((codes >> 7) == (1 if sign < 0 else 0)).all()   # the input's sign, zero included
    big = np.array([57345, 61440, 65535, 65536, 1e6, 3e38], dtype=np.float32)
    np.testing.assert_array_equal(O.e5m2_quantize(big), np.full(6, 0x7B, dtype=np.uint8))    # never infinity
    np.testing.assert_array_equal(O.e5m2_quantize(-big), np.full(6, 0xFB, dtype=np.uint8))


def test_e5m2_quantize_is_the_identity_on_the_grid():
    v = O.e5m2_decode(FINITE_E5M2).astype(np.float32)
    np.testing.assert_array_equal(O.e5m2_quantize(v), FINITE_E5M2)


@pytest.mark.parametrize("axis", [0, 1])
def test_absmax_scaling_to_57344(axis):
    rng = np.random.default_rng(13 + axis)
    x = O.bf16_bits_to_f64(WL.to_bf16_bits(rng.standard_normal((24, 40)).astype(np.float32)))
    q = O.absmax_quantize(x, axis, fmt="e5m2")
    vals = q.values()
    where = np.abs(x) == np.abs(x).max(axis=1 - axis, keepdims=True)
    assert (np.abs(vals[where]) == 57344.0).all()           # the absmax element sits on MAX
    assert np.isfinite(vals).all()
    step = np.where(np.abs(vals) >= 2.0 ** -14, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(vals), 1e-30))) - 2), 2.0 ** -16)
    assert (np.abs(vals - q.scaled.astype(np.float64)) <= step / 2 * (1 + 1e-12)).all()
    g, d = O.absmax_scales(q.amax, 57344.0)
    np.testing.assert_array_equal(g, (np.float32(57344) / q.amax).astype(np.float32))
    np.testing.assert_array_equal(d, (q.amax / np.float32(57344)).astype(np.float32))


@pytest.mark.parametrize("fmt_a,fmt_w,fmt_dy", [("e2m1", "e2m1", "e5m2"), ("e2m1", "e4m3", "e5m2"),
                                                ("e5m2", "e2m1", "e2m1"), ("e4m3", "e5m2", "e5m2")])
def test_mixed_layer_with_e5m2_against_exact_rationals(fmt_a, fmt_w, fmt_dy):
    test_mixed_layer_against_exact_rationals(fmt_a, fmt_w, fmt_dy)
