"""Pins of the oracle's E2M1 grid, look-up quantiser and absmax scaling.

Each check compares the oracle with something that is not the oracle: the paper's
printed table and chain (text fixtures), a nearest-value search, or an invariant.
"""
from fractions import Fraction

import numpy as np
import pytest

from conftest import golden_lines
from oracle import fp4_oracle as O


def test_decode_matches_table4():
    for ln in golden_lines("e2m1_table.txt"):
        code, val = ln.split()
        assert O.e2m1_decode(np.uint8(int(code, 2))) == float(val), ln


def test_grid_has_15_values_max_6():
    vals = O.e2m1_decode(np.arange(16, dtype=np.uint8))
    assert len(set(vals.tolist())) == 15          # +0 and -0 coincide
    assert vals.max() == 6.0 and vals.min() == -6.0


def _chain():
    rows = golden_lines("lut_chain.txt")
    th = [(float(a), float(b)) for a, b in (r.split() for r in rows[:-1])]
    return th, float(rows[-1].split()[1])


def _chain_eval(v, th, last):
    for t, r in th:
        if v < t:
            return r
    return last


def test_thresholds_are_midpoints_of_adjacent_grid_values():
    th, last = _chain()
    results = [r for _, r in th] + [last]
    assert results == sorted(set(O.e2m1_decode(np.arange(16, dtype=np.uint8)).tolist()))
    for (t, r), nxt in zip(th, results[1:]):
        assert Fraction(t) == (Fraction(r) + Fraction(nxt)) / 2


def test_lut_constants_match_printed_chain():
    th, last = _chain()
    assert [t for t, _ in th] == O.LUT_THRESHOLDS.tolist()
    assert [r for _, r in th] + [last] == O.LUT_VALUES.tolist()


def _all_bf16_finite():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    v = O.bf16_bits_to_f64(bits)
    return v[np.isfinite(v)]


def test_Q_is_nearest_grid_value_ties_to_larger_all_bf16():
    """Brute force over every finite BF16 number: Q = nearest grid value, ties -> larger."""
    v = _all_bf16_finite()
    grid = np.array(sorted(set(O.LUT_VALUES.tolist())))
    # beyond +-8 the nearest grid value is +-6; clipping keeps the distances exact in float64
    dist = np.abs(np.clip(v, -8.0, 8.0)[:, None] - grid[None, :])
    # nearest; among equally near, the larger value (argmin over the reversed grid)
    nearest = grid[::-1][np.argmin(dist[:, ::-1], axis=1)]
    got = O.e2m1_decode(O.lut_quantize(v.astype(np.float32)))
    np.testing.assert_array_equal(got, nearest)


def test_Q_around_every_threshold_fp32_neighbours():
    th, last = _chain()
    for t, _ in th:
        t32 = np.float32(t)
        for v in (np.nextafter(t32, np.float32(-np.inf)), t32, np.nextafter(t32, np.float32(np.inf))):
            got = float(O.e2m1_decode(O.lut_quantize(np.array([v], dtype=np.float32)))[0])
            assert got == _chain_eval(float(v), th, last), (t, v)


def test_tie_vectors():
    ties = {0.25: 0.5, 0.75: 1.0, 1.25: 1.5, 1.75: 2.0, 2.5: 3.0, 3.5: 4.0, 5.0: 6.0,
            -0.25: 0.0, -0.75: -0.5, -1.25: -1.0, -1.75: -1.5, -2.5: -2.0, -3.5: -3.0, -5.0: -4.0}
    v = np.array(list(ties), dtype=np.float32)
    np.testing.assert_array_equal(O.e2m1_decode(O.lut_quantize(v)), np.array(list(ties.values())))


def test_never_emits_negative_zero_code():
    v = np.array([-0.25, -0.2, -0.0, -1e-30, 0.0, 0.2], dtype=np.float32)
    assert (O.lut_quantize(v) == 0).all()
    codes = O.lut_quantize(np.linspace(-7, 7, 20001).astype(np.float32))
    assert not (codes == 8).any()


def test_nibble_packing_order():
    c = np.array([[0x2, 0xB, 0x5, 0x7]], dtype=np.uint8)
    np.testing.assert_array_equal(O.pack_nibbles(c), np.array([[0xB2, 0x75]], dtype=np.uint8))
    np.testing.assert_array_equal(O.unpack_nibbles(O.pack_nibbles(c)), c)


@pytest.mark.parametrize("axis", [0, 1])
def test_absmax_element_encodes_pm6_and_scaled_range(axis):
    rng = np.random.default_rng(3)
    x = O.bf16_bits_to_f64((rng.standard_normal((37, 64)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16))
    q = O.absmax_quantize(x, axis)
    vals = O.e2m1_decode(q.codes)
    assert np.abs(q.scaled).max() <= 6.0 * (1 + 2.0 ** -23)
    red = 1 - axis
    amax_pos = np.argmax(np.abs(x), axis=red)
    for i, j in enumerate(amax_pos):
        r, c = (i, j) if axis == 0 else (j, i)
        assert abs(vals[r, c]) == 6.0
        assert q.amax[i] == abs(x[r, c])
    # gamma is Eq. 1 rounded once to float32; d its reciprocal counterpart
    for i in range(q.amax.size):
        assert float(q.gamma[i]) == float(np.float32(Fraction(6) / Fraction(float(q.amax[i]))))
        assert float(q.descale[i]) == float(np.float32(Fraction(float(q.amax[i])) / 6))


def test_scaled_value_is_single_rounding_of_exact_product():
    rng = np.random.default_rng(5)
    bits = (rng.standard_normal((4, 32)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    x = O.bf16_bits_to_f64(bits)
    q = O.absmax_quantize(x, 0)
    for r in range(4):
        g = Fraction(float(q.gamma[r]))
        for c in range(32):
            exact = Fraction(float(x[r, c])) * g
            assert float(q.scaled[r, c]) == float(np.float32(exact))


def test_zero_vector():
    x = np.zeros((2, 8))
    x[1, 3] = 2.0
    q = O.absmax_quantize(x, 0)
    assert q.amax[0] == 0 and q.gamma[0] == 0 and q.descale[0] == 0
    assert (q.codes[0] == 0).all()
    assert O.e2m1_decode(q.codes[1, 3]) == 6.0


def test_prescale_is_applied_first_with_one_rounding():
    x = np.array([[1.0, 3.0, -0.5, 0.25]])
    p = np.array([0.1, 0.3, 0.7, 1.9], dtype=np.float32)
    q = O.absmax_quantize(x, 0, prescale=p)
    xs = (x[0] * p.astype(np.float64)).astype(np.float32)
    assert q.amax[0] == np.abs(xs).max()
    assert abs(O.e2m1_decode(q.codes)[0, np.argmax(np.abs(xs))]) == 6.0


def test_bf16_rounding_helper():
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6 (even)
    assert O.f64_to_bf16_f64(1 + 2.0 ** -8) == 1.0
    assert O.f64_to_bf16_f64(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6
    assert O.f64_to_bf16_f64(1 + 2.0 ** -8 + 2.0 ** -30) == 1 + 2.0 ** -7
    v = _all_bf16_finite()
    np.testing.assert_array_equal(O.f64_to_bf16_f64(v), v)
