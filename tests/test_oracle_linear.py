"""Pins of the oracle's GEMM, DGE and forward/backward composition."""
from fractions import Fraction

import numpy as np
import pytest
from scipy import integrate

from conftest import golden_lines
from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

GRID = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


# ------------------------------------------------------------------ GEMM ---- #
def test_gemm_codes_brute_force_fractions():
    rng = np.random.default_rng(0)
    ca = rng.integers(0, 16, (5, 12), dtype=np.uint8)
    cb = rng.integers(0, 16, (7, 12), dtype=np.uint8)
    table = {}
    for ln in golden_lines("e2m1_table.txt"):
        code, val = ln.split()
        table[int(code, 2)] = Fraction(val)
    acc = O.gemm_codes(ca, cb)
    for i in range(5):
        for j in range(7):
            s = sum(table[int(ca[i, c])] * table[int(cb[j, c])] for c in range(12))
            assert Fraction(float(acc[i, j])) == s


def test_accumulators_are_exact_quarter_integers_at_long_k():
    rng = np.random.default_rng(1)
    ca = rng.integers(0, 16, (3, 16384), dtype=np.uint8)
    cb = rng.integers(0, 16, (4, 16384), dtype=np.uint8)
    acc = O.gemm_codes(ca, cb)
    ia = (2 * O.e2m1_decode(ca)).astype(np.int64)
    ib = (2 * O.e2m1_decode(cb)).astype(np.int64)
    np.testing.assert_array_equal((acc * 4).astype(np.int64), ia @ ib.T)
    assert np.abs(acc * 4).max() < 2 ** 24            # also exact as float32


def test_descale_after_gemm_equals_gemm_of_descaled_values():
    """Appendix C.2: feeding W_q^scaled to the GEMM and de-scaling afterwards is the
    same as multiplying by the de-scaled W_q."""
    a_bits, w_bits, _ = WL.small_case(8, 32, 16, seed=3)
    f = O.linear_fwd(a_bits, w_bits, 1.0)
    aq = O.e2m1_decode(f.qa.codes) * f.qa.descale.astype(np.float64)[:, None]
    wq = O.e2m1_decode(f.qw.codes) * f.qw.descale.astype(np.float64)[None, :]
    np.testing.assert_allclose(f.y, aq @ wq, rtol=1e-13, atol=0)


# ------------------------------------------------------------------- DGE ---- #
def test_dge_spot_values():
    for ln in golden_lines("dge_spot_values.txt"):
        x, want = (float(t) for t in ln.split())
        assert O.dge_fprime(x) == pytest.approx(want, rel=2e-5), ln


def test_dge_f_fixes_grid_points_and_midpoints():
    g = np.array(GRID)
    np.testing.assert_allclose(O.dge_f(g), g, atol=1e-15)
    np.testing.assert_allclose(O.dge_f(-g), -g, atol=1e-15)
    mids = (g[:-1] + g[1:]) / 2
    np.testing.assert_allclose(O.dge_f(mids), mids, atol=1e-15)


def test_dge_first_interval_matches_eq7_literally():
    """Eq. 7 typed out for the first positive interval [0, 0.5] (Fig. 3a), delta = 0.5, k = 5."""
    d, k = 0.5, 5.0
    for x in np.linspace(0.001, 0.499, 97):
        t = 2 * x / d - 1
        want = d / 2 * (1 + np.sign(t) * abs(t) ** (1 / k))
        assert O.dge_f(x) == pytest.approx(want, rel=1e-14)
        if abs(t) > 0.05:
            assert O.dge_fprime(x) == pytest.approx(1 / k * abs(t) ** (1 / k - 1), rel=1e-14)


@pytest.mark.parametrize("lo,hi", list(zip(GRID[:-1], GRID[1:])))
def test_integral_of_uncapped_derivative_is_interval_width(lo, hi):
    mid = (lo + hi) / 2
    val = sum(integrate.quad(lambda x: float(O.dge_fprime(x, clip=np.inf)), a, b, limit=200)[0]
              for a, b in ((lo, mid), (mid, hi)))
    assert val == pytest.approx(hi - lo, rel=1e-6)


def test_derivative_matches_central_difference_of_f():
    xs = np.array([0.05, 0.13, 0.4, 0.62, 1.1, 1.9, 2.2, 2.8, 3.3, 4.4, 5.7, -0.4, -2.2, -5.7])
    h = 1e-6
    num = (O.dge_f(xs + h) - O.dge_f(xs - h)) / (2 * h)
    np.testing.assert_allclose(O.dge_fprime(xs), num, rtol=1e-5)


def test_cap_threshold_and_mean():
    u0 = 15.0 ** -1.25                                  # (3k)^(-k/(k-1)) for k = 5
    delta = 0.5
    x_in = delta / 2 * (1 + 0.99 * u0)
    x_out = delta / 2 * (1 + 1.01 * u0)
    assert O.dge_fprime(x_in) == 3.0
    assert O.dge_fprime(x_out) < 3.0
    # mean over one interval of the capped derivative: 1 - (u0^(1/5) - 3 u0)
    xs = (np.arange(2_000_000) + 0.5) / 2_000_000 * delta
    assert O.dge_fprime(xs).mean() == pytest.approx(1 - (u0 ** 0.2 - 3 * u0), rel=1e-5)


def test_dge_is_even_and_extends_past_6():
    xs = np.linspace(0.01, 6.5, 333)
    np.testing.assert_array_equal(O.dge_fprime(xs), O.dge_fprime(-xs))
    assert O.dge_fprime(6.0 * (1 + 2.0 ** -23)) == pytest.approx(0.2, rel=1e-5)


# --------------------------------------------------------------- linear ---- #
def _dense_reference_fwd(a, w, alpha):
    """Forward written out per element with Python floats on a tiny case."""
    M, K = a.shape
    N = w.shape[1]
    lo, hi, _ = O.quantile_thresholds(a, alpha)
    y = np.zeros((M, N))
    ac = np.clip(a, lo, hi)
    for m in range(M):
        ga = np.float32(6) / np.float32(np.abs(ac[m]).max())
        da = np.float32(np.abs(ac[m]).max()) / np.float32(6)
        for n in range(N):
            gw = np.float32(6) / np.float32(np.abs(w[:, n]).max())
            dw = np.float32(np.abs(w[:, n]).max()) / np.float32(6)
            s = 0.0
            comp = 0.0
            for k in range(K):
                qa = O.e2m1_decode(O.lut_quantize(np.array([np.float32(ac[m, k]) * ga], dtype=np.float32)))[0]
                qw = O.e2m1_decode(O.lut_quantize(np.array([np.float32(w[k, n]) * gw], dtype=np.float32)))[0]
                s += qa * qw
                comp += (a[m, k] - ac[m, k]) * w[k, n]
            y[m, n] = s * float(da) * float(dw) + comp
    return y


def test_forward_brute_force_tiny():
    a_bits, w_bits, _ = WL.small_case(4, 16, 6, seed=1, alpha_outliers=2)
    f = O.linear_fwd(a_bits, w_bits, 0.9)
    ref = _dense_reference_fwd(O.bf16_bits_to_f64(a_bits), O.bf16_bits_to_f64(w_bits), 0.9)
    np.testing.assert_allclose(f.y, ref, rtol=1e-12, atol=1e-300)
    assert f.qa.csr[0][-1] > 0


def test_compensation_restores_clamped_part_exactly():
    """Y - Y_fp4 equals (A - A_c) W: with the residual, only quantisation error is left."""
    a_bits, w_bits, _ = WL.small_case(16, 64, 32, seed=2)
    f = O.linear_fwd(a_bits, w_bits, 0.97)
    a = O.bf16_bits_to_f64(a_bits)
    w = O.bf16_bits_to_f64(w_bits)
    a_c, r = O.occ_split(a, f.qa.lo, f.qa.hi)
    np.testing.assert_allclose(f.y_comp, (a - a_c) @ w, rtol=1e-13)
    # the quantised branch approximates A_c W, the whole approximates A W better than without compensation
    err_with = np.linalg.norm(f.y - a @ w)
    err_without = np.linalg.norm(f.y_fp4 - a @ w)
    assert err_with < err_without


def test_wgrad_scale_cancellation():
    """Last equation of Appendix C.2: (dL/dW_q (.) 1/sf (.) Q'(W_scaled)) (.) sf == dL/dW_q (.) Q'."""
    a_bits, w_bits, dy_bits = WL.small_case(16, 32, 32, seed=4)
    f = O.linear_fwd(a_bits, w_bits, 0.97)
    b = O.linear_bwd(dy_bits, w_bits, f)
    sf = f.qw.gamma.astype(np.float64)[None, :]
    long_way = ((b.s * (1.0 / sf)) * b.dge) * sf
    np.testing.assert_allclose(b.dw, long_way, rtol=1e-14)
    ste = O.linear_bwd(dy_bits, w_bits, f, dge_on=False)
    np.testing.assert_array_equal(ste.dw, ste.s)
    np.testing.assert_array_equal(ste.da, b.da)


def test_dge_factor_uses_forward_scaled_weights():
    a_bits, w_bits, dy_bits = WL.small_case(8, 32, 16, seed=5)
    f = O.linear_fwd(a_bits, w_bits, 1.0)
    b = O.linear_bwd(dy_bits, w_bits, f)
    w = O.bf16_bits_to_f64(w_bits)
    for k, n in [(0, 0), (3, 7), (31, 15)]:
        gamma = np.float32(6) / np.float32(np.abs(w[:, n]).max())
        ws = float(np.float32(w[k, n]) * gamma)
        assert b.dge[k, n] == O.dge_fprime(ws)


def test_backward_folded_scales_identity_without_quantising_dy():
    """sum_n dY[m,n] d_W[n] val(codeW[k,n]) == (dY W_q^T)[m,k]; and likewise for wgrad.
    Checked in double with dY left unquantised, which isolates the folding of the scales."""
    a_bits, w_bits, dy_bits = WL.small_case(8, 32, 16, seed=6)
    f = O.linear_fwd(a_bits, w_bits, 1.0)
    dy = O.bf16_bits_to_f64(dy_bits)
    d_w = f.qw.descale.astype(np.float64)
    d_a = f.qa.descale.astype(np.float64)
    wq = O.e2m1_decode(f.qw.codes) * d_w[None, :]
    aq = O.e2m1_decode(f.qa.codes) * d_a[:, None]
    np.testing.assert_allclose((dy * d_w[None, :]) @ O.e2m1_decode(f.qw.codes).T, dy @ wq.T, rtol=1e-12)
    np.testing.assert_allclose(O.e2m1_decode(f.qa.codes).T @ (dy * d_a[:, None]), aq.T @ dy, rtol=1e-12)


def test_backward_brute_force_tiny():
    a_bits, w_bits, dy_bits = WL.small_case(4, 8, 6, seed=7, alpha_outliers=1)
    f = O.linear_fwd(a_bits, w_bits, 0.9)
    b = O.linear_bwd(dy_bits, w_bits, f)
    dy = O.bf16_bits_to_f64(dy_bits)
    M, K, N = 4, 8, 6
    va, vw = O.e2m1_decode(f.qa.codes), O.e2m1_decode(f.qw.codes)
    d_a, d_w = f.qa.descale, f.qw.descale
    # dgrad
    for m in range(M):
        g = np.array([np.float32(np.float32(dy[m, n]) * d_w[n]) for n in range(N)], dtype=np.float32)
        amax = np.abs(g).max()
        q = O.e2m1_decode(O.lut_quantize((g * (np.float32(6) / amax)).astype(np.float32)))
        for k in range(K):
            want = float(amax / np.float32(6)) * sum(q[n] * vw[k, n] for n in range(N))
            assert b.da[m, k] == pytest.approx(want, rel=1e-13, abs=1e-300)
    # wgrad
    for n in range(N):
        g = np.array([np.float32(np.float32(dy[m, n]) * d_a[m]) for m in range(M)], dtype=np.float32)
        amax = np.abs(g).max()
        q = O.e2m1_decode(O.lut_quantize((g * (np.float32(6) / amax)).astype(np.float32)))
        for k in range(K):
            s = float(amax / np.float32(6)) * sum(va[m, k] * q[m] for m in range(M))
            s += sum(f.qa.residual[m, k] * dy[m, n] for m in range(M))
            assert b.s[k, n] == pytest.approx(s, rel=1e-12, abs=1e-300)
            assert b.dw[k, n] == pytest.approx(s * float(O.dge_fprime(float(f.qw.scaled[k, n]))), rel=1e-12, abs=1e-300)


def test_fp4_linear_tracks_exact_product():
    """Sanity on config 0: the whole estimator stays close to the unquantised product."""
    cfg = WL.CONFIGS[0]
    a_bits = WL.activations(cfg, 1024)
    w_bits = WL.weights(cfg, 1024, 1024)
    f = O.linear_fwd(a_bits, w_bits, 0.99)
    exact = O.bf16_bits_to_f64(a_bits) @ O.bf16_bits_to_f64(w_bits)
    cos = (f.y * exact).sum() / np.linalg.norm(f.y) / np.linalg.norm(exact)
    assert cos > 0.98
    assert f.qa.n_tail == 2621
