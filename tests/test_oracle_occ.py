"""Pins of the oracle's outlier clamping and compensation (Section 3.2)."""
import numpy as np
import pytest

from conftest import golden_lines
from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL


def _bf16_normal(rng, shape):
    return O.bf16_bits_to_f64(WL.to_bf16_bits(rng.standard_normal(shape).astype(np.float32)))


def _load_example():
    lines = golden_lines("occ_worked_example.txt")
    it = iter(lines)
    ex = {}
    for ln in it:
        tok = ln.split()
        if tok[0] == "A":
            r, c = int(tok[1]), int(tok[2])
            ex["A"] = np.array([[float(x) for x in next(it).split()] for _ in range(r)])
        elif tok[0] in ("alpha", "lo", "hi", "gamma"):
            ex[tok[0]] = float(tok[1])
        elif tok[0] == "n_tail":
            ex["n_tail"] = int(tok[1])
        elif tok[0] == "residual":
            ex["residual"] = [tuple(float(x) for x in next(it).split()) for _ in range(int(tok[1]))]
        elif tok[0] == "amax":
            ex["amax"] = [float(x) for x in tok[1:]]
        elif tok[0] == "quantized":
            ex["quantized"] = np.array([[float(x) for x in next(it).split()] for _ in range(2)])
        elif tok[0] == "packed":
            ex["packed"] = np.array([[int(x, 16) for x in next(it).split()] for _ in range(2)], dtype=np.uint8)
    return ex


def test_worked_example():
    ex = _load_example()
    q = O.occ_quantize(ex["A"], ex["alpha"])
    assert (q.n_tail, q.lo, q.hi) == (ex["n_tail"], ex["lo"], ex["hi"])
    rowptr, col, val = q.csr
    got = [(float(r), float(c), float(v)) for r in range(2)
           for c, v in zip(col[rowptr[r]:rowptr[r + 1]], val[rowptr[r]:rowptr[r + 1]])]
    assert got == ex["residual"]
    assert q.amax.tolist() == ex["amax"]
    assert q.gamma.tolist() == [ex["gamma"]] * 2
    np.testing.assert_array_equal(O.e2m1_decode(q.codes), ex["quantized"])
    np.testing.assert_array_equal(q.packed(), ex["packed"])
    # CSC holds the same entries ordered by column, then row
    colptr, row, cval = q.csc
    got_c = sorted((float(r), float(c), float(v)) for c in range(8)
                   for r, v in zip(row[colptr[c]:colptr[c + 1]], cval[colptr[c]:colptr[c + 1]]))
    assert got_c == sorted(ex["residual"])


@pytest.mark.parametrize("n,alpha", [(101, 0.9), (64, 0.875), (1000, 0.99), (37, 0.97)])
def test_thresholds_by_counting(n, alpha):
    """Definition by counts instead of by sorting: lo is the value with
    #(a < lo) <= n_tail < #(a <= lo); mirrored for hi."""
    rng = np.random.default_rng(n)
    a = _bf16_normal(rng, (1, n))
    a[0, : n // 5] = a[0, n // 5: 2 * (n // 5)]          # force duplicates
    lo, hi, t = O.quantile_thresholds(a, alpha)
    assert t == int((1 - alpha) * n + 0.5)
    assert lo in a and hi in a
    assert (a < lo).sum() <= t < (a <= lo).sum()
    assert (a > hi).sum() <= t < (a >= hi).sum()


def test_thresholds_match_library_order_statistic():
    """np.quantile(method='lower'/'higher') is the order statistic when q (n-1) is an integer."""
    rng = np.random.default_rng(1)
    n, t = 2001, 20                                     # alpha = 0.99, (1-alpha) n = 20.01 -> 20
    a = rng.standard_normal(n)
    lo, hi, n_tail = O.quantile_thresholds(a[None, :], 0.99)
    assert n_tail == t
    assert lo == np.quantile(a, t / (n - 1), method="lower")
    assert hi == np.quantile(a, 1 - t / (n - 1), method="higher")


@pytest.mark.parametrize("alpha", [0.999, 0.99, 0.97])
def test_clamped_fraction_is_one_minus_alpha_per_tail(alpha):
    """For distinct values exactly n_tail entries are clamped on each side: density 2(1-alpha)."""
    rng = np.random.default_rng(7)
    a = rng.permutation(np.arange(-20000, 20000) + 0.5)[None, :].astype(np.float64)  # all distinct
    q_lo, q_hi, t = O.quantile_thresholds(a, alpha)
    a_c, r = O.occ_split(a, q_lo, q_hi)
    assert (a > q_hi).sum() == t and (a < q_lo).sum() == t
    assert (r != 0).sum() == 2 * t
    assert abs((r != 0).mean() - 2 * (1 - alpha)) < 1.0 / a.size


def test_occ_identity_bounds_and_nnz():
    rng = np.random.default_rng(11)
    a = _bf16_normal(rng, (64, 256))
    a[:, [5, 77]] *= 40
    a = O.bf16_bits_to_f64(WL.to_bf16_bits(a.astype(np.float32)))
    q = O.occ_quantize(a, 0.99)
    a_c, r = O.occ_split(a, q.lo, q.hi)
    np.testing.assert_array_equal(a_c + r, a)                       # exact identity
    assert a_c.min() >= q.lo and a_c.max() <= q.hi
    nnz = int(q.csr[0][-1])
    assert nnz == (r != 0).sum() <= 2 * q.n_tail
    assert nnz == int(q.csc[0][-1])
    # entries equal to a threshold are not emitted
    assert not np.isin(a[r != 0], [q.lo, q.hi]).any()
    # residual values are exact in float32
    np.testing.assert_array_equal(q.csr[2].astype(np.float64), r[r != 0])
    # rows with a clamped entry on the dominant side have amax == max(|lo|, |hi|)
    big = max(abs(q.lo), abs(q.hi))
    side = (a >= q.hi) if abs(q.hi) >= abs(q.lo) else (a <= q.lo)
    rows = side.any(axis=1)
    assert rows.any()
    assert (q.amax[rows] == np.float32(big)).all()
    # CSR order: columns ascending within each row
    rowptr, col, _ = q.csr
    for m in range(64):
        seg = col[rowptr[m]:rowptr[m + 1]]
        assert (np.diff(seg) > 0).all()
    colptr, row, _ = q.csc
    for k in range(256):
        seg = row[colptr[k]:colptr[k + 1]]
        assert (np.diff(seg) > 0).all()


def test_alpha_one_means_no_clamp():
    rng = np.random.default_rng(2)
    a = _bf16_normal(rng, (8, 32))
    q = O.occ_quantize(a, 1.0)
    p = O.absmax_quantize(a, 0)
    np.testing.assert_array_equal(q.codes, p.codes)
    assert q.csr[0][-1] == 0


def test_negative_zero_threshold_is_plus_zero():
    a = np.array([[-1.0, -0.0, -0.0, 0.0, 0.0, 0.0, 0.0, 1.0]])
    lo, hi, t = O.quantile_thresholds(a, 0.875)
    assert t == 1 and lo == 0 and hi == 0
    assert not np.signbit(lo) and not np.signbit(hi)


def _snr_db(ref, approx):
    return 10 * np.log10((ref ** 2).sum() / ((ref - approx) ** 2).sum())


def test_compensation_trend_of_table1():
    """Table 1's reliable trend on synthetic data: clamp + compensation beats a direct cast,
    and the SNR rises as alpha falls."""
    cfg = WL.CONFIGS[0]
    a = O.bf16_bits_to_f64(WL.activations(cfg, 1024))
    direct = O.absmax_quantize(a, 0)
    rec_direct = O.e2m1_decode(direct.codes) * direct.descale.astype(np.float64)[:, None]
    snr = [_snr_db(a, rec_direct)]
    for alpha in (0.999, 0.99, 0.97):
        q = O.occ_quantize(a, alpha)
        rec = O.e2m1_decode(q.codes) * q.descale.astype(np.float64)[:, None] + q.residual
        snr.append(_snr_db(a, rec))
    assert snr[1] > snr[0]
    assert snr[1] < snr[2] < snr[3]


# ---------------------------------------------------------------------------------------------
# The variant outside the paper: one threshold on the magnitudes
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,alpha", [(50, 0.9), (1000, 0.99), (4096, 0.97), (777, 0.999)])
def test_abs_threshold_by_counting(n, alpha):
    """t is characterised without sorting: at most 2 n_tail magnitudes lie above it and more than
    2 n_tail lie at or above it; the clamp is symmetric."""
    rng = np.random.default_rng(n)
    a = np.round(rng.standard_normal(n) * 8) / 8 * rng.choice([1.0, 30.0], n, p=[0.95, 0.05])   # with ties
    lo, hi, n_tail = O.quantile_thresholds(a, alpha, quantile="abs")
    assert lo == -hi and hi >= 0 and n_tail == O.tail_count(n, alpha)
    assert np.sum(np.abs(a) > hi) <= 2 * n_tail < np.sum(np.abs(a) >= hi)
    assert hi in np.abs(a)                                  # an order statistic, not an interpolation


def test_abs_threshold_on_a_hand_worked_case():
    a = np.array([0.5, -7.0, 2.0, -1.0, 3.0, 0.0, -0.25, 6.0, 1.5, -2.5])      # magnitudes sorted: 0 .25 .5 1 1.5 2 2.5 3 6 7
    lo, hi, n_tail = O.quantile_thresholds(a, 0.9, quantile="abs")              # n_tail = 1: two entries may leave
    assert (lo, hi, n_tail) == (-3.0, 3.0, 1)
    q = O.occ_quantize(a.reshape(1, -1), 0.9, quantile="abs")
    np.testing.assert_array_equal(q.residual, np.array([[0, -4.0, 0, 0, 0, 0, 0, 3.0, 0, 0]]))
    z = np.zeros(10)
    z[3] = -5.0
    assert O.quantile_thresholds(z, 0.8, quantile="abs")[:2] == (0.0, 0.0)      # t = 0: lo is +0, not -0
    assert not np.signbit(O.quantile_thresholds(z, 0.8, quantile="abs")[0])


def test_abs_and_signed_forms_agree_on_mirrored_data():
    """A tensor that holds -x for every x has symmetric order statistics: both forms clamp alike."""
    rng = np.random.default_rng(4)
    h = rng.standard_normal(500)
    a = np.concatenate([h, -h])
    s = O.quantile_thresholds(a, 0.99)
    b = O.quantile_thresholds(a, 0.99, quantile="abs")
    assert s[1] == b[1] and s[0] == b[0] == -s[1]


# ---------------------------------------------------------------------------------------------
# The variant outside the paper: thresholds per token
# ---------------------------------------------------------------------------------------------
def test_token_thresholds_are_the_rows_own_order_statistics():
    rng = np.random.default_rng(9)
    a = _bf16_normal(rng, (6, 200)) * np.array([[1], [10], [0.1], [1], [100], [1]])
    a[3, :50] = a[3, 50:100]                               # ties
    lo, hi, n_tail = O.token_thresholds(a, 0.97)
    assert n_tail == 6
    for m in range(6):
        row = a[m]
        assert (row < lo[m]).sum() <= n_tail < (row <= lo[m]).sum()     # by counting, not by sorting
        assert (row > hi[m]).sum() <= n_tail < (row >= hi[m]).sum()
        assert lo[m] in row and hi[m] in row
        # a row on its own is what the tensor-wide form makes of a one-row tensor
        assert (lo[m], hi[m]) == O.quantile_thresholds(row[None, :], 0.97)[:2]


def test_token_variant_identity_bounds_and_counts():
    rng = np.random.default_rng(10)
    a = _bf16_normal(rng, (16, 256))
    a[:, 7] *= 30.0
    q = O.occ_quantize(a, 0.99, quantile="token")
    assert q.n_tail == 3 and q.lo_rows.shape == (16,)
    a_c = np.minimum(np.maximum(a, q.lo_rows[:, None]), q.hi_rows[:, None])
    np.testing.assert_array_equal(a_c + q.residual, a)      # clamped + residual == original, exactly
    per_row = (q.residual != 0).sum(axis=1)
    assert (per_row <= 2 * q.n_tail).all() and per_row.max() > 0
    np.testing.assert_array_equal(q.amax, np.abs(a_c).max(axis=1).astype(np.float32))
    rowptr, col, val = q.csr
    np.testing.assert_array_equal(np.diff(rowptr), per_row)
    whole = O.occ_quantize(a, 0.99)                          # the paper's form clamps the outlier column only
    assert (whole.residual != 0).sum() <= 2 * whole.n_tail
    assert not np.array_equal(whole.codes, q.codes)
