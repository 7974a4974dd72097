"""Plain, slow, double-precision CPU oracle of the FP4-quantized linear layer.

TEST INFRASTRUCTURE.  This module is the yardstick the CUDA library is compared
with; it is not a fallback and must never be reached from the product path.  It
shares no code, table or helper with the CUDA sources.

Everything is written step by step in the order and notation of the paper
("Optimizing Large Language Model Training Using FP4 Quantization"):

* E2M1 value grid ................................ Table 4 (row ``e2m1``), Section 2
* absmax scaling  x_fp4 = Q(x * gamma) ............ Eq. 1
* look-up quantiser Q ............................. Appendix A (the 14-threshold chain)
* vector-wise granularity (token / channel) ....... Section 4.1, Appendix C.2
* outlier clamp + sparse residual (OCC) ........... Section 3.2
* FP4 GEMM followed by the two de-scales .......... Fig. 2, Appendix C.2
* DGE function f and derivative f' ................ Eq. 7, Eq. 8 (k = 5, cap 3.0)
* weight gradient dL/dW = dL/dW_q (.) Q'(W_scaled)  Eq. 6 and the last equation of Appendix C.2

Arithmetic is float64.  The few places where a float32 rounding is part of the
definition are explicit and marked ``RN32``: the quantiser of Appendix A acts on
float32 numbers, so the scale ``gamma`` and the scaled value are float32.

Readings of points the paper leaves open (each also listed in the design notes):

* Q sends a value that equals a threshold to the larger neighbour (strict ``<``
  chain of Appendix A), and never emits a negative zero code.
* ``gamma = RN32(6 / amax)``, scaled value ``RN32(x * gamma)``, de-scale
  ``d = RN32(amax / 6)``; an all-zero vector gets ``gamma = d = 0``.
* Quantiles are order statistics of the whole tensor, signed and two-sided:
  with ``n_tail = round((1 - alpha) * n)``, ``lo = sorted[n_tail]`` and
  ``hi = sorted[n - 1 - n_tail]`` (Section 3.2 gives a residual density of
  2(1 - alpha), Appendix B).
* The residual is multiplied by the original BF16 weight in high precision
  (Section 3.2 asks for a high-precision product of the sparse residual).
* Backward GEMMs take E2M1 operands as well (Appendix B counts the backward at
  the FP4 rate) and re-use the forward codes of A and W; the scale vector that
  lies along the contraction is folded into dY before dY is quantised.
  PARITY UNPINNED by the paper for this choice: it is pinned only by brute
  force and by an algebraic identity (see tests).
* FP8 operands (the W4A8 and W8A4 settings of the ablation in Section 4.3, and the
  reading of the backward that keeps dY in FP8): the paper names the settings, not
  the format's details.  Reading taken: OCP E4M3 (4 exponent bits, bias 7, 3 mantissa
  bits, no infinity, largest finite value 448), round to nearest even with saturation,
  the sign of the input kept, vector-wise absmax scaling along the same axes as for
  E2M1 with MAX = 448.  OCC belongs to 4-bit activations and DGE to 4-bit weights, so
  an E4M3 activation is not clamped and an E4M3 weight gets the straight-through
  estimator.  PARITY UNPINNED by the paper for all of this as well.  The other FP8
  variant the paper names (Section 2), E5M2 (5 exponent bits, bias 15, 2 mantissa
  bits, infinities and NaNs at exponent field 31, largest finite value 57344), is
  offered the same way, with MAX = 57344 and saturation to the largest finite value.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# --------------------------------------------------------------------------- #
# E2M1 format: Table 4, row "e2m1"; sign-magnitude 4-bit codes (Section 2).
# --------------------------------------------------------------------------- #
E2M1_MAGNITUDES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
FP4_MAX = 6.0  # the largest E2M1 magnitude: the value the text below Eq. 1 gives for MAX_fp4

# Appendix A: the 14 constants of the comparison chain and the 15 results.
LUT_THRESHOLDS = np.array(
    [-5.0, -3.5, -2.5, -1.75, -1.25, -0.75, -0.25, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
)
LUT_VALUES = np.array(
    [-6.0, -4.0, -3.0, -2.0, -1.5, -1.0, -0.5, 0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
)
# code of each LUT result: negatives 1111..1001, zero 0000, positives 0001..0111
_LUT_CODES = np.array(
    [0xF, 0xE, 0xD, 0xC, 0xB, 0xA, 0x9, 0x0, 0x1, 0x2, 0x3, 0x4, 0x5, 0x6, 0x7], dtype=np.uint8
)


def bf16_bits_to_f64(bits) -> np.ndarray:
    """Exact value of BF16 bit patterns (uint16) as float64."""
    b = np.asarray(bits, dtype=np.uint16)
    with np.errstate(invalid="ignore"):     # signalling-NaN patterns only matter to the brute-force tests
        return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_f64(x) -> np.ndarray:
    """Round float64 to the nearest BF16 value (ties to even), returned as float64.

    One rounding, straight from double: significand kept to 8 bits.  Only used to
    state what a correctly rounded BF16 store of an oracle result would hold.
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                      # x = m * 2**e, 0.5 <= |m| < 1
    q = np.rint(m * 256.0)                  # 8 significant bits, ties to even
    return np.ldexp(q, e - 8)


def e2m1_decode(codes) -> np.ndarray:
    """Value of 4-bit E2M1 codes: bit 3 sign, bits 2..0 index into the magnitude grid."""
    c = np.asarray(codes, dtype=np.uint8)
    mag = E2M1_MAGNITUDES[c & 7]
    return np.where((c & 8) != 0, -mag, mag)


def lut_quantize(v32) -> np.ndarray:
    """Q of Appendix A on float32 inputs -> E2M1 codes.

    The chain tests ``v < t_0``, ``v < t_1`` ... in order and the first true test
    wins, so the result index is the number of thresholds that are <= v.
    """
    v = np.asarray(v32)
    assert v.dtype == np.float32, "Q is defined on float32 numbers (Appendix A)"
    idx = np.zeros(v.shape, dtype=np.int64)
    for t in LUT_THRESHOLDS:                # 14 comparisons, in the paper's order
        idx += (v >= np.float32(t))
    return _LUT_CODES[idx]


def pack_nibbles(codes) -> np.ndarray:
    """Two codes per byte along the last axis: even index in bits 3:0, odd in 7:4."""
    c = np.asarray(codes, dtype=np.uint8)
    assert c.shape[-1] % 2 == 0
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)


def unpack_nibbles(packed) -> np.ndarray:
    p = np.asarray(packed, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = p & 0xF
    out[..., 1::2] = p >> 4
    return out


# --------------------------------------------------------------------------- #
# absmax vector-wise quantisation: Eq. 1, Section 4.1, Appendix C.2
# --------------------------------------------------------------------------- #
def rn32(x) -> np.ndarray:
    """Round float64 to float32 (IEEE nearest-even) and return it as float64."""
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def absmax_scales(amax, fmax: float = FP4_MAX):
    """gamma = RN32(MAX / amax) (Eq. 1) and the de-scale d = RN32(amax / MAX)."""
    a32 = np.asarray(amax, dtype=np.float32)
    top = np.float32(fmax)
    with np.errstate(divide="ignore", invalid="ignore"):
        gamma = np.where(a32 > 0, top / a32, np.float32(0)).astype(np.float32)
        d = (a32 / top).astype(np.float32)
    return gamma, d


# --------------------------------------------------------------------------- #
# FP8 E4M3 (Section 2 names the format; Section 4.3 the W4A8 / W8A4 settings)
# --------------------------------------------------------------------------- #
E4M3_MAX = 448.0


def e4m3_decode(codes) -> np.ndarray:
    """Value of every E4M3 byte: S.EEEE.MMM, bias 7, subnormals at E = 0, S.1111.111 is NaN."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    e = (c >> 3) & 0xF
    m = (c & 7).astype(np.float64)
    mag = np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    mag = np.where((c & 0x7F) == 0x7F, np.nan, mag)
    return np.where(c & 0x80, -mag, mag)


def e4m3_quantize(v32) -> np.ndarray:
    """Nearest E4M3 value of float32 numbers (ties to the even mantissa), saturating at 448.

    Returns the codes; the sign bit is the sign of the input, also when the result is zero.
    """
    v = np.asarray(v32, dtype=np.float32).astype(np.float64)
    a = np.minimum(np.abs(v), E4M3_MAX)
    _, ex = np.frexp(a)                                  # a = m * 2**ex with m in [0.5, 1)
    e = np.clip(ex - 1, -6, 8)                           # binade of a (subnormals share e = -6)
    step = np.exp2((e - 3).astype(np.float64))           # spacing of the grid inside that binade
    q = np.minimum(np.rint(a / step) * step, E4M3_MAX)   # np.rint rounds halves to even
    _, exq = np.frexp(q)
    eq = np.clip(exq - 1, -6, 8)
    normal = q >= 2.0 ** -6
    field_e = np.where(normal, eq + 7, 0).astype(np.int64)
    field_m = np.where(normal, np.rint((q / np.exp2(eq.astype(np.float64)) - 1.0) * 8.0),
                       np.rint(q / 2.0 ** -9)).astype(np.int64)
    sign = np.signbit(v).astype(np.int64)
    return ((sign << 7) | (field_e << 3) | field_m).astype(np.uint8)


# --------------------------------------------------------------------------- #
# FP8 E5M2 (the other variant Section 2 names)
# --------------------------------------------------------------------------- #
E5M2_MAX = 57344.0


def e5m2_decode(codes) -> np.ndarray:
    """Value of every E5M2 byte: S.EEEEE.MM, bias 15, subnormals at E = 0, E = 31 is infinity (M = 0) or NaN."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    e = (c >> 2) & 0x1F
    m = (c & 3).astype(np.float64)
    mag = np.where(e == 0, m / 4.0 * 2.0 ** -14, (1.0 + m / 4.0) * np.exp2((e - 15).astype(np.float64)))
    mag = np.where(e == 31, np.where(m == 0, np.inf, np.nan), mag)
    return np.where(c & 0x80, -mag, mag)


def e5m2_quantize(v32) -> np.ndarray:
    """Nearest E5M2 value of float32 numbers (ties to the even mantissa), saturating at 57344.

    Returns the codes; the sign bit is the sign of the input, also when the result is zero.
    """
    v = np.asarray(v32, dtype=np.float32).astype(np.float64)
    a = np.minimum(np.abs(v), E5M2_MAX)
    _, ex = np.frexp(a)
    e = np.clip(ex - 1, -14, 15)                         # binade of a (subnormals share e = -14)
    step = np.exp2((e - 2).astype(np.float64))           # spacing of the grid inside that binade
    q = np.minimum(np.rint(a / step) * step, E5M2_MAX)   # np.rint rounds halves to even
    _, exq = np.frexp(q)
    eq = np.clip(exq - 1, -14, 15)
    normal = q >= 2.0 ** -14
    field_e = np.where(normal, eq + 15, 0).astype(np.int64)
    field_m = np.where(normal, np.rint((q / np.exp2(eq.astype(np.float64)) - 1.0) * 4.0),
                       np.rint(q / 2.0 ** -16)).astype(np.int64)
    sign = np.signbit(v).astype(np.int64)
    return ((sign << 7) | (field_e << 2) | field_m).astype(np.uint8)


FORMAT_MAX = {"e2m1": 6.0, "e4m3": E4M3_MAX, "e5m2": E5M2_MAX}


@dataclass
class Quantized:
    """Everything one call of the quantiser produces (all host arrays)."""
    rows: int
    cols: int
    scale_axis: int
    codes: np.ndarray            # [rows, cols] uint8, one code per element
    amax: np.ndarray             # float32, [rows] (scale_axis 0) or [cols] (scale_axis 1)
    scaled: np.ndarray           # float32 [rows, cols]: the numbers Q was applied to
    lo: float = 0.0              # clamp thresholds (OCC only)
    hi: float = 0.0
    n_tail: int = 0
    csr: tuple = field(default=None)   # (rowptr int32[rows+1], col int32[nnz], val float32[nnz])
    csc: tuple = field(default=None)   # (colptr int32[cols+1], row int32[nnz], val float32[nnz])
    residual: np.ndarray = None  # dense float64 [rows, cols] (zeros outside the tails)
    fmt: str = "e2m1"            # "e2m1": one nibble code per element; "e4m3" / "e5m2": one byte per element
    lo_rows: np.ndarray = None   # per-token variant of the clamp: thresholds of every row
    hi_rows: np.ndarray = None

    @property
    def fmax(self):
        return FORMAT_MAX[self.fmt]

    @property
    def gamma(self):
        return absmax_scales(self.amax, self.fmax)[0]

    @property
    def descale(self):
        return absmax_scales(self.amax, self.fmax)[1]

    def values(self):
        """The numbers the codes stand for, float64 [rows, cols]."""
        return {"e2m1": e2m1_decode, "e4m3": e4m3_decode, "e5m2": e5m2_decode}[self.fmt](self.codes)

    def packed(self):
        """[rows, cols/2] bytes, column pairs packed."""
        return pack_nibbles(self.codes)

    def packed_t(self):
        """[cols, rows/2] bytes, row pairs packed (the transposed layout)."""
        return pack_nibbles(np.ascontiguousarray(self.codes.T))


def absmax_quantize(x, scale_axis: int, prescale=None, fmt: str = "e2m1") -> Quantized:
    """Vector-wise absmax quantisation of a 2-D float64 array of BF16-exact numbers.

    ``scale_axis`` 0: one scale per row (token-wise, activations, Section 4.1);
    ``scale_axis`` 1: one scale per column (channel-wise, weights W[c_i x c_o],
    Appendix C.2 where sf is 1 x c_o).
    ``prescale``: optional float32 vector laid along the *other* axis that
    multiplies x first, x <- RN32(x * prescale) (used for dY in the backward).
    ``fmt``: "e2m1" (Eq. 1 with MAX = 6 and the quantiser of Appendix A), "e4m3"
    (MAX = 448, nearest-even rounding: the FP8 operand of the W4A8 / W8A4 settings) or "e5m2"
    (MAX = 57344, the same rounding).
    """
    x = np.asarray(x, dtype=np.float64)
    rows, cols = x.shape
    if prescale is not None:
        p = np.asarray(prescale, dtype=np.float32).astype(np.float64)
        p = p[None, :] if scale_axis == 0 else p[:, None]
        x = rn32(x * p)                     # exact double product, one rounding
    amax = np.max(np.abs(x), axis=1 - scale_axis).astype(np.float32)
    gamma, _ = absmax_scales(amax, FORMAT_MAX[fmt])
    g = gamma.astype(np.float64)
    g = g[:, None] if scale_axis == 0 else g[None, :]
    scaled = (x * g).astype(np.float32)     # RN32(x * gamma): the product is exact in double
    codes = {"e2m1": lut_quantize, "e4m3": e4m3_quantize, "e5m2": e5m2_quantize}[fmt](scaled)
    return Quantized(rows, cols, scale_axis, codes, amax, scaled, fmt=fmt)


# --------------------------------------------------------------------------- #
# Outlier clamping and compensation: Section 3.2
# --------------------------------------------------------------------------- #
def tail_count(n: int, alpha: float) -> int:
    """Entries beyond each quantile: round((1 - alpha) * n), halves away from zero."""
    return int(math.floor((1.0 - float(alpha)) * float(n) + 0.5))


def quantile_thresholds(a, alpha: float, quantile: str = "signed"):
    """(lo, hi, n_tail): the (1-alpha)- and alpha-quantiles as order statistics.

    ``quantile`` = "signed" is the paper's form (Section 3.2: clamp between the alpha-quantile and
    the (1-alpha)-quantile of the values).  "abs" is a variant outside the paper: one threshold t
    on the magnitudes, the order statistic of |x| that at most 2 n_tail entries exceed, with
    lo = -t and hi = +t (the same number of entries may leave the clamp as in the signed form).
    """
    a = np.asarray(a, dtype=np.float64)
    n = a.size
    n_tail = tail_count(n, alpha)
    if not (2 * n_tail < n):
        raise ValueError("alpha leaves nothing between the two tails")
    if quantile == "abs":
        t = float(np.sort(np.abs(a).ravel())[n - 1 - 2 * n_tail])
        return -t + 0.0, t, n_tail            # "+ 0.0" turns -0.0 into +0.0
    if quantile != "signed":
        raise ValueError(quantile)
    s = np.sort(a.ravel())
    lo = float(s[n_tail]) + 0.0             # "+ 0.0" turns -0.0 into +0.0
    hi = float(s[n - 1 - n_tail]) + 0.0
    return lo, hi, n_tail


def occ_split(a, lo: float, hi: float):
    """Y_c = clamp(Y, max=hi, min=lo) and the residual dY = Y - Y_c (Section 3.2)."""
    a = np.asarray(a, dtype=np.float64)
    a_c = np.minimum(np.maximum(a, lo), hi)
    return a_c, a - a_c


def sparse_from_dense(r):
    """CSR (rows, then columns ascending) and CSC (columns, then rows ascending) of r != 0."""
    rows, cols = r.shape
    ri, ci = np.nonzero(r)                  # row-major order
    rowptr = np.zeros(rows + 1, dtype=np.int32)
    np.cumsum(np.bincount(ri, minlength=rows), out=rowptr[1:])
    csr = (rowptr, ci.astype(np.int32), r[ri, ci].astype(np.float32))
    rt = np.ascontiguousarray(r.T)
    cj, rj = np.nonzero(rt)
    colptr = np.zeros(cols + 1, dtype=np.int32)
    np.cumsum(np.bincount(cj, minlength=cols), out=colptr[1:])
    csc = (colptr, rj.astype(np.int32), rt[cj, rj].astype(np.float32))
    return csr, csc


def token_thresholds(a, alpha: float):
    """(lo[rows], hi[rows], n_tail): the signed order statistics of every token (row) on its own.

    A variant outside the paper (which takes the quantiles of the whole tensor): n_tail =
    round((1 - alpha) * cols) entries of every row may leave the clamp on either side.
    """
    a = np.asarray(a, dtype=np.float64)
    cols = a.shape[1]
    n_tail = tail_count(cols, alpha)
    if not (2 * n_tail < cols):
        raise ValueError("alpha leaves nothing between the two tails of a row")
    s = np.sort(a, axis=1)
    return s[:, n_tail] + 0.0, s[:, cols - 1 - n_tail] + 0.0, n_tail      # "+ 0.0" turns -0.0 into +0.0


def occ_quantize(a, alpha: float, quantile: str = "signed") -> Quantized:
    """Clamp at the quantiles, keep the sparse residual, then token-wise absmax + Q.

    The clamp comes first: its purpose is to shrink the range the absmax scale
    has to cover (Section 3.2, first paragraph).  ``quantile`` = "token" takes the thresholds of
    every row from that row alone (``lo_rows`` / ``hi_rows`` of the result; ``lo`` / ``hi`` are NaN).
    """
    a = np.asarray(a, dtype=np.float64)
    if alpha < 1.0 and quantile == "token":
        lo_r, hi_r, n_tail = token_thresholds(a, alpha)
        a_c = np.minimum(np.maximum(a, lo_r[:, None]), hi_r[:, None])
        r = a - a_c
        q = absmax_quantize(a_c, 0)
        q.lo, q.hi, q.n_tail = float("nan"), float("nan"), n_tail
        q.lo_rows, q.hi_rows = lo_r, hi_r
        q.residual = r
        q.csr, q.csc = sparse_from_dense(r)
        return q
    if alpha >= 1.0:
        q = absmax_quantize(a, 0)
        q.residual = np.zeros_like(a)
        q.csr, q.csc = sparse_from_dense(q.residual)
        q.lo, q.hi = float("-inf"), float("inf")
        return q
    lo, hi, n_tail = quantile_thresholds(a, alpha, quantile)
    a_c, r = occ_split(a, lo, hi)
    q = absmax_quantize(a_c, 0)
    q.lo, q.hi, q.n_tail = lo, hi, n_tail
    q.residual = r
    q.csr, q.csc = sparse_from_dense(r)
    return q


# --------------------------------------------------------------------------- #
# FP4 GEMM: Fig. 2 (both scale vectors are applied to the accumulated result)
# --------------------------------------------------------------------------- #
def gemm_codes(codes_a, codes_b) -> np.ndarray:
    """acc[i, j] = sum_c val(codes_a[i, c]) * val(codes_b[j, c]), exact.

    Every E2M1 value is a multiple of 1/2, so the doubled values are small
    integers and their float64 matrix product is an exact integer.
    """
    a2 = 2.0 * e2m1_decode(codes_a)
    b2 = 2.0 * e2m1_decode(codes_b)
    return (a2 @ b2.T) / 4.0


def gemm_values(qa: Quantized, qb: Quantized, transpose_a: bool = False, transpose_b: bool = False) -> np.ndarray:
    """acc[i, j] = sum_c val_a[i, c] * val_b[j, c] for operands of either format, exact.

    E2M1 values are multiples of 2^-1 up to 6 and E4M3 values multiples of 2^-9 up to 448, so
    every product is a multiple of 2^-18 below 2^18 and sums of up to 2^17 of them are exact in
    float64.  E5M2 values are multiples of 2^-16 up to 57344: with an E2M1 partner the sums are
    still exact (multiples of 2^-17 below 2^19), with an 8-bit partner they are float64 sums
    (2^-53 of the summed magnitudes).  ``transpose_*`` takes the operand's codes transposed first.
    """
    va = qa.values().T if transpose_a else qa.values()
    vb = qb.values().T if transpose_b else qb.values()
    return va @ vb.T


# --------------------------------------------------------------------------- #
# Differentiable gradient estimator: Eq. 7, Eq. 8
# --------------------------------------------------------------------------- #
def _interval(a):
    """Lower grid point g and width delta of the E2M1 interval that holds |x| = a.

    Widths: 0.5 below 2, 1 on [2, 4), 2 from 4 up (the last interval's formula is
    simply continued past 6).  Seven intervals per sign: the "14 intervals".
    """
    a = np.asarray(a, dtype=np.float64)
    g = np.where(a < 2.0, 0.5 * np.floor(2.0 * a), np.where(a < 4.0, np.floor(a), 4.0))
    delta = np.where(a < 2.0, 0.5, np.where(a < 4.0, 1.0, 2.0))
    return g, delta


def dge_f(x, k: float = 5.0) -> np.ndarray:
    """Eq. 7 applied inside every quantisation interval; odd in x."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    g, delta = _interval(a)
    t = 2.0 * (a - g) / delta - 1.0
    y = g + 0.5 * delta * (1.0 + np.sign(t) * np.abs(t) ** (1.0 / k))
    return np.sign(x) * y


def dge_fprime(x, k: float = 5.0, clip: float = 3.0) -> np.ndarray:
    """Eq. 8 with the magnitude capped at ``clip`` (3.0 in the paper); even in x."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    g, delta = _interval(a)
    t = np.abs(2.0 * (a - g) / delta - 1.0)
    with np.errstate(divide="ignore"):
        d = (1.0 / k) * t ** (1.0 / k - 1.0)
    return np.minimum(d, clip)


# --------------------------------------------------------------------------- #
# The linear layer, forward and backward
# --------------------------------------------------------------------------- #
@dataclass
class Forward:
    y: np.ndarray          # float64 [M, N]: FP4 branch + compensation
    y_fp4: np.ndarray      # float64 [M, N]: (acc * d_A[m]) * d_W[n]
    y_comp: np.ndarray     # float64 [M, N]: residual @ W
    acc: np.ndarray        # exact accumulators
    qa: Quantized
    qw: Quantized


def linear_fwd(a_bits, w_bits, alpha: float, fmt_a: str = "e2m1", fmt_w: str = "e2m1",
               quantile: str = "signed") -> Forward:
    """Y = (Q(A_c) Q(W)) (.) scales + dA W  (Fig. 2, Section 3.2).

    ``a_bits`` uint16 [M, K] and ``w_bits`` uint16 [K, N] are BF16 bit patterns.
    ``fmt_a`` / ``fmt_w`` = "e4m3" give the W4A8 / W8A4 settings of Section 4.3: an E4M3
    activation is quantised token-wise without clamping (alpha must then be 1).
    """
    a = bf16_bits_to_f64(a_bits)
    w = bf16_bits_to_f64(w_bits)
    if fmt_a == "e2m1":
        qa = occ_quantize(a, alpha, quantile)   # token-wise, with OCC
    else:
        if alpha != 1.0:
            raise ValueError("outlier clamping belongs to 4-bit activations")
        qa = absmax_quantize(a, 0, fmt=fmt_a)
        qa.residual = np.zeros_like(a)
    qw = absmax_quantize(w, 1, fmt=fmt_w)       # channel-wise (per output channel)
    if fmt_a == "e2m1" and fmt_w == "e2m1":
        acc = gemm_codes(qa.codes, qw.codes.T)  # contraction over k
    else:
        acc = gemm_values(qa, qw, transpose_b=True)
    d_a = qa.descale.astype(np.float64)
    d_w = qw.descale.astype(np.float64)
    y_fp4 = (acc * d_a[:, None]) * d_w[None, :]
    y_comp = qa.residual @ w
    return Forward(y_fp4 + y_comp, y_fp4, y_comp, acc, qa, qw)


@dataclass
class Backward:
    da: np.ndarray         # float64 [M, K]
    dw: np.ndarray         # float64 [K, N]
    s: np.ndarray          # float64 [K, N]: dL/dW_q before the DGE factor
    s_fp4: np.ndarray
    s_comp: np.ndarray
    dge: np.ndarray        # float64 [K, N]: Q'(W_scaled) (ones when DGE is off)
    qg_dgrad: Quantized    # dY (.) d_W, token-wise
    qg_wgrad: Quantized    # dY (.) d_A, channel-wise


def linear_bwd(dy_bits, w_bits, fwd: Forward, dge_on: bool = True,
               k: float = 5.0, clip: float = 3.0, fmt_dy: str = "e2m1") -> Backward:
    """dL/dA = dL/dY W_q^T and dL/dW = (A^T dL/dY) (.) Q'(W_scaled) (Eq. 3, Eq. 6, App. C.2).

    ``fmt_dy`` = "e4m3" keeps both quantised copies of dY in FP8.  The operands saved by the
    forward keep the format the forward gave them.  The DGE factor belongs to 4-bit weights:
    with an E4M3 weight the straight-through estimator is used whatever ``dge_on`` says.
    """
    dy = bf16_bits_to_f64(dy_bits)
    qa, qw = fwd.qa, fwd.qw
    d_a, d_w = qa.descale, qw.descale
    all_fp4 = qa.fmt == "e2m1" and qw.fmt == "e2m1" and fmt_dy == "e2m1"
    # dgrad: sum_n dY[m,n] d_W[n] val(codeW[k,n]); the W de-scale is folded into dY.
    qg1 = absmax_quantize(dy, 0, prescale=d_w, fmt=fmt_dy)
    acc1 = gemm_codes(qg1.codes, qw.codes) if all_fp4 else gemm_values(qg1, qw)
    da = acc1 * qg1.descale.astype(np.float64)[:, None]
    # wgrad: sum_m d_A[m] val(codeA[m,k]) dY[m,n]; the A de-scale is folded into dY.
    qg2 = absmax_quantize(dy, 1, prescale=d_a, fmt=fmt_dy)
    acc2 = gemm_codes(qa.codes.T, qg2.codes.T) if all_fp4 else gemm_values(qa, qg2, transpose_a=True, transpose_b=True)
    s_fp4 = acc2 * qg2.descale.astype(np.float64)[None, :]
    s_comp = qa.residual.T @ dy
    s = s_fp4 + s_comp
    if dge_on and qw.fmt == "e2m1":
        factor = dge_fprime(qw.scaled.astype(np.float64), k, clip)
    else:
        factor = np.ones_like(s)            # straight-through estimator, f' = 1
    return Backward(da, s * factor, s, s_fp4, s_comp, factor, qg1, qg2)
