"""GPU parity of the E4M3 operands (the W4A8 / W8A4 settings of Section 4.3 and dY in FP8):
codes and scales bit for bit, layer outputs at the GEMM tolerance."""
import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

pytestmark = pytest.mark.gpu
RTOL = 1e-3


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0, 1 << 30)
    yield c
    c.close()


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (384, 1152)])
def test_e4m3_quantize_matches_oracle(lib, ctx, axis, shape):
    rng = np.random.default_rng(shape[0] + shape[1] + axis)
    bits = WL.to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * np.float32(0.02))
    bits[3, :] = 0                                    # a zero row
    bits[:, 5] = 0 if axis == 1 else bits[:, 5]
    bits[7, 9] = 0x8000                               # negative zero input keeps its sign
    ctx.status.zero_()
    q = lib.fp4_quantize(ctx, _dev(bits), axis, fmt=lib.FP4_FORMAT_E4M3)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    ref = O.absmax_quantize(O.bf16_bits_to_f64(bits), axis, fmt="e4m3")
    np.testing.assert_array_equal(q.amax.cpu().numpy(), ref.amax)
    np.testing.assert_array_equal(q.codes.cpu().numpy(), ref.codes)
    np.testing.assert_array_equal(q.codes_t.cpu().numpy(), np.ascontiguousarray(ref.codes.T))


def test_e4m3_conversion_on_every_tie_and_beyond_the_range(lib, ctx):
    """Rows whose amax is 448 (gamma = 1) carry every E4M3 value, every midpoint between two of
    them and its float32 neighbours... as far as BF16 inputs reach: all BF16 values up to 448."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    v = O.bf16_bits_to_f64(bits)
    keep = bits[np.isfinite(v) & (np.abs(v) <= 448.0)]
    cols = 256
    rows = -(-keep.size // (cols - 1))
    rows = -(-rows // 128) * 128
    x = np.zeros((rows, cols), dtype=np.uint16)
    x[:, 0] = 0x43E0                                   # 448.0 in every row -> gamma = 1
    body = np.zeros(rows * (cols - 1), dtype=np.uint16)
    body[:keep.size] = keep
    x[:, 1:] = body.reshape(rows, cols - 1)
    q = lib.fp4_quantize(ctx, _dev(x), 0, fmt=lib.FP4_FORMAT_E4M3)
    torch.cuda.synchronize()
    ref = O.absmax_quantize(O.bf16_bits_to_f64(x), 0, fmt="e4m3")
    assert (ref.amax == 448.0).all()
    np.testing.assert_array_equal(q.codes.cpu().numpy(), ref.codes)


def test_clamping_is_refused_for_e4m3(lib, ctx):
    x = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_quantize(ctx, x, 0, alpha=0.99, out=lib.QTensor(128, 128, 0, x.device, 1000, fmt=lib.FP4_FORMAT_E4M3))
    assert e.value.code == -7
    with pytest.raises(lib.Fp4Error) as e:          # E4M3 operands need the byte-container GEMM
        lib.fp4_linear_fwd(ctx, x, x, 1.0, fmt_a=lib.FP4_FORMAT_E4M3, gemm_kind=lib.FP4_GEMM_MXF4)
    assert e.value.code == -7


def _close(got, want, a, b=None, what=""):
    scale = np.abs(a) + (0 if b is None else np.abs(b))
    err = np.abs(got.astype(np.float64) - want)
    bad = err > RTOL * scale + 1e-300
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, worst {np.max(err / (scale + 1e-300))}"


CASES = [
    # M, K, N, fmt_a, fmt_w, fmt_dy, alpha
    (256, 384, 640, "e4m3", "e2m1", "e2m1", 1.0),     # W4A8
    (256, 384, 640, "e2m1", "e4m3", "e2m1", 0.98),    # W8A4 with clamping and compensation
    (384, 640, 384, "e2m1", "e2m1", "e4m3", 0.99),    # dY in FP8
    (128, 256, 128, "e4m3", "e2m1", "e4m3", 1.0),
    (256, 1152, 256, "e2m1", "e4m3", "e4m3", 0.99),
    (384, 640, 384, "e2m1", "e2m1", "e5m2", 0.99),    # dY in E5M2, the usual FP8 format of gradients
    (256, 384, 640, "e2m1", "e4m3", "e5m2", 0.98),    # W8A4 with E5M2 gradients
    (128, 256, 128, "e5m2", "e2m1", "e5m2", 1.0),
]


@pytest.mark.parametrize("M,K,N,fmt_a,fmt_w,fmt_dy,alpha", CASES)
def test_mixed_precision_layer_matches_oracle(lib, ctx, M, K, N, fmt_a, fmt_w, fmt_dy, alpha):
    code = {"e2m1": lib.FP4_FORMAT_E2M1, "e4m3": lib.FP4_FORMAT_E4M3, "e5m2": lib.FP4_FORMAT_E5M2}
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=M + K + N)
    f = O.linear_fwd(a_bits, w_bits, alpha, fmt_a=fmt_a, fmt_w=fmt_w)
    b = O.linear_bwd(dy_bits, w_bits, f, fmt_dy=fmt_dy)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    kind = lib.FP4_GEMM_F8F6F4
    ctx.status.zero_()
    y32, sa, sw = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind, out_f32=True, fmt_a=code[fmt_a], fmt_w=code[fmt_w])
    da32, dw32 = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind, out_f32=True, dy_fmt=code[fmt_dy])
    da_only, _ = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind, out_f32=True, dy_fmt=code[fmt_dy],
                                    want_dw=False)
    _, dw_only = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind, out_f32=True, dy_fmt=code[fmt_dy],
                                    want_da=False)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    # saved operands: bit for bit
    np.testing.assert_array_equal(sa.amax.cpu().numpy(), f.qa.amax)
    np.testing.assert_array_equal(sw.amax.cpu().numpy(), f.qw.amax)
    np.testing.assert_array_equal(sa.codes.cpu().numpy(), f.qa.packed() if fmt_a == "e2m1" else f.qa.codes)
    np.testing.assert_array_equal(sw.codes_t.cpu().numpy(),
                                  f.qw.packed_t() if fmt_w == "e2m1" else np.ascontiguousarray(f.qw.codes.T))
    _close(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y")
    _close(da32.cpu().numpy(), b.da, b.da, None, "dA")
    _close(dw32.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, "dW")
    assert torch.equal(da_only, da32) and torch.equal(dw_only, dw32)     # one-gradient calls take the same path
    if fmt_w != "e2m1":
        assert (b.dge == 1.0).all()


@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384)])
def test_e5m2_quantize_matches_oracle(lib, ctx, axis, shape):
    rng = np.random.default_rng(shape[0] + shape[1] + axis + 50)
    x = rng.standard_normal(shape).astype(np.float32) * np.exp2(rng.integers(-12, 4, size=shape)).astype(np.float32)
    bits = WL.to_bf16_bits(x)                          # wide range: E5M2 subnormals are reached
    bits[3, :] = 0
    bits[7, 9] = 0x8000                               # negative zero input keeps its sign
    ctx.status.zero_()
    q = lib.fp4_quantize(ctx, _dev(bits), axis, fmt=lib.FP4_FORMAT_E5M2)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    ref = O.absmax_quantize(O.bf16_bits_to_f64(bits), axis, fmt="e5m2")
    np.testing.assert_array_equal(q.amax.cpu().numpy(), ref.amax)
    np.testing.assert_array_equal(q.codes.cpu().numpy(), ref.codes)
    np.testing.assert_array_equal(q.codes_t.cpu().numpy(), np.ascontiguousarray(ref.codes.T))


def test_e5m2_conversion_on_every_bf16_value_in_range(lib, ctx):
    """Rows whose amax is 57344 (gamma = 1) carry every BF16 value up to 57344: every E5M2 value,
    every midpoint between two of them (BF16 has five more mantissa bits) and their neighbours."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    v = O.bf16_bits_to_f64(bits)
    keep = bits[np.isfinite(v) & (np.abs(v) <= 57344.0)]
    cols = 256
    rows = -(-keep.size // (cols - 1))
    rows = -(-rows // 128) * 128
    x = np.zeros((rows, cols), dtype=np.uint16)
    x[:, 0] = 0x4760                                   # 57344.0 in every row -> gamma = 1
    body = np.zeros(rows * (cols - 1), dtype=np.uint16)
    body[:keep.size] = keep
    x[:, 1:] = body.reshape(rows, cols - 1)
    q = lib.fp4_quantize(ctx, _dev(x), 0, fmt=lib.FP4_FORMAT_E5M2)
    torch.cuda.synchronize()
    ref = O.absmax_quantize(O.bf16_bits_to_f64(x), 0, fmt="e5m2")
    assert (ref.amax == 57344.0).all()
    np.testing.assert_array_equal(q.codes.cpu().numpy(), ref.codes)


def test_gemm_with_e5m2_operands(lib, ctx):
    """fp4_gemm on the byte-container kind with an E5M2 operand on either side."""
    rng = np.random.default_rng(9)
    I, J, C = 128, 256, 384
    xa = O.bf16_bits_to_f64(WL.to_bf16_bits(rng.standard_normal((I, C)).astype(np.float32)))
    xb = O.bf16_bits_to_f64(WL.to_bf16_bits(rng.standard_normal((J, C)).astype(np.float32)))
    for fa, fb, kind in (("e5m2", "e2m1", lib.FP4_GEMM_F8F6F4_A8 | lib.FP4_GEMM_A_E5M2),
                         ("e2m1", "e5m2", lib.FP4_GEMM_F8F6F4_B8 | lib.FP4_GEMM_B_E5M2),
                         ("e5m2", "e4m3", lib.FP4_GEMM_F8F6F4_A8B8 | lib.FP4_GEMM_A_E5M2)):
        qa, qb = O.absmax_quantize(xa, 0, fmt=fa), O.absmax_quantize(xb, 0, fmt=fb)
        ca = torch.from_numpy(qa.packed() if fa == "e2m1" else qa.codes).cuda()
        cb = torch.from_numpy(qb.packed() if fb == "e2m1" else qb.codes).cuda()
        got = lib.fp4_gemm(ctx, ca, cb, torch.from_numpy(qa.amax).cuda(), torch.from_numpy(qb.amax).cuda(),
                           gemm_kind=kind)
        torch.cuda.synchronize()
        want = (O.gemm_values(qa, qb) * qa.descale.astype(np.float64)[:, None]) * qb.descale.astype(np.float64)[None, :]
        terms = (np.abs(qa.values()) @ np.abs(qb.values()).T) * qa.descale.astype(np.float64)[:, None] \
            * qb.descale.astype(np.float64)[None, :]
        err = np.abs(got.cpu().numpy().astype(np.float64) - want)
        assert (err <= RTOL * np.abs(want) + 2 * (C // 32) * 2.0 ** -23 * terms).all(), (fa, fb)
    with pytest.raises(lib.Fp4Error):                  # the E5M2 flag qualifies an 8-bit operand
        lib.fp4_gemm(ctx, ca, cb, None, None, gemm_kind=lib.FP4_GEMM_F8F6F4 | lib.FP4_GEMM_A_E5M2)


def test_fp8_accumulation_stays_inside_its_floor(lib, ctx):
    """Measures what the accumulation floor of GEMMs with an 8-bit operand allows for (one tensor-core
    addition per 32 contraction columns, each off by at most 2 * 2^-23 of the running sum).  Rows of
    A against rows of B whose products alternate in sign cancel to a small fraction of their summed
    magnitudes; the GPU's sum must stay within half of that floor (plus the rounding of the two
    de-scales), at the longest contraction the workloads have."""
    rng = np.random.default_rng(31)
    I, J, C = 128, 128, 16384
    xa = np.abs(rng.standard_normal((I, C))).astype(np.float32)
    xb = np.abs(rng.standard_normal((J, C))).astype(np.float32)
    xb[:, ::2] *= -1.0                                                # alternating signs along the contraction
    xa = O.bf16_bits_to_f64(WL.to_bf16_bits(xa))
    xb = O.bf16_bits_to_f64(WL.to_bf16_bits(xb))
    qa, qb = O.absmax_quantize(xa, 0, fmt="e4m3"), O.absmax_quantize(xb, 0, fmt="e2m1")
    ca, cb = torch.from_numpy(qa.codes).cuda(), torch.from_numpy(qb.packed()).cuda()
    got = lib.fp4_gemm(ctx, ca, cb, torch.from_numpy(qa.amax).cuda(), torch.from_numpy(qb.amax).cuda(),
                       gemm_kind=lib.FP4_GEMM_F8F6F4_A8)
    torch.cuda.synchronize()
    scale = qa.descale.astype(np.float64)[:, None] * qb.descale.astype(np.float64)[None, :]
    want = O.gemm_values(qa, qb) * scale
    terms = (np.abs(qa.values()) @ np.abs(qb.values()).T) * scale
    assert np.median(np.abs(want) / terms) < 0.05                     # the sums do cancel
    floor = 2.0 * (C // 32) * 2.0 ** -23 * terms
    err = np.abs(got.cpu().numpy().astype(np.float64) - want)
    assert (err <= 0.5 * floor + 4 * 2.0 ** -23 * np.abs(want)).all(), f"{np.max(err / floor):.3f} of the floor"
