"""GPU parity of fp4_quantize against the oracle: codes (both layouts), amax, thresholds and
the sparse residual are compared bit for bit."""
import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0, 512 << 20)
    yield c
    c.close()


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _check_dense(q, ref: O.Quantized):
    np.testing.assert_array_equal(q.amax.cpu().numpy(), ref.amax)
    if q.codes is not None:
        np.testing.assert_array_equal(q.codes.cpu().numpy(), ref.packed())
    if q.codes_t is not None:
        np.testing.assert_array_equal(q.codes_t.cpu().numpy(), ref.packed_t())


def _check_sparse(q, ref: O.Quantized):
    th = q.thresholds.cpu().numpy()
    assert (float(th[0]), float(th[1])) == (ref.lo, ref.hi)
    assert not (np.signbit(th) & (th == 0)).any()        # a zero threshold is +0
    nnz = int(q.nnz.item())
    rowptr, col, val = ref.csr
    colptr, row, cval = ref.csc
    assert nnz == rowptr[-1]
    np.testing.assert_array_equal(q.csr_rowptr.cpu().numpy(), rowptr)
    np.testing.assert_array_equal(q.csr_col.cpu().numpy()[:nnz], col)
    np.testing.assert_array_equal(q.csr_val.cpu().numpy()[:nnz], val)
    np.testing.assert_array_equal(q.csc_colptr.cpu().numpy(), colptr)
    np.testing.assert_array_equal(q.csc_row.cpu().numpy()[:nnz], row)
    np.testing.assert_array_equal(q.csc_val.cpu().numpy()[:nnz], cval)


@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (384, 1152), (1024, 640)])
def test_absmax_quantize_matches_oracle(lib, ctx, axis, shape):
    rng = np.random.default_rng(shape[0] + shape[1] + axis)
    bits = WL.to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * np.float32(0.02))
    bits[3, :] = 0                                    # a zero row: amax 0 when axis == 0
    bits[:, 5] = 0 if axis == 1 else bits[:, 5]       # a zero column when axis == 1
    bits[7, 9] = 0x8000                               # negative zero input
    ctx.status.zero_()
    q = lib.fp4_quantize(ctx, _dev(bits), axis)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    _check_dense(q, O.absmax_quantize(O.bf16_bits_to_f64(bits), axis))


@pytest.mark.parametrize("axis", [0, 1])
def test_prescaled_quantize_matches_oracle(lib, ctx, axis):
    rng = np.random.default_rng(17 + axis)
    rows, cols = 256, 384
    bits = WL.to_bf16_bits(rng.standard_normal((rows, cols)).astype(np.float32) * np.float32(1e-3))
    p = (rng.random(cols if axis == 0 else rows).astype(np.float32) * 3 + np.float32(0.01))
    q = lib.fp4_quantize(ctx, _dev(bits), axis, prescale=torch.from_numpy(p).cuda())
    torch.cuda.synchronize()
    _check_dense(q, O.absmax_quantize(O.bf16_bits_to_f64(bits), axis, prescale=p))


def test_Q_on_chosen_float32_values(lib, ctx):
    """Drive the encoder with arbitrary float32 inputs: x = 1 and a prescale vector of the probe
    values; one probe is 6 so that gamma = 1 and the scaled value is the probe itself.  Probes:
    every threshold of the chain, its float32 neighbours, grid points, zeros, tiny and large."""
    probes = [6.0]
    for t in O.LUT_THRESHOLDS:
        t32 = np.float32(t)
        probes += [t32, np.nextafter(t32, np.float32(-np.inf)), np.nextafter(t32, np.float32(np.inf)),
                   np.nextafter(np.nextafter(t32, np.float32(-np.inf)), np.float32(-np.inf)),
                   np.nextafter(np.nextafter(t32, np.float32(np.inf)), np.float32(np.inf))]
    probes += list(O.LUT_VALUES) + [0.0, -0.0, 1e-30, -1e-30, 1e-42, -1e-42, 5.9999995, -5.9999995, 0.1, -0.1]
    rng = np.random.default_rng(3)
    probes += list(rng.uniform(-6, 6, 384 - len(probes)))
    p = np.array(probes, dtype=np.float32)
    assert p.size == 384 and np.abs(p).max() == 6.0
    ones = np.full((128, 384), 0x3F80, dtype=np.uint16)
    q = lib.fp4_quantize(ctx, _dev(ones), 0, prescale=torch.from_numpy(p).cuda())
    torch.cuda.synchronize()
    got = O.unpack_nibbles(q.codes.cpu().numpy())
    want = O.lut_quantize(p)
    np.testing.assert_array_equal(got[0], want)
    np.testing.assert_array_equal(got, np.broadcast_to(want, got.shape))
    assert not (got == 8).any()


def test_Q_on_every_bf16_value(lib, ctx):
    """All finite BF16 patterns of magnitude <= 6 in one tensor whose rows all have amax 6."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    v = O.bf16_bits_to_f64(bits)
    keep = bits[np.isfinite(v) & (np.abs(v) <= 6.0)]
    cols = 256
    rows = -(-keep.size // (cols - 1))
    rows = -(-rows // 128) * 128
    x = np.zeros((rows, cols), dtype=np.uint16)
    x[:, 0] = 0x40C0                                   # 6.0 in every row -> gamma = 1
    body = np.zeros(rows * (cols - 1), dtype=np.uint16)
    body[:keep.size] = keep
    x[:, 1:] = body.reshape(rows, cols - 1)
    q = lib.fp4_quantize(ctx, _dev(x), 0)
    torch.cuda.synchronize()
    _check_dense(q, O.absmax_quantize(O.bf16_bits_to_f64(x), 0))


@pytest.mark.parametrize("shape,alpha,dist", [((128, 128), 0.99, "normal"), ((256, 384), 0.97, "student_t3"),
                                              ((384, 1152), 0.999, "laplace"), ((1024, 640), 0.99, "normal")])
def test_occ_quantize_matches_oracle(lib, ctx, shape, alpha, dist):
    cfg = WL.Config(50, "t", shape[0], (), dist, 3, 40.0, "channels_count", (alpha,))
    bits = WL.activations(cfg, shape[1], seed=1, layer=shape[0])
    ctx.status.zero_()
    q = lib.fp4_quantize(ctx, _dev(bits), 0, alpha=alpha)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha)
    _check_sparse(q, ref)
    _check_dense(q, ref)


def test_occ_tall_tensor_many_rows_per_block(lib, ctx):
    """81 920 rows of 128: more rows per histogram block than its shared row slots hold at once, so
    the row extremes are reduced in several batches."""
    rows, cols, alpha = 81920, 128, 0.999
    cfg = WL.Config(51, "tall", rows, (), "normal", 2, 40.0, "channels_count", (alpha,))
    bits = WL.activations(cfg, cols, seed=2, layer=7)
    big = lib.Context(0, int(lib.load_library().fp4_workspace_bytes(rows, cols, 128)))
    big.status.zero_()
    q = lib.fp4_quantize(big, _dev(bits), 0, alpha=alpha)
    torch.cuda.synchronize()
    assert big.read_status() == 0
    ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha)
    _check_sparse(q, ref)
    _check_dense(q, ref)
    big.close()


def test_occ_with_heavy_ties_and_zeros(lib, ctx):
    """Few distinct values: thresholds sit on big ties (entries equal to a threshold carry no
    residual), one bin holds far more than 2^16 entries, and lo is a zero."""
    rng = np.random.default_rng(8)
    vals = np.array([0.0, -0.0, 0.5, 1.0, -1.0, 2.5, -3.0, 64.0], dtype=np.float32)
    prob = np.array([0.86, 0.05, 0.03, 0.02, 0.005, 0.02, 0.005, 0.01])
    a = rng.choice(vals, size=(512, 1024), p=prob)
    bits = WL.to_bf16_bits(a)
    for alpha in (0.99, 0.97):
        q = lib.fp4_quantize(ctx, _dev(bits), 0, alpha=alpha)
        torch.cuda.synchronize()
        ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha)
        _check_sparse(q, ref)
        _check_dense(q, ref)


def test_occ_values_outside_the_histogram_window(lib, ctx):
    """The histogram kernel keeps shared counters for a window of exponents chosen from the first
    elements each block sees; everything else must still be counted exactly.  Here the head of the
    tensor is small, the rest is a million times larger, and tiny / subnormal values are sprinkled in."""
    rng = np.random.default_rng(12)
    a = rng.standard_normal((1024, 2048)).astype(np.float32)
    a[:640] *= np.float32(1e-3)
    a[640:] *= np.float32(1e3)
    a[700:, 17] *= np.float32(1e4)
    tiny = rng.random(a.shape) < 0.01
    a[tiny] = (rng.standard_normal(int(tiny.sum())) * 1e-30).astype(np.float32)
    a[rng.random(a.shape) < 0.001] = np.float32(1e-39)          # below the smallest normal BF16
    bits = WL.to_bf16_bits(a)
    for alpha in (0.999, 0.9):
        ctx.status.zero_()
        q = lib.fp4_quantize(ctx, _dev(bits), 0, alpha=alpha)
        torch.cuda.synchronize()
        assert ctx.read_status() == 0
        ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha)
        _check_sparse(q, ref)
        _check_dense(q, ref)


def _occ_equals_oracle(lib, c, bits, alpha):
    c.status.zero_()
    q = lib.fp4_quantize(c, _dev(bits), 0, alpha=alpha)
    torch.cuda.synchronize()
    assert c.read_status() == 0
    ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha)
    _check_sparse(q, ref)
    _check_dense(q, ref)


@pytest.mark.parametrize("kind", ["positive", "negative", "relu", "two_scales", "constant", "tiny"])
def test_selection_on_tensors_whose_bulk_is_not_around_zero(lib, ctx, kind):
    """One-signed tensors (both thresholds on one side of zero), a tensor with more exact zeros than
    the clamped share (lo = 0), rows of very different scale, a constant tensor and one no larger than
    the sample of the selection."""
    rng = np.random.default_rng(32)
    a = rng.standard_normal((256, 1024)).astype(np.float32)
    if kind == "positive":
        a = np.abs(a) + np.float32(0.5)
    elif kind == "negative":
        a = -np.abs(a) * np.float32(100.0) - np.float32(1.0)
    elif kind == "relu":
        a = np.maximum(a, np.float32(0.0))
    elif kind == "two_scales":
        a[::2] *= np.float32(1e-4)
        a[1::2] *= np.float32(50.0)
    elif kind == "constant":
        a[:] = np.float32(-1.5)
    else:
        a = np.ascontiguousarray(a[:128, :128])
    bits = WL.to_bf16_bits(a)
    for alpha in (0.99, 0.97, 0.9999):
        if round((1.0 - alpha) * a.size) < 1:
            continue
        _occ_equals_oracle(lib, ctx, bits, alpha)


def test_config0_activation_and_weight(lib, ctx):
    cfg = WL.CONFIGS[0]
    a_bits = WL.activations(cfg, 1024)
    w_bits = WL.weights(cfg, 1024, 1024)
    qa = lib.fp4_quantize(ctx, _dev(a_bits), 0, alpha=0.99)
    qw = lib.fp4_quantize(ctx, _dev(w_bits), 1)
    torch.cuda.synchronize()
    ra = O.occ_quantize(O.bf16_bits_to_f64(a_bits), 0.99)
    assert ra.n_tail == 2621
    _check_sparse(qa, ra)
    _check_dense(qa, ra)
    _check_dense(qw, O.absmax_quantize(O.bf16_bits_to_f64(w_bits), 1))
    # the bound that sizes the sparse buffers
    assert int(qa.nnz.item()) <= 2 * ra.n_tail == qa.sparse_cap


def test_run_to_run_determinism(lib, ctx):
    cfg = WL.CONFIGS[0]
    x = _dev(WL.activations(cfg, 1024))
    a = lib.fp4_quantize(ctx, x, 0, alpha=0.99)
    b = lib.fp4_quantize(ctx, x, 0, alpha=0.99)
    torch.cuda.synchronize()
    for name in ("codes", "codes_t", "amax", "thresholds", "csr_rowptr", "csr_col", "csr_val", "csc_colptr",
                 "csc_row", "csc_val", "nnz"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


@pytest.mark.parametrize("bad", [0x7F80, 0xFF80, 0x7FC0])          # +inf, -inf, NaN
def test_non_finite_inputs_raise_the_status_bit(lib, ctx, bad):
    """An infinity or a NaN anywhere in the input sets FP4_DEV_NONFINITE (outputs are then unspecified
    but every write stays in bounds); finite inputs leave the word at zero."""
    rng = np.random.default_rng(bad)
    bits = WL.to_bf16_bits(rng.standard_normal((256, 384)).astype(np.float32))
    dirty = bits.copy()
    dirty[200, 301] = bad
    for x, want in ((bits, 0), (dirty, lib.FP4_DEV_NONFINITE)):
        for axis, alpha in ((0, 1.0), (1, 1.0), (0, 0.99)):
            ctx.status.zero_()
            lib.fp4_quantize(ctx, _dev(x), axis, alpha=alpha)
            torch.cuda.synchronize()
            assert ctx.read_status() & lib.FP4_DEV_NONFINITE == want, (axis, alpha)
    # through the layer: a bad output gradient is seen by the backward's quantiser
    a_bits, w_bits, dy_bits = WL.small_case(256, 384, 256, seed=3)
    ctx.status.zero_()
    _, sa, sw = lib.fp4_linear_fwd(ctx, _dev(a_bits), _dev(w_bits), 0.99)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    dy_bits = dy_bits.copy()
    dy_bits[17, 5] = bad
    lib.fp4_linear_bwd(ctx, _dev(dy_bits), _dev(w_bits), sa, sw)
    torch.cuda.synchronize()
    assert ctx.read_status() & lib.FP4_DEV_NONFINITE


def test_host_side_argument_errors(lib, ctx):
    x = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_quantize(ctx, x[:, :64].contiguous(), 0)
    assert e.value.code == -2                                   # shape
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_quantize(ctx, x, 0, alpha=0.4, out=lib.QTensor(128, 128, 0, x.device, 64))
    assert e.value.code == -3                                   # alpha
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_quantize(ctx, x, 1, alpha=0.99, out=lib.QTensor(128, 128, 1, x.device, 1000))
    assert e.value.code == -7                                   # clamp needs token-wise scaling
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_quantize(ctx, x, 0, alpha=0.99, out=lib.QTensor(128, 128, 0, x.device, 10))
    assert e.value.code == -8                                   # capacity below 2 * n_tail
    small = lib.Context(0, 1024)
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_quantize(small, x, 0)
    assert e.value.code == -5                                   # workspace
    small.close()


@pytest.mark.parametrize("shape,alpha,dist", [((128, 128), 0.99, "normal"), ((256, 384), 0.97, "student_t3"),
                                              ((1024, 640), 0.999, "laplace")])
def test_magnitude_quantile_variant_matches_oracle(lib, shape, alpha, dist):
    """FP4_QUANTILE_ABS: one threshold on |x| (a variant outside the paper) -- thresholds, codes, amax
    and the sparse residual bit for bit; the default mode of another context is untouched."""
    cfg = WL.Config(52, "t", shape[0], (), dist, 3, 40.0, "channels_count", (alpha,))
    bits = WL.activations(cfg, shape[1], seed=3, layer=shape[0])
    c = lib.Context(0, 256 << 20)
    c.set_quantile_mode(lib.FP4_QUANTILE_ABS)
    q = lib.fp4_quantize(c, _dev(bits), 0, alpha=alpha)
    torch.cuda.synchronize()
    assert c.read_status() == 0
    ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha, quantile="abs")
    assert ref.lo == -ref.hi
    _check_sparse(q, ref)
    _check_dense(q, ref)
    c.set_quantile_mode(lib.FP4_QUANTILE_SIGNED)
    q = lib.fp4_quantize(c, _dev(bits), 0, alpha=alpha)
    torch.cuda.synchronize()
    _check_sparse(q, O.occ_quantize(O.bf16_bits_to_f64(bits), alpha))
    with pytest.raises(lib.Fp4Error):
        c.set_quantile_mode(7)
    c.close()


def test_magnitude_quantile_with_ties_and_a_zero_threshold(lib):
    rng = np.random.default_rng(21)
    vals = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -3.0, 64.0], dtype=np.float32)
    for prob, alpha in (([0.5, 0.3, 0.05, 0.05, 0.05, 0.03, 0.02], 0.9),        # t = 0.5 sits on a big tie
                        ([0.6, 0.37, 0.01, 0.01, 0.005, 0.003, 0.002], 0.99)):   # t = 0: lo must be +0
        a = rng.choice(vals, size=(256, 512), p=prob)
        bits = WL.to_bf16_bits(a)
        c = lib.Context(0, 256 << 20)
        c.set_quantile_mode(lib.FP4_QUANTILE_ABS)
        q = lib.fp4_quantize(c, _dev(bits), 0, alpha=alpha)
        torch.cuda.synchronize()
        ref = O.occ_quantize(O.bf16_bits_to_f64(bits), alpha, quantile="abs")
        _check_sparse(q, ref)
        _check_dense(q, ref)
        c.close()


def _check_token_mode(q, ref):
    th = q.thresholds_rows.cpu().numpy()
    rows = ref.rows
    np.testing.assert_array_equal(th[0:2 * rows:2], ref.lo_rows.astype(np.float32))
    np.testing.assert_array_equal(th[1:2 * rows:2], ref.hi_rows.astype(np.float32))
    assert not (np.signbit(th) & (th == 0)).any()        # a zero threshold is +0
    nnz = int(q.nnz.item())
    rowptr, col, val = ref.csr
    colptr, row, cval = ref.csc
    assert nnz == rowptr[-1]
    np.testing.assert_array_equal(q.csr_rowptr.cpu().numpy(), rowptr)
    np.testing.assert_array_equal(q.csr_col.cpu().numpy()[:nnz], col)
    np.testing.assert_array_equal(q.csr_val.cpu().numpy()[:nnz], val)
    np.testing.assert_array_equal(q.csc_colptr.cpu().numpy(), colptr)
    np.testing.assert_array_equal(q.csc_row.cpu().numpy()[:nnz], row)
    np.testing.assert_array_equal(q.csc_val.cpu().numpy()[:nnz], cval)
    _check_dense(q, ref)


@pytest.mark.parametrize("shape,alpha,dist", [((128, 128), 0.97, "normal"), ((256, 384), 0.99, "student_t3"),
                                              ((384, 1152), 0.999, "laplace"), ((128, 2048), 0.9, "normal")])
def test_per_token_thresholds_variant_matches_oracle(lib, shape, alpha, dist):
    """FP4_QUANTILE_TOKEN: every row clamped at its own order statistics (a variant outside the paper):
    2 * rows thresholds, codes, amax and the sparse residual bit for bit."""
    cfg = WL.Config(53, "t", shape[0], (), dist, 3, 40.0, "channels_count", (alpha,))
    bits = WL.activations(cfg, shape[1], seed=4, layer=shape[0])
    bits[5, :] = 0                                       # a zero row: thresholds +0, nothing clamped
    bits[6, ::2] = bits[6, 1::2]                         # a row of pairs: ties
    c = lib.Context(0, 256 << 20)
    c.set_quantile_mode(lib.FP4_QUANTILE_TOKEN)
    q = lib.fp4_quantize(c, _dev(bits), 0, alpha=alpha)
    torch.cuda.synchronize()
    assert c.read_status() == 0
    _check_token_mode(q, O.occ_quantize(O.bf16_bits_to_f64(bits), alpha, quantile="token"))
    c.close()


def test_per_token_thresholds_through_the_layer(lib):
    """Forward and backward with thresholds per token: the residual, its compensation in both passes
    and the saved operands follow the oracle's variant."""
    from test_gpu_linear import assert_close_f32
    M, K, N, alpha = 256, 384, 256, 0.98
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=17)
    f = O.linear_fwd(a_bits, w_bits, alpha, quantile="token")
    b = O.linear_bwd(dy_bits, w_bits, f)
    c = lib.Context(0, 512 << 20)
    c.set_quantile_mode(lib.FP4_QUANTILE_TOKEN)
    y32, sa, sw = lib.fp4_linear_fwd(c, _dev(a_bits), _dev(w_bits), alpha, out_f32=True)
    da32, dw32 = lib.fp4_linear_bwd(c, _dev(dy_bits), _dev(w_bits), sa, sw, out_f32=True)
    torch.cuda.synchronize()
    assert c.read_status() == 0
    _check_token_mode(sa, f.qa)
    assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y")
    assert_close_f32(da32.cpu().numpy(), b.da, b.da, None, "dA")
    assert_close_f32(dw32.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, "dW")
    c.close()
