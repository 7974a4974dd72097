"""GPU parity of fp4_linear_fwd / fp4_linear_bwd against the oracle.

Tolerance (fp32-accumulated results against the double oracle): an output that is the sum of
an FP4 branch and a compensation branch must satisfy
    |gpu - oracle| <= 1e-3 * (|fp4 branch| + |compensation branch|)
in float output mode.  In BF16 output mode the stored value must be the BF16 rounding of the
oracle value, or a neighbouring BF16 number where the oracle value lies within 1e-3 (relative)
of a rounding boundary; at least 99 % of the values must be the rounding itself.  Where the two
branches nearly cancel, "relative" is taken against |fp4 branch| + |compensation branch| as in
float mode (callers that pass the branches), since that is what the fp32 sum before the rounding
is held to.

Accumulation floor of the dense tail.  With a heavy residual the hot columns' products are added
inside the tensor cores, whose fp32 accumulation rounds toward zero: up to 24 additions (6 blocks
of 64 FP16 columns, 4 instructions each), each off by at most 2^-23 of the running sum, plus 2^-21
from the two-term FP16 splits, i.e. at most 4e-6 of sum_k |dA[m,k]| |W[k,n]|.  Where both branches
cancel to a thousandth of their terms that floor can exceed 1e-3 of the branches, so the cases that
can take the tail add TAIL_FLOOR * (|dA| |W|)[m,n] to the allowance.  The weight operand of the tail
is W / d_W in FP16, whose smallest step (with the scaled low half) is 2^-31 of a unit: a weight
more than ten orders of magnitude below its column's largest is not resolved, hence the second term
of `tail_floor`, 2^-33 d_W[n] sum_k |dA[m,k]| (1e-9 of the first for ordinary weights).

Accumulation floor of the per-entry compensation.  The compensation products are accumulated in
fp32 (one fused multiply-add per residual entry, then the sum with the FP4 branch and the DGE
factor): by the standard bound for a sum of n terms its error is at most (n + 4) * 2^-24 of the
sum of the terms' magnitudes.  That is far below 1e-3 of the branches unless the terms cancel
by more than four orders of magnitude, which the randomised runs do meet (one output in 4e8: 83
terms of up to 8.5e-3 adding up to 4e-9 beside an FP4 branch of exactly 0, where the GPU's value
is the fp32 sum to the last bit); `fp32_sum_floor` gives that bound for the cases drawn at random.
"""
import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

pytestmark = pytest.mark.gpu
RTOL = 1e-3
TAIL_FLOOR = 4e-6


def tail_floor(f: "O.Forward", w_bits):
    """Allowance for the dense tail: TAIL_FLOOR * (|dA| |W|) for the tensor cores' accumulation and the
    FP16 splits, plus the absolute resolution of the weight operand W / d_W in FP16 (2^-31 of a unit
    with the scaled low half; the operand is 4 W / d_W against dA / (4 d_A)), which matters only for
    weights ten orders of magnitude below their column's largest."""
    r = np.abs(f.qa.residual)
    return (TAIL_FLOOR * (r @ np.abs(O.bf16_bits_to_f64(w_bits)))
            + 2.0 ** -33 * r.sum(axis=1)[:, None] * f.qw.descale.astype(np.float64)[None, :])


def fp32_sum_floor(residual, dense_abs, transpose=False):
    """(n + 4) 2^-24 sum |terms| for the fp32-accumulated product of the sparse residual [M x K] with
    a dense matrix: residual @ dense [M x N] (n = entries of the row), or with `transpose`
    residual^T @ dense [K x N] (n = entries of the column)."""
    r = np.abs(residual.T if transpose else residual)
    n = np.count_nonzero(r, axis=1).astype(np.float64)
    return (n[:, None] + 4.0) * 2.0 ** -24 * (r @ dense_abs)


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0, 1 << 30)
    yield c
    c.close()


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def assert_close_f32(got, want, branch_a, branch_b=None, what="", floor=0.0):
    scale = np.abs(branch_a) + (0 if branch_b is None else np.abs(branch_b))
    err = np.abs(got.astype(np.float64) - want)
    bad = err > RTOL * scale + floor + 1e-300
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, worst {np.max(err / (scale + 1e-300))}"


def assert_bf16_rounding(got_bf16: torch.Tensor, want, what="", branch_a=None, branch_b=None, floor=0.0):
    got = got_bf16.float().cpu().numpy().astype(np.float64)
    r = O.f64_to_bf16_f64(want)
    exact = got == r
    scale = np.abs(want) if branch_a is None else np.abs(branch_a) + (0 if branch_b is None else np.abs(branch_b))
    # a neighbouring BF16 value is accepted only if the oracle value is within RTOL of the midpoint
    near = np.abs(got - want) <= np.abs(r - want) + RTOL * scale + floor
    ok = exact | near
    assert ok.all(), f"{what}: {np.sum(~ok)} of {ok.size} values are not the BF16 rounding of the oracle"
    assert exact.mean() > 0.99, f"{what}: only {exact.mean():.4f} match the rounding exactly"


def _saved_matches(sa, sw, f: O.Forward):
    np.testing.assert_array_equal(sa.codes.cpu().numpy(), f.qa.packed())
    np.testing.assert_array_equal(sa.codes_t.cpu().numpy(), f.qa.packed_t())
    np.testing.assert_array_equal(sa.amax.cpu().numpy(), f.qa.amax)
    np.testing.assert_array_equal(sw.codes.cpu().numpy(), f.qw.packed())
    np.testing.assert_array_equal(sw.codes_t.cpu().numpy(), f.qw.packed_t())
    np.testing.assert_array_equal(sw.amax.cpu().numpy(), f.qw.amax)


CASES = [
    # M, K, N, alpha, gemm kind
    (128, 128, 128, 0.99, 0),
    (256, 384, 640, 0.97, 0),
    (384, 640, 384, 0.999, 1),
    (128, 256, 128, 1.0, 0),
    (256, 1152, 256, 0.99, 1),
]


@pytest.mark.parametrize("M,K,N,alpha,kind", CASES)
def test_forward_and_backward_match_oracle(lib, ctx, M, K, N, alpha, kind):
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=M + K + N)
    f = O.linear_fwd(a_bits, w_bits, alpha)
    b = O.linear_bwd(dy_bits, w_bits, f)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    ctx.status.zero_()
    y32, sa, sw = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind, out_f32=True)
    da32, dw32 = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind, out_f32=True)
    y16, _, _ = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind)
    da16, dw16 = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    _saved_matches(sa, sw, f)
    assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y")
    assert_close_f32(da32.cpu().numpy(), b.da, b.da, None, "dA")
    assert_close_f32(dw32.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, "dW")
    assert_bf16_rounding(y16, f.y, "Y")
    assert_bf16_rounding(da16, b.da, "dA")
    assert_bf16_rounding(dw16, b.dw, "dW")


def test_ste_switch_and_dge_parameters(lib, ctx):
    a_bits, w_bits, dy_bits = WL.small_case(128, 256, 128, seed=21)
    f = O.linear_fwd(a_bits, w_bits, 0.99)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    _, sa, sw = lib.fp4_linear_fwd(ctx, A, W, 0.99)
    for dge_on, k, clip in ((False, 5.0, 3.0), (True, 3.0, 2.0), (True, 7.0, 10.0)):
        b = O.linear_bwd(dy_bits, w_bits, f, dge_on=dge_on, k=k, clip=clip)
        _, dw = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, dge_on=dge_on, dge_k=k, dge_clip=clip, out_f32=True,
                                   want_da=False)
        torch.cuda.synchronize()
        assert_close_f32(dw.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, f"dW dge={dge_on} k={k}")


@pytest.mark.parametrize("M,K,N,hot,alpha", [
    (128, 256, 128, 40, 0.92),     # 40 nearly full columns
    (512, 256, 384, 20, 0.98),     # 20 nearly full columns of 512 entries: long columns, many rounds per warp
    (256, 384, 128, 3, 0.999),     # few entries: short columns only
    (1024, 512, 256, 200, 0.78),   # 200 full columns of 1024 entries: more than the dense class takes (160); the rest are long
    (1024, 256, 384, 12, 0.97),    # 12 full columns: dense class (two passes of 8), several chunks of tokens
])
def test_weight_gradient_compensation_column_classes(lib, ctx, M, K, N, hot, alpha):
    """The compensation of the weight gradient treats dense, long and short residual columns
    differently; all must give the oracle's sums, run to run identically."""
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=hot, alpha_outliers=hot)
    f = O.linear_fwd(a_bits, w_bits, alpha)
    b = O.linear_bwd(dy_bits, w_bits, f)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    ctx.status.zero_()
    _, sa, sw = lib.fp4_linear_fwd(ctx, A, W, alpha)
    _, dw = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, out_f32=True, want_da=False)
    _, dw_again = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, out_f32=True, want_da=False)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    counts = np.diff(sa.csc_colptr.cpu().numpy())
    if M >= 1024:
        assert (counts >= 512).sum() >= hot // 2                      # the case does reach the dense / long classes
    assert np.abs(b.s_comp).max() > 0
    assert_close_f32(dw.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, "dW")
    assert torch.equal(dw, dw_again)                                   # fixed summation order


@pytest.mark.parametrize("M,K,N,hot,alpha,kind", [
    (1024, 512, 256, 12, 0.97, 0),     # 12 hot columns: one block of the tail
    (1024, 512, 384, 100, 0.90, 0),    # 100 hot columns: two blocks; N is not a multiple of the tile width
    (1024, 512, 256, 200, 0.78, 0),    # more hot columns than the tail takes (128): the rest stay per-entry
    (1024, 256, 384, 70, 0.90, 1),     # the byte-container kind
    (512, 256, 128, 3, 0.97, 0),       # heavy residual but no hot column: an empty tail
])
def test_forward_dense_tail(lib, ctx, M, K, N, hot, alpha, kind):
    """Heavy residuals send their hot columns through the GEMM as FP16 contraction columns (two-term
    splits) and the other entries through the per-entry kernel: the sum must still be the oracle's
    Y, to the same bar as without a tail, and identical run to run."""
    a_bits, w_bits, _ = WL.small_case(M, K, N, seed=hot + 1, alpha_outliers=hot)
    f = O.linear_fwd(a_bits, w_bits, alpha)
    A, W = _dev(a_bits), _dev(w_bits)
    ctx.status.zero_()
    y32, sa, _ = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind, out_f32=True)
    y16, _, _ = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind)
    y16_again, _, _ = lib.fp4_linear_fwd(ctx, A, W, alpha, gemm_kind=kind)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    counts = np.diff(sa.csc_colptr.cpu().numpy())
    n_hot = int((counts >= max(M // 4, 512)).sum())
    assert (n_hot > 0) == (hot >= 12)                                   # the case is in the regime it names
    assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y", tail_floor(f, w_bits))
    assert_bf16_rounding(y16, f.y, "Y bf16", f.y_fp4, f.y_comp, tail_floor(f, w_bits))
    assert torch.equal(y16, y16_again)


def test_forward_dense_tail_with_e4m3_weights(lib, ctx):
    """W8A4 with a heavy residual: the tail's weight operand is divided by the E4M3 de-scale (amax / 448)."""
    M, K, N, hot, alpha = 1024, 256, 384, 20, 0.92
    a_bits, w_bits, _ = WL.small_case(M, K, N, seed=31, alpha_outliers=hot)
    f = O.linear_fwd(a_bits, w_bits, alpha, fmt_w="e4m3")
    ctx.status.zero_()
    y32, sa, _ = lib.fp4_linear_fwd(ctx, _dev(a_bits), _dev(w_bits), alpha, gemm_kind=lib.FP4_GEMM_F8F6F4, out_f32=True,
                                    fmt_w=lib.FP4_FORMAT_E4M3)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    assert int((np.diff(sa.csc_colptr.cpu().numpy()) >= 512).sum()) > 0
    assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y", tail_floor(f, w_bits))


def test_forward_dense_tail_falls_back_on_huge_outliers(lib, ctx):
    """A residual too large for the tail's FP16 operands (relative to its token's scale) switches the
    tail off on the device for that call; the per-entry kernel then adds every entry."""
    M, K, N = 1024, 256, 128
    a_bits, w_bits, _ = WL.small_case(M, K, N, seed=77, alpha_outliers=12)
    a = O.bf16_bits_to_f64(a_bits)
    counts_col = int(np.argmax(np.abs(a).mean(axis=0)))                 # a hot column
    a[5, counts_col] = 3.0e30
    a_bits = WL.to_bf16_bits(a.astype(np.float32))
    f = O.linear_fwd(a_bits, w_bits, 0.97)
    ctx.status.zero_()
    y32, _, _ = lib.fp4_linear_fwd(ctx, _dev(a_bits), _dev(w_bits), 0.97, out_f32=True)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y")


def test_reuse_quantised_weight(lib, ctx):
    a_bits, w_bits, _ = WL.small_case(128, 256, 256, seed=5)
    a2_bits, _, _ = WL.small_case(128, 256, 256, seed=6)
    W = _dev(w_bits)
    y1, sa, sw = lib.fp4_linear_fwd(ctx, _dev(a_bits), W, 0.99)
    y2, _, _ = lib.fp4_linear_fwd(ctx, _dev(a2_bits), W, 0.99, saved_w=sw, reuse_w=True)
    y2_fresh, _, _ = lib.fp4_linear_fwd(ctx, _dev(a2_bits), W, 0.99)
    torch.cuda.synchronize()
    assert torch.equal(y2, y2_fresh)


def test_reuse_quantised_activation(lib, ctx):
    """q/k/v-style sharing: a second weight applied to an activation that is already quantised."""
    a_bits, w_bits, dy_bits = WL.small_case(256, 384, 256, seed=9)
    _, w2_bits, _ = WL.small_case(256, 384, 256, seed=10)
    A, W1, W2, dY = _dev(a_bits), _dev(w_bits), _dev(w2_bits), _dev(dy_bits)
    _, sa, _ = lib.fp4_linear_fwd(ctx, A, W1, 0.99)
    y_shared, _, sw2 = lib.fp4_linear_fwd(ctx, A, W2, 0.99, saved_a=sa, reuse_a=True)
    da_s, dw_s = lib.fp4_linear_bwd(ctx, dY, W2, sa, sw2)
    y_fresh, sa2, sw2b = lib.fp4_linear_fwd(ctx, A, W2, 0.99)
    da_f, dw_f = lib.fp4_linear_bwd(ctx, dY, W2, sa2, sw2b)
    torch.cuda.synchronize()
    assert torch.equal(y_shared, y_fresh) and torch.equal(da_s, da_f) and torch.equal(dw_s, dw_f)


def test_linears_that_share_an_input_as_one_call(lib, ctx):
    """q/k/v-style grouping: with the group's weights stored side by side ([K x (N1 + N2 + N3)]) one
    call does the work of three.  Weights are scaled per output channel and dY for the weight
    gradient per output channel too, so Y of the fused call is the separate calls' Y bit for bit,
    column block by column block (heavy residual: dense tail included), and dW the same sums: equal
    bit for bit except where the tensor-core dense class groups its token ranges differently for a
    different N (fp32 additions of the same partial products: a few ulp).  dA of the fused call is the gradient with respect to the shared input -- the
    sum over the group, accumulated in fp32 inside one GEMM with dY quantised token-wise over the
    whole row -- and is held to the oracle's value for the fused linear."""
    M, K, alpha = 1024, 512, 0.97
    a_bits, w1, dy1 = WL.small_case(M, K, 256, seed=41, alpha_outliers=12)
    _, w2, dy2 = WL.small_case(M, K, 384, seed=42)
    _, w3, dy3 = WL.small_case(M, K, 128, seed=43)
    w_cat = np.ascontiguousarray(np.concatenate([w1, w2, w3], axis=1))
    dy_cat = np.ascontiguousarray(np.concatenate([dy1, dy2, dy3], axis=1))
    A = _dev(a_bits)
    ctx.status.zero_()
    y_cat, sa, sw = lib.fp4_linear_fwd(ctx, A, _dev(w_cat), alpha)
    da_cat, dw_cat = lib.fp4_linear_bwd(ctx, _dev(dy_cat), _dev(w_cat), sa, sw, out_f32=True)
    n0 = 0
    for w_bits, dy_bits in ((w1, dy1), (w2, dy2), (w3, dy3)):
        n1 = n0 + w_bits.shape[1]
        y, sa_g, sw_g = lib.fp4_linear_fwd(ctx, A, _dev(w_bits), alpha)
        _, dw = lib.fp4_linear_bwd(ctx, _dev(dy_bits), _dev(w_bits), sa_g, sw_g, out_f32=True, want_da=False)
        torch.cuda.synchronize()
        assert torch.equal(y_cat[:, n0:n1], y)
        got, want = dw_cat[:, n0:n1].double(), dw.double()
        assert ((got - want).abs() <= 1e-5 * want.abs().max()).all()
        assert (got == want).double().mean() > 0.9
        n0 = n1
    assert ctx.read_status() == 0
    f = O.linear_fwd(a_bits, w_cat, alpha)
    b = O.linear_bwd(dy_cat, w_cat, f)
    assert_close_f32(da_cat.cpu().numpy(), b.da, b.da, None, "dA of the fused linear")


def test_config0_full_layer(lib, ctx):
    """The small configuration in full: X[256 x 1024] with 8 outlier channels, alpha = 0.99, DGE on."""
    cfg = WL.CONFIGS[0]
    a_bits = WL.activations(cfg, 1024)
    w_bits = WL.weights(cfg, 1024, 1024)
    dy_bits = WL.output_grads(cfg, 1024)
    f = O.linear_fwd(a_bits, w_bits, 0.99)
    b = O.linear_bwd(dy_bits, w_bits, f)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    for kind in (0, 1):
        ctx.status.zero_()
        y32, sa, sw = lib.fp4_linear_fwd(ctx, A, W, 0.99, gemm_kind=kind, out_f32=True)
        da32, dw32 = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, gemm_kind=kind, out_f32=True)
        y16, _, _ = lib.fp4_linear_fwd(ctx, A, W, 0.99, gemm_kind=kind)
        torch.cuda.synchronize()
        assert ctx.read_status() == 0
        _saved_matches(sa, sw, f)
        assert_close_f32(y32.cpu().numpy(), f.y, f.y_fp4, f.y_comp, "Y")
        assert_close_f32(da32.cpu().numpy(), b.da, b.da, None, "dA")
        assert_close_f32(dw32.cpu().numpy(), b.dw, b.s_fp4 * b.dge, b.s_comp * b.dge, "dW")
        assert_bf16_rounding(y16, f.y, "Y")


def test_dge_factor_alone_on_every_scaled_weight(lib, ctx):
    """Q' of Eq. 8 (k = 5, cap 3.0) read by itself.  One token of sixes (de-scale exactly 1)
    against one row of dY of 0.75 (de-scale exactly 1/8) makes the weight-gradient sum S exactly
    6 * 6 / 8 = 4.5 everywhere (no clamp, no residual), so dW in float mode is 4.5 times the factor:
    it is held to 1e-5 relative of the oracle's closed form on every BF16 weight pattern of magnitude
    <= 6, under column scales gamma = 1, 2 and 1/4 (the scaled weight is formed in fp32 on both sides)."""
    M, K, N = 128, 256, 256
    pats = np.arange(0x0000, 0x40C1, dtype=np.uint16)                 # +0 ... +6.0
    pats = np.concatenate([pats, pats | np.uint16(0x8000)])           # and the negatives
    assert pats.size <= (K - 1) * N
    w = np.zeros((K, N), dtype=np.uint16)
    body = np.resize(pats, (K - 1) * N).reshape(K - 1, N)
    w[1:] = body
    w[0] = 0x40C0                                                      # 6.0 in every column: amax = 6, gamma = 1
    # other column scales: amax = 3 (gamma 2; patterns up to 3.0 only) and amax = 24 (gamma 1/4)
    w[0, 64:128] = 0x4040                                              # 3.0
    big = (w[1:, 64:128] & np.uint16(0x7FFF)) > 0x4040
    w[1:, 64:128][big] = 0x3F80                                        # 1.0 where the pattern would exceed the column's amax
    w[0, 128:192] = 0x41C0                                             # 24.0
    a = np.zeros((M, K), dtype=np.uint16)
    a[0] = 0x40C0                                                      # token 0: sixes
    dy = np.zeros((M, N), dtype=np.uint16)
    dy[0] = 0x3F40                                                     # 0.75
    f = O.linear_fwd(a, w, 1.0)
    b = O.linear_bwd(dy, w, f)
    assert np.all(b.s_fp4 == 4.5) and not np.any(b.s_comp)             # the sum is exact: dW is 4.5 times the factor
    A, W, dY = _dev(a), _dev(w), _dev(dy)
    ctx.status.zero_()
    _, sa, sw = lib.fp4_linear_fwd(ctx, A, W, 1.0)
    _, dw = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, out_f32=True, want_da=False)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    got = dw.cpu().numpy().astype(np.float64) / 4.5
    assert np.array_equal(b.dw, 4.5 * b.dge)
    rel = np.abs(got - b.dge) / b.dge
    assert rel.max() <= 1e-5, f"DGE factor off by {rel.max():.2e} relative"
    assert (b.dge == 3.0).sum() > 50 and (b.dge < 0.21).sum() > 100    # the cap and the grid points are both in the sample
    assert np.array_equal(got[b.dge == 3.0], b.dge[b.dge == 3.0])      # the cap is exact


def test_tensor_core_accumulation_stays_inside_its_floor(lib, ctx):
    """Measures what TAIL_FLOOR allows for.  120 hot columns whose residual entries alternate in
    sign against weights of one sign make the compensation branch cancel (sums of ~120 terms far
    below the sum of their magnitudes), which is where the tensor cores' truncating fp32 additions
    show.  Derivation of the floor: 24 additions per accumulator, each off by at most 2^-23 of the
    running sum, plus 2^-21 from the two-term FP16 splits: 3.4e-6 of sum |dA| |W|, rounded up to
    4e-6.  The forward (dense tail of the GEMM) and the weight gradient (dense columns, chunks of
    128 tokens) must both stay within half of TAIL_FLOOR beyond the fp32 rounding of the two
    branches; a constant that is too tight or a kernel that loses precision fails here."""
    assert 24 * 2.0 ** -23 + 2.0 ** -21 <= TAIL_FLOOR
    M, K, N, hot, alpha = 1024, 512, 384, 120, 0.85
    a_bits, w_bits, dy_bits = WL.small_case(M, K, N, seed=1234, alpha_outliers=hot)
    a = O.bf16_bits_to_f64(a_bits)
    # hot columns: magnitudes kept, signs alternating along the columns, so that a token's residual sums cancel
    col_energy = np.abs(a).sum(axis=0)
    hot_cols = np.argsort(col_energy)[-hot:]
    sign = np.where(np.arange(hot) % 2 == 0, 1.0, -1.0)
    a[:, hot_cols] = np.abs(a[:, hot_cols]) * sign[None, :]
    a_bits = WL.to_bf16_bits(a.astype(np.float32))
    w = np.abs(O.bf16_bits_to_f64(w_bits))                             # weights of one sign
    w_bits = WL.to_bf16_bits(w.astype(np.float32))
    dy = np.abs(O.bf16_bits_to_f64(dy_bits))
    dy[::2] *= -1.0                                                    # tokens alternate in sign: the sums over tokens cancel
    dy_bits = WL.to_bf16_bits(dy.astype(np.float32))
    f = O.linear_fwd(a_bits, w_bits, alpha)
    b = O.linear_bwd(dy_bits, w_bits, f)
    mags_y = np.abs(f.qa.residual) @ np.abs(O.bf16_bits_to_f64(w_bits))
    mags_w = np.abs(f.qa.residual).T @ np.abs(O.bf16_bits_to_f64(dy_bits))
    assert np.median(np.abs(f.y_comp) / mags_y) < 0.2                  # the compensation sums do cancel
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)
    ctx.status.zero_()
    y, sa, sw = lib.fp4_linear_fwd(ctx, A, W, alpha, out_f32=True)
    _, dw = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, out_f32=True, want_da=False)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    counts = np.diff(sa.csc_colptr.cpu().numpy())
    assert (counts >= 512).sum() >= 100                                # the dense paths are taken
    ulp = 2.0 ** -23
    err_y = np.abs(y.cpu().numpy().astype(np.float64) - f.y)
    allow_y = 0.5 * TAIL_FLOOR * mags_y + 8 * ulp * (np.abs(f.y_fp4) + np.abs(f.y_comp))
    assert (err_y <= allow_y).all(), f"forward tail: {np.max(err_y / (TAIL_FLOOR * mags_y + 1e-300)):.3f} of the floor"
    err_w = np.abs(dw.cpu().numpy().astype(np.float64) - b.dw)
    allow_w = (0.5 * TAIL_FLOOR * mags_w + 8 * ulp * (np.abs(b.s_fp4) + np.abs(b.s_comp))) * b.dge * (1 + 1e-5)
    # entries added per entry in fp32 (the scattered ones) get the ordinary summation bound on top
    allow_w += 64 * ulp * mags_w * b.dge
    assert (err_w <= allow_w).all(), f"weight gradient: {np.max(err_w / (TAIL_FLOOR * mags_w * b.dge + 1e-300)):.3f} of the floor"
