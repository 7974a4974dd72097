"""GPU parity of fp4_gemm against the oracle: exact accumulators and the two de-scales."""
import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(lib):
    c = lib.Context(0, 64 << 20)
    yield c
    c.close()


def _codes(rng, rows, cols):
    c = rng.integers(0, 16, (rows, cols), dtype=np.uint8)
    c[c == 8] = 0                      # the library never writes a negative-zero code
    return c


def _run(lib, ctx, ca, cb, kind, **kw):
    a = torch.from_numpy(O.pack_nibbles(ca)).cuda()
    b = torch.from_numpy(O.pack_nibbles(cb)).cuda()
    ctx.status.zero_()
    out = lib.fp4_gemm(ctx, a, b, gemm_kind=kind, **kw)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    return out


KINDS = [0, 1]          # FP4_GEMM_MXF4, FP4_GEMM_F8F6F4
SHAPES = [(128, 128, 128), (128, 256, 256), (256, 384, 640), (384, 640, 1152), (512, 1024, 4096)]


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("shape", SHAPES)
def test_accumulators_are_exact(lib, ctx, kind, shape):
    """Every product is a multiple of 1/4 and the sums stay below 2^24 quarter units, so the
    fp32 accumulators must equal the oracle's integers exactly, in any summation order."""
    I, J, C = shape
    rng = np.random.default_rng(I + J + C + kind)
    ca, cb = _codes(rng, I, C), _codes(rng, J, C)
    got = _run(lib, ctx, ca, cb, kind).cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(got, O.gemm_codes(ca, cb))


@pytest.mark.parametrize("kind", KINDS)
def test_extreme_codes_long_contraction(lib, ctx, kind):
    """All +-6 operands over the longest contraction of the workloads (16384): |acc| up to 589824."""
    rng = np.random.default_rng(5)
    I, J, C = 128, 128, 16384
    ca = np.where(rng.random((I, C)) < 0.5, 0x7, 0xF).astype(np.uint8)
    cb = np.full((J, C), 0x7, dtype=np.uint8)
    cb[1::2] = 0xF
    ca[0] = 0x7                          # one row with no cancellation at all
    got = _run(lib, ctx, ca, cb, kind).cpu().numpy().astype(np.float64)
    ref = O.gemm_codes(ca, cb)
    assert abs(ref[0, 0]) == 36.0 * C
    np.testing.assert_array_equal(got, ref)


@pytest.mark.parametrize("kind", KINDS)
def test_descales_fp32_and_bf16(lib, ctx, kind):
    rng = np.random.default_rng(9)
    I, J, C = 256, 384, 512
    ca, cb = _codes(rng, I, C), _codes(rng, J, C)
    ra = (rng.random(I) * 4 + 0.1).astype(np.float32)
    cam = (rng.random(J) * 0.1 + 0.01).astype(np.float32)
    acc = O.gemm_codes(ca, cb)
    six = np.float32(6)
    want32 = ((acc.astype(np.float32) * (ra / six)[:, None]).astype(np.float32) * (cam / six)[None, :]).astype(np.float32)
    out = _run(lib, ctx, ca, cb, kind, row_amax=torch.from_numpy(ra).cuda(), col_amax=torch.from_numpy(cam).cuda())
    np.testing.assert_array_equal(out.cpu().numpy(), want32)     # two float multiplies, in this order
    outb = _run(lib, ctx, ca, cb, kind, row_amax=torch.from_numpy(ra).cuda(), col_amax=torch.from_numpy(cam).cuda(),
                out_f32=False)
    wantb = torch.from_numpy(want32).to(torch.bfloat16)
    assert torch.equal(outb.cpu(), wantb)


@pytest.mark.parametrize("kind_name", ["FP4_GEMM_F8F6F4_A8", "FP4_GEMM_F8F6F4_B8", "FP4_GEMM_F8F6F4_A8B8"])
@pytest.mark.parametrize("shape", [(128, 256, 256), (384, 640, 1152), (256, 512, 4096)])
def test_mixed_e4m3_operands(lib, ctx, kind_name, shape):
    """E4M3 bytes as one or both operands of the byte-container kind (the W4A8 / W8A4 settings).
    The products are not all on one binary scale, so the fp32 accumulation is compared at the
    GEMM tolerance of 1e-3 of the summed magnitudes, and is in fact far closer."""
    I, J, C = shape
    kind = getattr(lib, kind_name)
    a8 = kind_name in ("FP4_GEMM_F8F6F4_A8", "FP4_GEMM_F8F6F4_A8B8")
    b8 = kind_name in ("FP4_GEMM_F8F6F4_B8", "FP4_GEMM_F8F6F4_A8B8")
    rng = np.random.default_rng(I + J + C + len(kind_name))

    def fp8(rows):
        c = rng.integers(0, 256, (rows, C), dtype=np.uint8)
        c[(c & 0x7F) == 0x7F] = 0x38                       # no NaN codes
        return c

    ca = fp8(I) if a8 else _codes(rng, I, C)
    cb = fp8(J) if b8 else _codes(rng, J, C)
    va = O.e4m3_decode(ca) if a8 else O.e2m1_decode(ca)
    vb = O.e4m3_decode(cb) if b8 else O.e2m1_decode(cb)
    a = torch.from_numpy(ca if a8 else O.pack_nibbles(ca)).cuda()
    b = torch.from_numpy(cb if b8 else O.pack_nibbles(cb)).cuda()
    ra = (rng.random(I) * 4 + 0.1).astype(np.float32)
    cam = (rng.random(J) * 0.1 + 0.01).astype(np.float32)
    ctx.status.zero_()
    raw = lib.fp4_gemm(ctx, a, b, gemm_kind=kind)
    out = lib.fp4_gemm(ctx, a, b, torch.from_numpy(ra).cuda(), torch.from_numpy(cam).cuda(), gemm_kind=kind)
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    ref = va @ vb.T
    mag = np.abs(va) @ np.abs(vb).T
    err = np.abs(raw.cpu().numpy().astype(np.float64) - ref)
    assert (err <= 1e-3 * mag).all()
    assert (err <= 2.0 ** -18 * mag).all()                 # what fp32 accumulation of exact products gives
    d_row = (ra / np.float32(448 if a8 else 6)).astype(np.float32)
    d_col = (cam / np.float32(448 if b8 else 6)).astype(np.float32)
    want = (raw.cpu().numpy() * d_row[:, None]).astype(np.float32) * d_col[None, :]
    np.testing.assert_array_equal(out.cpu().numpy(), want.astype(np.float32))   # the two de-scales, in this order


def test_argument_errors(lib, ctx):
    a = torch.zeros((128, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_gemm(ctx, a[:100], a)                     # I not a multiple of 128
    assert e.value.code == -2
    with pytest.raises(lib.Fp4Error) as e:
        lib.fp4_gemm(ctx, a, a, gemm_kind=7)
    assert e.value.code == -7


def test_a_wait_that_runs_out_raises_timeout_and_leaves_the_context_usable(lib):
    """Every device-side wait of the GEMM is bounded.  With the debug switches of the library the
    producer of the first CTA leaves out one fill of the shared-memory ring while the limit of the
    waits is 1 ms: the consumer's wait runs out, the kernel raises FP4_DEV_TIMEOUT, frees its tensor
    memory and returns; the next GEMM on the same context is exact again."""
    rng = np.random.default_rng(77)
    ca, cb = _codes(rng, 256, 4096), _codes(rng, 256, 4096)          # 16 fills per tile (MXF4), 32 (byte containers)
    want = O.gemm_codes(ca, cb)
    a = torch.from_numpy(O.pack_nibbles(ca)).cuda()
    b = torch.from_numpy(O.pack_nibbles(cb)).cuda()
    c = lib.Context(0, 64 << 20)
    for kind in KINDS:
        c.debug_set(lib.binding.FP4_DEBUG_WAIT_LIMIT_US, 1000)
        c.debug_set(lib.binding.FP4_DEBUG_SKIP_FILL, 6)
        c.status.zero_()
        lib.fp4_gemm(c, a, b, gemm_kind=kind)
        torch.cuda.synchronize()                                       # the kernel returned
        assert c.read_status() & lib.FP4_DEV_TIMEOUT
        c.debug_set(lib.binding.FP4_DEBUG_SKIP_FILL, -1)
        c.debug_set(lib.binding.FP4_DEBUG_WAIT_LIMIT_US, 0)
        c.status.zero_()
        out = lib.fp4_gemm(c, a, b, gemm_kind=kind)
        torch.cuda.synchronize()
        assert c.read_status() == 0
        np.testing.assert_array_equal(out.cpu().numpy().astype(np.float64), want)
    c.close()
