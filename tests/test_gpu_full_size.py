"""Parity at the full sizes of the workload list, through the same calls bench.py times.

The oracle cannot produce whole outputs at these sizes in seconds, so it is evaluated on
samples: thresholds, every amax, the residual count and the CSR row pointer are compared in
full (they are cheap vector operations), while codes, sparse entries and the outputs of the
three GEMMs are compared on sampled rows / columns / entries, each computed by the oracle's own
functions on the slice that determines it (a row of A with the tensor-wide thresholds, a column
of W, a row or column of dY with the folded de-scale vector).
"""
import numpy as np
import pytest
import torch

from oracle import fp4_oracle as O
from paper_2501_17116_b200 import workloads as WL

pytestmark = pytest.mark.gpu
RTOL = 1e-3

# (config index, linear name, alpha): an attention and an MLP linear of every layer set, both swept
# alphas of the 7B MLP block
CASES = [(1, "q", 0.999), (1, "gate", 0.999), (1, "down", 0.999),
         (2, "gate", 0.99), (2, "down", 0.99), (2, "gate", 0.999), (2, "down", 0.999),
         (3, "q", 0.9999),
         (4, "q", 0.99), (4, "gate", 0.99), (4, "down", 0.99)]


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _f32(bits):
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _nibbles_of_rows(packed_t_dev, rows):
    """codes_t is [cols x rows/2]: gather the codes of the given source rows -> [len(rows), cols]."""
    r = torch.as_tensor(rows, device="cuda")
    b = packed_t_dev[:, r // 2].cpu().numpy()                       # [cols, len(rows)]
    odd = (np.asarray(rows) % 2 == 1)[None, :]
    return np.where(odd, b >> 4, b & 0xF).T.astype(np.uint8)


def _close(got, want, scale, what, floor=0.0):
    err = np.abs(np.asarray(got, dtype=np.float64) - want)
    bad = err > RTOL * scale + floor + 1e-300
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance"


def _bf16(out16, rows, cols, want, scale, what, floor=0.0):
    """The BF16 output on the sampled entries: the rounding of the oracle value, or a neighbouring
    BF16 number where the oracle value lies within the tolerance of a rounding boundary."""
    got = out16[torch.as_tensor(rows, device="cuda")][:, torch.as_tensor(cols, device="cuda")].float().cpu().numpy()
    got = got.astype(np.float64)
    r = O.f64_to_bf16_f64(want)
    ok = (got == r) | (np.abs(got - want) <= np.abs(r - want) + RTOL * scale + floor)
    assert ok.all(), f"{what}: {np.sum(~ok)} of {ok.size} values are not the BF16 rounding of the oracle"
    assert (got == r).mean() > 0.99, f"{what}: only {(got == r).mean():.4f} match the rounding exactly"


@pytest.mark.parametrize("ci,lname,alpha", CASES)
def test_full_size_layer_matches_sampled_oracle(lib, ci, lname, alpha):
    cfg = WL.CONFIGS[ci]
    lin = next(l for l in cfg.linears if l.name == lname)
    M, K, N = cfg.M, lin.K, lin.N
    rng = np.random.default_rng(ci * 100 + K)
    a_bits = WL.activations(cfg, K)
    w_bits = WL.weights(cfg, K, N)
    dy_bits = WL.output_grads(cfg, N)
    A, W, dY = _dev(a_bits), _dev(w_bits), _dev(dy_bits)

    ctx = lib.Context.for_shape(M, K, N)
    y32, sa, sw = lib.fp4_linear_fwd(ctx, A, W, alpha, out_f32=True)
    da32, dw32 = lib.fp4_linear_bwd(ctx, dY, W, sa, sw, out_f32=True)
    # the BF16 outputs the benchmark times, in the form it times them: forward and backward captured
    # into a CUDA graph (after one plain call, as after the benchmark's warm-up) and replayed
    y16 = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    da16 = torch.empty((M, K), dtype=torch.bfloat16, device=A.device)
    dw16 = torch.empty((K, N), dtype=torch.bfloat16, device=A.device)
    sa2 = lib.QTensor(M, K, 0, A.device, lib.tail_capacity(M, K, alpha))
    sw2 = lib.QTensor(K, N, 1, A.device)

    def step():
        lib.fp4_linear_fwd(ctx, A, W, alpha, sa2, sw2, out=y16)
        lib.fp4_linear_bwd(ctx, dY, W, sa2, sw2, dA=da16, dW=dw16)

    step()
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            step()
    for t in (y16, da16, dw16):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert ctx.read_status() == 0
    del graph, sa2, sw2

    # ---- thresholds, counts, amax: in full -------------------------------------------------
    a32, w32, dy32 = _f32(a_bits), _f32(w_bits), _f32(dy_bits)
    n = M * K
    n_tail = O.tail_count(n, alpha)
    srt = np.sort(a32, axis=None)                                    # the order statistics of R7
    lo, hi = float(srt[n_tail]) + 0.0, float(srt[n - 1 - n_tail]) + 0.0
    del srt
    th = sa.thresholds.cpu().numpy()
    assert (float(th[0]), float(th[1])) == (lo, hi)
    out_mask = (a32 > hi) | (a32 < lo)
    assert int(sa.nnz.item()) == int(out_mask.sum()) <= 2 * n_tail
    rowptr = np.concatenate([[0], np.cumsum(out_mask.sum(axis=1))]).astype(np.int32)
    colptr = np.concatenate([[0], np.cumsum(out_mask.sum(axis=0))]).astype(np.int32)
    np.testing.assert_array_equal(sa.csr_rowptr.cpu().numpy(), rowptr)
    np.testing.assert_array_equal(sa.csc_colptr.cpu().numpy(), colptr)
    amax_a = np.abs(np.clip(a32, np.float32(lo), np.float32(hi))).max(axis=1)
    amax_w = np.abs(w32).max(axis=0)
    np.testing.assert_array_equal(sa.amax.cpu().numpy(), amax_a)
    np.testing.assert_array_equal(sw.amax.cpu().numpy(), amax_w)
    _, d_a = O.absmax_scales(amax_a)
    _, d_w = O.absmax_scales(amax_w)

    # ---- sampled rows of A: codes (both layouts), CSR entries ---------------------------------
    hot_cols = np.argsort(out_mask.sum(axis=0))[-4:]
    rows = np.unique(np.concatenate([rng.choice(M, 24, replace=False), [0, M - 1, 63, 64]]))
    a_rows = O.bf16_bits_to_f64(a_bits[rows])
    a_c, resid = O.occ_split(a_rows, lo, hi)
    qa = O.absmax_quantize(a_c, 0)
    np.testing.assert_array_equal(sa.codes[torch.as_tensor(rows, device="cuda")].cpu().numpy(), qa.packed())
    np.testing.assert_array_equal(_nibbles_of_rows(sa.codes_t, rows), qa.codes)
    csr_col, csr_val = sa.csr_col.cpu().numpy(), sa.csr_val.cpu().numpy()
    for i, m in enumerate(rows):
        seg = slice(rowptr[m], rowptr[m + 1])
        cols_ref = np.nonzero(resid[i])[0]
        np.testing.assert_array_equal(csr_col[seg], cols_ref)
        np.testing.assert_array_equal(csr_val[seg], resid[i, cols_ref].astype(np.float32))
    # ---- sampled columns of A: CSC entries -----------------------------------------------------
    csc_row, csc_val = sa.csc_row.cpu().numpy(), sa.csc_val.cpu().numpy()
    cols_a = np.unique(np.concatenate([rng.choice(K, 12, replace=False), hot_cols, [0, K - 1]]))
    a_cols = O.bf16_bits_to_f64(a_bits[:, cols_a])
    ac_cols, resid_cols = O.occ_split(a_cols, lo, hi)
    for j, k in enumerate(cols_a):
        seg = slice(colptr[k], colptr[k + 1])
        rows_ref = np.nonzero(resid_cols[:, j])[0]
        np.testing.assert_array_equal(csc_row[seg], rows_ref)
        np.testing.assert_array_equal(csc_val[seg], resid_cols[rows_ref, j].astype(np.float32))

    # ---- sampled columns of W: codes (both layouts) -------------------------------------------
    cols_w = np.unique(np.concatenate([rng.choice(N, 28, replace=False), [0, N - 1, 239, 240]]))
    qw = O.absmax_quantize(O.bf16_bits_to_f64(w_bits[:, cols_w]), 1)
    np.testing.assert_array_equal(sw.codes_t[torch.as_tensor(cols_w, device="cuda")].cpu().numpy(), qw.packed_t())
    # the row-major layout of W holds the same codes: rows of W are pairs of nibbles along n
    w_codes_rows = O.unpack_nibbles(sw.codes[:, torch.as_tensor(cols_w // 2, device="cuda")].cpu().numpy())
    pick = np.arange(len(cols_w)) * 2 + (cols_w % 2)
    np.testing.assert_array_equal(w_codes_rows[:, pick], qw.codes)

    # ---- forward: Y on rows x cols_w -------------------------------------------------------------
    w_cols = O.bf16_bits_to_f64(w_bits[:, cols_w])
    y_fp4 = (O.gemm_codes(qa.codes, qw.codes.T) * d_a[rows].astype(np.float64)[:, None]) \
        * d_w[cols_w].astype(np.float64)[None, :]
    y_comp = resid @ w_cols
    got = y32[torch.as_tensor(rows, device="cuda")][:, torch.as_tensor(cols_w, device="cuda")].cpu().numpy()
    # heavy residuals send their hot columns through the GEMM's dense tail: accumulation floor of
    # the tensor cores as in test_gpu_linear.py (4e-6 of the summed magnitudes of the residual's products)
    floor = 4e-6 * (np.abs(resid) @ np.abs(w_cols)) if alpha <= 0.995 else 0.0
    _close(got, y_fp4 + y_comp, np.abs(y_fp4) + np.abs(y_comp), "Y", floor)
    _bf16(y16, rows, cols_w, y_fp4 + y_comp, np.abs(y_fp4) + np.abs(y_comp), "Y (BF16)", floor)

    # ---- dgrad: dA on rows x cols_a ----------------------------------------------------------------
    qg1 = O.absmax_quantize(O.bf16_bits_to_f64(dy_bits[rows]), 0, prescale=d_w)
    # codes of W rows cols_a (all N): scaled by the per-column gamma of the full tensor
    gamma_w, _ = O.absmax_scales(amax_w)
    w_sel = O.bf16_bits_to_f64(w_bits[cols_a])                       # [len(cols_a), N]
    w_sel_codes = O.lut_quantize((w_sel * gamma_w.astype(np.float64)[None, :]).astype(np.float32))
    da_ref = O.gemm_codes(qg1.codes, w_sel_codes) * qg1.descale.astype(np.float64)[:, None]
    got = da32[torch.as_tensor(rows, device="cuda")][:, torch.as_tensor(cols_a, device="cuda")].cpu().numpy()
    _close(got, da_ref, np.abs(da_ref), "dA")
    _bf16(da16, rows, cols_a, da_ref, np.abs(da_ref), "dA (BF16)")

    # ---- wgrad: dW on cols_a x cols_w ----------------------------------------------------------------
    gamma_a, _ = O.absmax_scales(amax_a)
    a_sel_codes = O.lut_quantize((ac_cols * gamma_a.astype(np.float64)[:, None]).astype(np.float32))   # [M, len(cols_a)]
    qg2 = O.absmax_quantize(O.bf16_bits_to_f64(dy_bits[:, cols_w]), 1, prescale=d_a)
    s_fp4 = O.gemm_codes(a_sel_codes.T, qg2.codes.T) * qg2.descale.astype(np.float64)[None, :]
    s_comp = resid_cols.T @ O.bf16_bits_to_f64(dy_bits[:, cols_w])
    w_scaled = (O.bf16_bits_to_f64(w_bits[np.ix_(cols_a, cols_w)]) * gamma_w[cols_w].astype(np.float64)[None, :]).astype(np.float32)
    factor = O.dge_fprime(w_scaled.astype(np.float64))
    got = dw32[torch.as_tensor(cols_a, device="cuda")][:, torch.as_tensor(cols_w, device="cuda")].cpu().numpy()
    # dense residual columns are summed on the tensor cores in chunks of 128 tokens: the same
    # accumulation floor as the forward tail, against the summed magnitudes of the column's products
    floor_w = 4e-6 * (np.abs(resid_cols).T @ np.abs(O.bf16_bits_to_f64(dy_bits[:, cols_w]))) * factor
    _close(got, (s_fp4 + s_comp) * factor, (np.abs(s_fp4) + np.abs(s_comp)) * factor, "dW", floor_w)
    _bf16(dw16, cols_a, cols_w, (s_fp4 + s_comp) * factor, (np.abs(s_fp4) + np.abs(s_comp)) * factor, "dW (BF16)",
          floor_w)
    ctx.close()
