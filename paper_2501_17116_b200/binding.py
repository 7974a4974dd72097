"""Thin ctypes binding of libfp4linear.so: argument marshalling only.

Function names and argument order follow include/fp4_linear.h.  PyTorch is used for device
memory and the current stream; every step of the path runs inside the library's kernels.
There is no CPU fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from .build import LIB_PATH

FP4_GEMM_MXF4 = 0
FP4_GEMM_F8F6F4 = 1
FP4_GEMM_F8F6F4_A8 = 2
FP4_GEMM_F8F6F4_B8 = 3
FP4_GEMM_F8F6F4_A8B8 = 4
FP4_GEMM_A_E5M2 = 0x10
FP4_GEMM_B_E5M2 = 0x20
FP4_BWD_DY_E4M3 = 0x100
FP4_BWD_DY_E5M2 = 0x200
FP4_FORMAT_E2M1 = 0
FP4_FORMAT_E4M3 = 1
FP4_FORMAT_E5M2 = 2
FP4_DEV_NONFINITE = 2
FP4_DEV_TIMEOUT = 4

EXPORTS = ("fp4_create", "fp4_destroy", "fp4_workspace_bytes", "fp4_status_string", "fp4_quantize",
           "fp4_gemm", "fp4_linear_fwd", "fp4_linear_bwd", "fp4_step_host_workspace_bytes",
           "fp4_linear_step_host", "fp4_profile_enable", "fp4_profile_reset", "fp4_profile_read",
           "fp4_launch_count", "fp4_quantile_thresholds_static", "fp4_set_overlap", "fp4_l2_read_probe", "fp4_debug_set", "fp4_sparse_capacity",
           "fp4_set_quantile_mode")
FP4_STATIC_MAX_ROWS = 65536
FP4_QUANTILE_SIGNED = 0
FP4_QUANTILE_ABS = 1
FP4_QUANTILE_TOKEN = 2
FP4_DEBUG_WAIT_LIMIT_US = 1
FP4_DEBUG_SKIP_FILL = 2
KERNEL_CLASSES = ("gemm", "select", "encode", "absmax", "sparse", "comp_fwd", "comp_wgrad_dge")


class fp4_qtensor(C.Structure):
    _fields_ = [
        ("rows", C.c_int64), ("cols", C.c_int64),
        ("codes", C.c_void_p), ("codes_t", C.c_void_p), ("amax", C.c_void_p), ("thresholds", C.c_void_p),
        ("csr_rowptr", C.c_void_p), ("csr_col", C.c_void_p), ("csr_val", C.c_void_p),
        ("csc_colptr", C.c_void_p), ("csc_row", C.c_void_p), ("csc_val", C.c_void_p),
        ("sparse_cap", C.c_int64), ("nnz", C.c_void_p), ("format", C.c_int32), ("reserved", C.c_int32),
    ]


_lib = None


def load_library(path: str | None = None) -> C.CDLL:
    """dlopen the in-tree library and declare its prototypes.  Raises if it was not built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} is missing: build it with `python -m paper_2501_17116_b200.build` "
            "(there is no fallback path)")
    lib = C.CDLL(path)
    vp, i64, i32p = C.c_void_p, C.c_int64, C.c_void_p
    lib.fp4_create.argtypes = [C.POINTER(vp), C.c_int, C.c_size_t]
    lib.fp4_create.restype = C.c_int
    lib.fp4_destroy.argtypes = [vp]
    lib.fp4_destroy.restype = C.c_int
    lib.fp4_workspace_bytes.argtypes = [i64, i64, i64]
    lib.fp4_workspace_bytes.restype = C.c_size_t
    lib.fp4_status_string.argtypes = [C.c_int]
    lib.fp4_status_string.restype = C.c_char_p
    lib.fp4_quantize.argtypes = [vp, vp, vp, i64, i64, C.c_int, C.c_double, vp, C.POINTER(fp4_qtensor), i32p]
    lib.fp4_quantize.restype = C.c_int
    lib.fp4_gemm.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, vp, vp, C.c_int, C.c_int, i32p]
    lib.fp4_gemm.restype = C.c_int
    lib.fp4_linear_fwd.argtypes = [vp, vp, vp, vp, i64, i64, i64, C.c_double, C.c_int, C.c_int, vp, C.c_int,
                                   C.POINTER(fp4_qtensor), C.POINTER(fp4_qtensor), i32p]
    lib.fp4_linear_fwd.restype = C.c_int
    lib.fp4_linear_bwd.argtypes = [vp, vp, vp, vp, C.POINTER(fp4_qtensor), C.POINTER(fp4_qtensor), i64, i64, i64,
                                   C.c_int, C.c_float, C.c_float, C.c_int, vp, vp, C.c_int, i32p]
    lib.fp4_linear_bwd.restype = C.c_int
    lib.fp4_step_host_workspace_bytes.argtypes = [i64, i64, i64, C.c_double]
    lib.fp4_step_host_workspace_bytes.restype = C.c_size_t
    lib.fp4_linear_step_host.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, C.c_double, C.c_int, C.c_float,
                                         C.c_float, C.c_int, vp, vp, vp, C.POINTER(C.c_int32)]
    lib.fp4_linear_step_host.restype = C.c_int
    lib.fp4_profile_enable.argtypes = [vp, C.c_int]
    lib.fp4_profile_enable.restype = C.c_int
    lib.fp4_profile_reset.argtypes = [vp]
    lib.fp4_profile_reset.restype = C.c_int
    lib.fp4_profile_read.argtypes = [vp, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.fp4_profile_read.restype = C.c_int
    lib.fp4_l2_read_probe.argtypes = [vp, vp, C.c_size_t, C.c_int, C.c_int, vp]
    lib.fp4_l2_read_probe.restype = C.c_int
    lib.fp4_debug_set.argtypes = [vp, C.c_int, i64]
    lib.fp4_debug_set.restype = C.c_int
    lib.fp4_sparse_capacity.argtypes = [i64, i64, C.c_double, C.c_int]
    lib.fp4_sparse_capacity.restype = C.c_int64
    lib.fp4_set_overlap.argtypes = [vp, C.c_int]
    lib.fp4_set_quantile_mode.argtypes = [vp, C.c_int]
    lib.fp4_set_quantile_mode.restype = C.c_int
    lib.fp4_set_overlap.restype = C.c_int
    lib.fp4_launch_count.argtypes = [vp]
    lib.fp4_launch_count.restype = C.c_int64
    lib.fp4_quantile_thresholds_static.argtypes = [vp, vp, i64, i64, C.c_double, vp]
    lib.fp4_quantile_thresholds_static.restype = C.c_int
    if path == LIB_PATH:
        _lib = lib
    return lib


class Fp4Error(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"fp4 error {code}: {load_library().fp4_status_string(code).decode()}")


def _check(rc: int):
    if rc != 0:
        raise Fp4Error(rc)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Context:
    """fp4_create / fp4_destroy.  Owns the workspace and a device status word."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self.lib = load_library()
        self.device = device
        self.handle = C.c_void_p()
        torch.cuda.set_device(device)
        _check(self.lib.fp4_create(C.byref(self.handle), device, workspace_bytes))
        self.workspace_bytes = workspace_bytes
        self.status = torch.zeros(1, dtype=torch.int32, device=f"cuda:{device}")

    @classmethod
    def for_shape(cls, M: int, K: int, N: int, device: int = 0):
        return cls(device, int(load_library().fp4_workspace_bytes(M, K, N)))

    def close(self):
        if self.handle:
            self.lib.fp4_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def read_status(self) -> int:
        """Device status word (synchronises)."""
        return int(self.status.item())

    # measurement support -------------------------------------------------------------------
    def profile_enable(self, on: bool = True):
        _check(self.lib.fp4_profile_enable(self.handle, int(on)))

    def profile_reset(self):
        _check(self.lib.fp4_profile_reset(self.handle))

    def profile_read(self) -> dict:
        """{kernel class: (total device ms, kernels)} since the last reset (waits for the events)."""
        out = {}
        for kc, name in enumerate(KERNEL_CLASSES):
            ms, n = C.c_double(), C.c_int64()
            _check(self.lib.fp4_profile_read(self.handle, kc, C.byref(ms), C.byref(n)))
            out[name] = (ms.value, n.value)
        return out

    def set_overlap(self, on: bool = True):
        _check(self.lib.fp4_set_overlap(self.handle, int(on)))

    def set_quantile_mode(self, mode: int):
        """FP4_QUANTILE_SIGNED (the paper's clamp, default), FP4_QUANTILE_ABS (one threshold on |x|) or
        FP4_QUANTILE_TOKEN (signed thresholds per token)."""
        _check(self.lib.fp4_set_quantile_mode(self.handle, int(mode)))

    def debug_set(self, key: int, value: int):
        """Failure-path testing: FP4_DEBUG_WAIT_LIMIT_US / FP4_DEBUG_SKIP_FILL (fp4_debug_set)."""
        _check(self.lib.fp4_debug_set(self.handle, int(key), int(value)))

    def launch_count(self) -> int:
        return int(self.lib.fp4_launch_count(self.handle))


class QTensor:
    """Caller-owned buffers of one quantised operand (struct fp4_qtensor)."""

    def __init__(self, rows: int, cols: int, scale_axis: int, device, sparse_cap: int = 0,
                 codes: bool = True, codes_t: bool = True, fmt: int = FP4_FORMAT_E2M1):
        dev = device
        self.rows, self.cols, self.scale_axis, self.fmt = rows, cols, scale_axis, fmt
        per_byte = 2 if fmt == FP4_FORMAT_E2M1 else 1          # E2M1 nibbles or FP8 bytes
        self.codes = torch.empty((rows, cols // per_byte), dtype=torch.uint8, device=dev) if codes else None
        self.codes_t = torch.empty((cols, rows // per_byte), dtype=torch.uint8, device=dev) if codes_t else None
        self.amax = torch.empty(rows if scale_axis == 0 else cols, dtype=torch.float32, device=dev)
        self.sparse_cap = int(sparse_cap)
        if sparse_cap > 0:
            cap = max(int(sparse_cap), 1)
            # lo, hi of the tensor; with thresholds per token the library fills all 2 * rows (lo, hi of every row)
            self.thresholds_rows = torch.zeros(2 * rows, dtype=torch.float32, device=dev)
            self.thresholds = self.thresholds_rows[:2]
            self.csr_rowptr = torch.zeros(rows + 1, dtype=torch.int32, device=dev)
            self.csr_col = torch.zeros(cap, dtype=torch.int32, device=dev)
            self.csr_val = torch.zeros(cap, dtype=torch.float32, device=dev)
            self.csc_colptr = torch.zeros(cols + 1, dtype=torch.int32, device=dev)
            self.csc_row = torch.zeros(cap, dtype=torch.int32, device=dev)
            self.csc_val = torch.zeros(cap, dtype=torch.float32, device=dev)
            self.nnz = torch.zeros(1, dtype=torch.int32, device=dev)
        else:
            self.thresholds = self.thresholds_rows = self.csr_rowptr = self.csr_col = self.csr_val = None
            self.csc_colptr = self.csc_row = self.csc_val = self.nnz = None
        self.struct = fp4_qtensor(
            rows, cols, _ptr(self.codes), _ptr(self.codes_t), _ptr(self.amax), _ptr(self.thresholds),
            _ptr(self.csr_rowptr), _ptr(self.csr_col), _ptr(self.csr_val),
            _ptr(self.csc_colptr), _ptr(self.csc_row), _ptr(self.csc_val), self.sparse_cap, _ptr(self.nnz), fmt, 0)


def tail_capacity(rows: int, cols: int, alpha: float) -> int:
    """A `sparse_cap` that suffices whichever form of the clamp is set on the context: the larger of
    fp4_sparse_capacity for the tensor-wide clamp and for thresholds per token."""
    lib = load_library()
    caps = [int(lib.fp4_sparse_capacity(rows, cols, float(alpha), m)) for m in (FP4_QUANTILE_SIGNED, FP4_QUANTILE_TOKEN)]
    assert min(caps) >= 0, "rows, cols or alpha outside their range"
    return max(caps)


def fp4_quantize(ctx: Context, x: torch.Tensor, scale_axis: int, alpha: float = 1.0, prescale=None,
                 codes: bool = True, codes_t: bool = True, out: QTensor | None = None,
                 fmt: int = FP4_FORMAT_E2M1) -> QTensor:
    assert x.dtype == torch.bfloat16 and x.is_cuda and x.is_contiguous() and x.dim() == 2
    rows, cols = x.shape
    if out is None:
        out = QTensor(rows, cols, scale_axis, x.device, tail_capacity(rows, cols, alpha), codes, codes_t, fmt)
    _check(ctx.lib.fp4_quantize(ctx.handle, _stream(), _ptr(x), rows, cols, scale_axis, float(alpha),
                                _ptr(prescale), C.byref(out.struct), _ptr(ctx.status)))
    return out


def fp4_gemm(ctx: Context, a_codes: torch.Tensor, b_codes: torch.Tensor, row_amax=None, col_amax=None,
             out_f32: bool = True, gemm_kind: int = FP4_GEMM_MXF4, out: torch.Tensor | None = None):
    """out = (a b^T) with the two de-scales; E2M1 operands are packed two per byte, FP8 operands
    (FP4_GEMM_F8F6F4_A8 / _B8 / _A8B8: E4M3, or E5M2 with FP4_GEMM_A_E5M2 / _B_E5M2 OR-ed in) one per byte."""
    base_kind = gemm_kind & ~(FP4_GEMM_A_E5M2 | FP4_GEMM_B_E5M2)
    a8 = base_kind in (FP4_GEMM_F8F6F4_A8, FP4_GEMM_F8F6F4_A8B8)
    b8 = base_kind in (FP4_GEMM_F8F6F4_B8, FP4_GEMM_F8F6F4_A8B8)
    I, J = a_codes.shape[0], b_codes.shape[0]
    Cc = a_codes.shape[1] * (1 if a8 else 2)
    assert b_codes.shape[1] * (1 if b8 else 2) == Cc
    if out is None:
        out = torch.empty((I, J), dtype=torch.float32 if out_f32 else torch.bfloat16, device=a_codes.device)
    _check(ctx.lib.fp4_gemm(ctx.handle, _stream(), _ptr(a_codes), _ptr(b_codes), I, J, Cc, _ptr(row_amax),
                            _ptr(col_amax), _ptr(out), int(out_f32), gemm_kind, _ptr(ctx.status)))
    return out


def fp4_linear_fwd(ctx: Context, A: torch.Tensor, W: torch.Tensor, alpha: float, saved_a: QTensor | None = None,
                   saved_w: QTensor | None = None, reuse_w: bool = False, gemm_kind: int = FP4_GEMM_MXF4,
                   reuse_a: bool = False,
                   out_f32: bool = False, out: torch.Tensor | None = None,
                   fmt_a: int = FP4_FORMAT_E2M1, fmt_w: int = FP4_FORMAT_E2M1):
    """Forward of the layer.  `fmt_a` / `fmt_w` = FP4_FORMAT_E4M3 give the W4A8 / W8A4 settings (the
    formats are those of the saved operands; they need gemm_kind = FP4_GEMM_F8F6F4)."""
    M, K = A.shape
    K2, N = W.shape
    assert K == K2 and A.dtype == torch.bfloat16 and W.dtype == torch.bfloat16
    if saved_a is None:
        saved_a = QTensor(M, K, 0, A.device, tail_capacity(M, K, alpha), fmt=fmt_a)
    if saved_w is None:
        saved_w = QTensor(K, N, 1, A.device, fmt=fmt_w)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32 if out_f32 else torch.bfloat16, device=A.device)
    _check(ctx.lib.fp4_linear_fwd(ctx.handle, _stream(), _ptr(A), _ptr(W), M, K, N, float(alpha), int(reuse_w) | (2 if reuse_a else 0),
                                  gemm_kind, _ptr(out), int(out_f32), C.byref(saved_a.struct),
                                  C.byref(saved_w.struct), _ptr(ctx.status)))
    return out, saved_a, saved_w


def fp4_linear_bwd(ctx: Context, dY: torch.Tensor, W: torch.Tensor, saved_a: QTensor, saved_w: QTensor,
                   dge_on: bool = True, dge_k: float = 5.0, dge_clip: float = 3.0,
                   gemm_kind: int = FP4_GEMM_MXF4, out_f32: bool = False, dA=None, dW=None,
                   want_da: bool = True, want_dw: bool = True, dy_e4m3: bool = False,
                   dy_fmt: int = FP4_FORMAT_E2M1):
    """Backward of the layer.  `dy_fmt` = FP4_FORMAT_E4M3 / FP4_FORMAT_E5M2 (or `dy_e4m3`) quantises dY
    to FP8 bytes instead of E2M1 nibbles."""
    if dy_e4m3 or dy_fmt == FP4_FORMAT_E4M3:
        gemm_kind |= FP4_BWD_DY_E4M3
    elif dy_fmt == FP4_FORMAT_E5M2:
        gemm_kind |= FP4_BWD_DY_E5M2
    M, N = dY.shape
    K = W.shape[0]
    dt = torch.float32 if out_f32 else torch.bfloat16
    if dA is None and want_da:
        dA = torch.empty((M, K), dtype=dt, device=dY.device)
    if dW is None and want_dw:
        dW = torch.empty((K, N), dtype=dt, device=dY.device)
    _check(ctx.lib.fp4_linear_bwd(ctx.handle, _stream(), _ptr(dY), _ptr(W), C.byref(saved_a.struct),
                                  C.byref(saved_w.struct), M, K, N, int(dge_on), float(dge_k), float(dge_clip),
                                  gemm_kind, _ptr(dA), _ptr(dW), int(out_f32), _ptr(ctx.status)))
    return dA, dW


def fp4_linear_step_host(ctx: Context, A_host: torch.Tensor, W_host: torch.Tensor, dY_host: torch.Tensor,
                         alpha: float, Y_host: torch.Tensor, dA_host: torch.Tensor, dW_host: torch.Tensor,
                         dge_on: bool = True, dge_k: float = 5.0, dge_clip: float = 3.0,
                         gemm_kind: int = FP4_GEMM_MXF4, read_status: bool = True) -> int:
    """Forward + backward with host (pinned) BF16 tensors; returns the device status word."""
    M, K = A_host.shape
    N = W_host.shape[1]
    for t in (A_host, W_host, dY_host, Y_host, dA_host, dW_host):
        assert not t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    st = C.c_int32(0)
    _check(ctx.lib.fp4_linear_step_host(ctx.handle, _stream(), _ptr(A_host), _ptr(W_host), _ptr(dY_host), M, K, N,
                                        float(alpha), int(dge_on), float(dge_k), float(dge_clip), gemm_kind,
                                        _ptr(Y_host), _ptr(dA_host), _ptr(dW_host),
                                        C.byref(st) if read_status else None))
    return st.value


def fp4_quantile_thresholds_static(x: torch.Tensor, alpha: float, out: torch.Tensor | None = None) -> torch.Tensor:
    """{lo, hi} of `x` through the entry point that allocates nothing on the device.

    For callers that may not call cudaMalloc (and so cannot own a Context): the scratch is a
    fixed array inside the library.  `out` (float32[2] on the device) may be passed so that this
    wrapper does not allocate either.  Calls on one device must not overlap on the GPU.
    """
    assert x.dtype == torch.bfloat16 and x.is_cuda and x.is_contiguous() and x.dim() == 2
    if out is None:
        out = torch.empty(2, dtype=torch.float32, device=x.device)
    _check(load_library().fp4_quantile_thresholds_static(_stream(), _ptr(x), x.shape[0], x.shape[1], float(alpha),
                                                         _ptr(out)))
    return out


def fp4_l2_read_probe(buf: torch.Tensor, repeats: int, blocks: int, sink: torch.Tensor):
    """Measurement support: `blocks` blocks read all of `buf` `repeats` times through L2 (the caller times it)."""
    _check(load_library().fp4_l2_read_probe(_stream(), _ptr(buf), buf.numel() * buf.element_size(), int(repeats),
                                            int(blocks), _ptr(sink)))
