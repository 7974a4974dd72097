"""Kernel microbenchmarks of the library at sizes of the caller's choosing (CUDA-event timing).

    python -m paper_2501_17116_b200.microbench gemm 8192x8192x8192 [--kind 0|1] [--f32] [--reps 20]
    python -m paper_2501_17116_b200.microbench quantize 16384 5120 [--alpha 0.99] [--reps 5]

`gemm` times fp4_gemm alone on random codes (several shapes may be given, comma-separated) and
prints TFLOP/s.  `quantize` times the clamping token-wise quantiser (histogram / select, encoder,
sparse extraction) and the plain channel-wise quantiser (absmax, encoder) on a synthetic activation
of the given shape, per kernel class, and prints GB/s of the 2 bytes per element each class reads.
The numbers quoted for large tensors in the repository's notes come from these two commands.
"""
import argparse

import numpy as np
import torch

from . import binding as fp4
from . import workloads as WL


def bench_gemm(shapes, kind: int, out_f32: bool, reps: int):
    ctx = fp4.Context(0, 1 << 20)
    for (I, J, C) in shapes:
        a = torch.randint(0, 255, (I, C // 2), dtype=torch.uint8, device="cuda")
        b = torch.randint(0, 255, (J, C // 2), dtype=torch.uint8, device="cuda")
        ra, ca = torch.rand(I, device="cuda"), torch.rand(J, device="cuda")
        out = torch.empty((I, J), dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
        for _ in range(3):
            fp4.fp4_gemm(ctx, a, b, ra, ca, out_f32=out_f32, gemm_kind=kind, out=out)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fp4.fp4_gemm(ctx, a, b, ra, ca, out_f32=out_f32, gemm_kind=kind, out=out)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        print(f"gemm kind={'f8f6f4' if kind else 'mxf4'} {I}x{J}x{C} out={'f32' if out_f32 else 'bf16'}: "
              f"{us:.1f} us  {2.0 * I * J * C / us / 1e6:.0f} TFLOP/s  status={ctx.read_status()}", flush=True)
    ctx.close()


def bench_quantize(M: int, K: int, alpha: float, reps: int):
    cfg = WL.CONFIGS[4] if alpha < 0.995 else WL.CONFIGS[1]      # heavy or light outlier recipe
    x = torch.from_numpy(WL.activations(cfg, K, M=M).view(np.int16)).cuda().view(torch.bfloat16)
    ctx = fp4.Context(0, int(fp4.load_library().fp4_workspace_bytes(M, K, 128)))
    q = fp4.QTensor(M, K, 0, x.device, fp4.tail_capacity(M, K, alpha))
    qw = fp4.QTensor(M, K, 1, x.device)
    for _ in range(2):
        fp4.fp4_quantize(ctx, x, 0, alpha=alpha, out=q)
        fp4.fp4_quantize(ctx, x, 1, out=qw)
    torch.cuda.synchronize()
    ctx.set_overlap(False)                 # one kernel at a time: class times are not inflated by sharing
    ctx.profile_reset()
    ctx.profile_enable(True)
    for _ in range(reps):
        fp4.fp4_quantize(ctx, x, 0, alpha=alpha, out=q)
        fp4.fp4_quantize(ctx, x, 1, out=qw)
    torch.cuda.synchronize()
    print(f"quantize {M}x{K} alpha={alpha}: token-wise with clamping + channel-wise without, per kernel class")
    for k, (ms, n) in ctx.profile_read().items():
        if n:
            print(f"  {k:10s} {1e3 * ms / reps:9.1f} us per pair of calls ({n // reps} kernels) -> "
                  f"{M * K * 2 / (ms / reps * 1e-3) / 1e9:7.0f} GB/s of one read of the tensor")
    print(f"  residual entries {int(q.nnz.item())}, status {ctx.read_status()}")
    ctx.close()


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="what", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("shapes", help="IxJxC[,IxJxC...] (multiples of 128)")
    g.add_argument("--kind", type=int, default=0, help="0 mxf4, 1 f8f6f4")
    g.add_argument("--f32", action="store_true", help="fp32 output instead of BF16")
    g.add_argument("--reps", type=int, default=20)
    q = sub.add_parser("quantize")
    q.add_argument("rows", type=int)
    q.add_argument("cols", type=int)
    q.add_argument("--alpha", type=float, default=0.99)
    q.add_argument("--reps", type=int, default=5)
    args = ap.parse_args()
    if args.what == "gemm":
        bench_gemm([tuple(int(v) for v in s.split("x")) for s in args.shapes.split(",")], args.kind, args.f32, args.reps)
    else:
        bench_quantize(args.rows, args.cols, args.alpha, args.reps)


if __name__ == "__main__":
    main()
