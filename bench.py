#!/usr/bin/env python
"""Benchmark of the FP4 linear layer, forward + backward, on synthetic LLaMA-shaped layers.

One step = one pass of the whole hot path (quantile select, clamp, quantise, FP4 GEMM,
compensation; dY quantisation, dgrad, wgrad, compensation, DGE) over every linear of the
workload.  The default workload is the largest single-GPU configuration: the seven linears of a
LLaMA-13B-shaped decoder layer at 16384 tokens, alpha = 0.99, DGE on (the last entry of the
configuration list); `--config I` selects another.  Inputs are seeded and synthetic.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

Prints ONE JSON line.  `value` = sum over linears of 6 M K N flop / device time of the step,
inputs resident in HBM.  `e2e` = the same through fp4_linear_step_host with pinned host buffers,
host<->device copies inside the timed region.  `roofline` describes the kernel class that takes
the largest share of the step, timed live with CUDA events on the launching stream; `kernels`
lists every class; `kernels_isolated` times single kernels alone (the GEMM at 8192^3 and at the
workload's largest GEMM, the quantiser kernels on the workload's largest tensor), each with its
own clock samples.  With `--impl reference` the CPU oracle is timed on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fp4_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"
# fallback peaks (an earlier measurement on this machine), used only if MEASURED_PEAKS.json is absent
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0
FP4_OVER_BF16 = 4.0                 # nominal dense ratio 9 : 2.25 PFLOP/s
SM_COUNT, FMA_LANES = 148, 128      # plain fp32 pipe: 148 SMs x 128 FMA lanes x 2 flop
BURST_SECONDS = 1.0                 # a class timed inside a region shorter than this is held to the burst peak

# DRAM bytes (read + write) per launch of a kernel class, from the ncu captures summarised under
# profiles/, keyed by workload; a class without a capture on that workload reports null.
NCU_TRAFFIC_PER_LAUNCH = {
    "llama-1.3b-layer": {
        "gemm": 17.4e6,        # profiles/gemm_fp4_llama1p3b.md: forward 6.4 MB, backward (two GEMMs per launch) 28.3 MB
        "encode": 14.0e6,      # profiles/quantizer_encode_llama1p3b.md (writes still in L2 at kernel end)
        "select": 16.9e6,      # profiles/quantizer_select_absmax_llama1p3b.md
        "absmax": 12.6e6,
        "comp_fwd": 36.1e6,    # profiles/compensation_llama1p3b.md
        "comp_wgrad_dge": 6.5e6,
    },
    # profiles/compensation_gather_llama7b_mlp.md: captured on the 7B MLP block (same kernels, same
    # residual density; the 13B layer is too large for a multi-pass capture) and scaled to the mean
    # launch of this workload by the units processed: comp_fwd_kept moves 6.85 B per output element
    # (fp32 FP4-branch read, BF16 store, the weight once), comp_wgrad_short reads dY once plus the
    # entries (1.14 x 2 B per element of dY) and writes its fp32 rows (0.87 x 4 B per weight element).
    "llama-13b-layer": {
        "comp_fwd": 6.85 * 124.6e6,
        "comp_wgrad_dge": 1.14 * 2 * 124.6e6 + 0.87 * 4 * 45.3e6,
    },
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p["bf16_tflops_sustained"]),
                    sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_burst=FALLBACK_BF16_TFLOPS,
                bf16_sustained=FALLBACK_BF16_TFLOPS_SUSTAINED, sm_max_mhz=1965.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def layer_inputs(cfg, WL, seed=0):
    """Per linear: (name, K, N, A bits, W bits, dY bits).  q/k/v and gate/up read the same activation."""
    groups = {"q": 0, "k": 0, "v": 0, "o": 1, "gate": 2, "up": 2, "down": 3, "fc": 0}
    acts = {}
    out = []
    for li, lin in enumerate(cfg.linears):
        g = (groups[lin.name], lin.K)
        if g not in acts:
            acts[g] = WL.activations(cfg, lin.K, seed, layer=groups[lin.name])
        out.append((lin.name, lin.K, lin.N, acts[g], WL.weights(cfg, lin.K, lin.N, seed, layer=li),
                    WL.output_grads(cfg, lin.N, seed, layer=li)))
    return out


def fuse_shared(layers_in):
    """q|k|v and gate|up as one linear each: the group's weights (and output gradients) side by side."""
    groups = (("q", "k", "v"), ("gate", "up"))
    by_name = {t[0]: t for t in layers_in}
    out, done = [], set()
    for t in layers_in:
        name = t[0]
        if name in done:
            continue
        grp = next((g for g in groups if name in g and all(n in by_name for n in g)), None)
        if grp is None:
            out.append(t)
            continue
        members = [by_name[n] for n in grp]
        done.update(grp)
        out.append(("|".join(grp), members[0][1], sum(m[2] for m in members), members[0][3],
                    np.ascontiguousarray(np.concatenate([m[4] for m in members], axis=1)),
                    np.ascontiguousarray(np.concatenate([m[5] for m in members], axis=1))))
    return out


ORACLE_SAMPLE_TOKENS = 1024         # tokens of the first linear the oracle is timed on (a bounded sample)


def oracle_sample_tflops(cfg, WL, reps: int, m_rows: int):
    """The oracle as it stands on the first linear of the workload, `m_rows` tokens; TFLOP/s."""
    from oracle import fp4_oracle as O
    lin = cfg.linears[0]
    a = WL.activations(cfg, lin.K, M=m_rows)
    w = WL.weights(cfg, lin.K, lin.N)
    dy = WL.output_grads(cfg, lin.N, M=m_rows)
    alpha = cfg.alphas[0]
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        f = O.linear_fwd(a, w, alpha)
        O.linear_bwd(dy, w, f)
        times.append(time.perf_counter() - t0)
    flop = 6.0 * m_rows * lin.K * lin.N
    return flop / 1e12, times


def oracle_sample_text(cfg, m_rows: int) -> str:
    lin = cfg.linears[0]
    return (f"oracle fwd+bwd (select, clamp, quantise, GEMMs, compensation, DGE) of linear '{lin.name}' "
            f"({lin.K}x{lin.N}) on the first {m_rows} of {cfg.M} tokens")


def run_reference(args):
    """CPU oracle on the host cores; rank 0 alone works and prints."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2501_17116_b200 import workloads as WL
    cfg = WL.CONFIGS[args.config]
    m_rows = min(ORACLE_SAMPLE_TOKENS, cfg.M)
    tf, times = oracle_sample_tflops(cfg, WL, args.warmup + args.steps, m_rows)
    timed = times[args.warmup:]
    sec = float(np.sum(timed))
    value = tf * len(timed) / sec
    cores = os.cpu_count()
    sample = oracle_sample_text(cfg, m_rows) + " per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec / len(timed),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "tokens": cfg.M, "alpha": cfg.alphas[0], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def timed_with_clocks(gpu_index: int, fn, min_seconds: float = 0.4):
    """Runs fn() repeatedly for at least `min_seconds` of device time with the clocks sampled
    beside it; returns (reps, elapsed ms by CUDA events on the current stream, clock record)."""
    import torch
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fn()
    e1.record()
    torch.cuda.synchronize()
    reps = max(5, int(min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.12)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    return reps, ms, sampler.stop()


def isolated_kernels(fp4, WL, cfg, dev, gpu_index: int, kind: int, peaks) -> dict:
    """Single kernels timed alone, each with its own clock samples: the GEMM at 8192^3 and at the
    workload's largest GEMM, the quantiser kernels on the workload's largest activation-sized
    tensor (larger than L2, so every repetition reads it from HBM)."""
    import torch
    out = {}
    burst = (FP4_OVER_BF16 if kind == 0 else FP4_OVER_BF16 / 2) * peaks["bf16_burst"]
    ctx = fp4.Context(gpu_index, 1 << 20)
    big = max(cfg.linears, key=lambda l: l.K * l.N)
    for label, (I, J, Cc) in (("gemm_8192x8192x8192", (8192, 8192, 8192)),
                              (f"gemm_fwd_{big.name}_{cfg.M}x{big.N}x{big.K}", (cfg.M, big.N, big.K))):
        a = torch.randint(0, 255, (I, Cc // 2), dtype=torch.uint8, device=dev)
        b = torch.randint(0, 255, (J, Cc // 2), dtype=torch.uint8, device=dev)
        ra, ca = torch.rand(I, device=dev), torch.rand(J, device=dev)
        o = torch.empty((I, J), dtype=torch.bfloat16, device=dev)
        reps, ms, clk = timed_with_clocks(
            gpu_index, lambda: fp4.fp4_gemm(ctx, a, b, ra, ca, out_f32=False, gemm_kind=kind, out=o))
        tf = 2.0 * I * J * Cc * reps / (ms / 1e3) / 1e12
        out[label] = {"bound": "tensor", "us": round(1e3 * ms / reps, 2), "achieved": round(tf, 1), "unit": "TFLOP/s",
                      "peak": round(burst, 1), "frac": round(tf / burst, 4),
                      "peak_source": "4 x burst bf16 cuBLAS (kernel timed alone)", "reps": reps, "clocks": clk}
        del a, b, o
    assert ctx.read_status() == 0
    ctx.close()

    # quantiser kernels on the largest activation-sized tensor of the workload
    M = cfg.M
    Kq = max(max(l.K for l in cfg.linears), max(l.N for l in cfg.linears))
    alpha = cfg.alphas[0]
    x = torch.from_numpy(WL.activations(cfg, Kq, M=M).view(np.int16)).to(dev).view(torch.bfloat16)
    ctx = fp4.Context(gpu_index, int(fp4.load_library().fp4_workspace_bytes(M, Kq, 128)))
    q = fp4.QTensor(M, Kq, 0, dev, fp4.tail_capacity(M, Kq, alpha))
    qw = fp4.QTensor(M, Kq, 1, dev)
    ctx.set_overlap(False)
    elems = float(M) * Kq

    def both():
        fp4.fp4_quantize(ctx, x, 0, alpha=alpha, out=q)      # token-wise with clamping: select, encode, sparse
        fp4.fp4_quantize(ctx, x, 1, out=qw)                  # channel-wise, no clamp: absmax, encode

    for _ in range(2):
        both()
    torch.cuda.synchronize()
    ctx.profile_reset()
    ctx.profile_enable(True)
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.12)
    reps = 0
    t0 = time.perf_counter()
    while reps < 5 or time.perf_counter() - t0 < 0.4:
        fp4.fp4_quantize(ctx, x, 0, alpha=alpha, out=q)
        reps += 1
        torch.cuda.synchronize()
    occ = ctx.profile_read()
    ctx.profile_reset()
    reps_w = 0
    t0 = time.perf_counter()
    while reps_w < 5 or time.perf_counter() - t0 < 0.4:
        fp4.fp4_quantize(ctx, x, 1, out=qw)
        reps_w += 1
        torch.cuda.synchronize()
    plain = ctx.profile_read()
    clk = sampler.stop()
    ctx.profile_enable(False)
    shape = f"{M}x{Kq}"
    for label, rec, n, bytes_per_elem in (
            (f"select_{shape}", occ["select"], reps, 2.0),
            (f"encode_clamped_{shape}", occ["encode"], reps, 3.125),
            (f"absmax_{shape}", plain["absmax"], reps_w, 2.0),
            (f"encode_{shape}", plain["encode"], reps_w, 3.0)):
        ms = rec[0] / n
        gbs = bytes_per_elem * elems / (ms / 1e3) / 1e9 if ms > 0 else 0.0
        out[label] = {"bound": "hbm", "us": round(1e3 * ms, 2), "achieved": round(gbs, 1), "unit": "GB/s",
                      "peak": peaks["hbm_gbs"], "frac": round(gbs / peaks["hbm_gbs"], 4),
                      "bytes_per_element": bytes_per_elem, "reps": n, "clocks": clk}
    assert ctx.read_status() == 0
    ctx.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--gemm-kind", type=int, default=0, help="0 mxf4 (K=64), 1 f8f6f4 (K=32)")
    ap.add_argument("--precision", default="w4a4", choices=["w4a4", "w4a8", "w8a4", "w4a4-dy8", "w4a4-dy8e5m2"],
                    help="operand formats: w4a4 (the method, default); w4a8 / w8a4: E4M3 activations / weights "
                         "(the ablation settings); w4a4-dy8 / w4a4-dy8e5m2: dY quantised to E4M3 / E5M2.  All but w4a4 need --gemm-kind 1")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fuse-shared", action="store_true",
                    help="q|k|v and gate|up as one linear each (weights stored side by side): Y and dW are those of the "
                         "separate linears, dA is the gradient with respect to the shared input")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer measurement (profiling runs)")
    ap.add_argument("--no-isolated", action="store_true", help="skip the single-kernel measurements")
    ap.add_argument("--no-share-activations", action="store_true",
                    help="quantise the activation of every linear, also where q/k/v or gate/up read the same tensor")
    ap.add_argument("--cache-weights", action="store_true",
                    help="micro-batch steps of gradient accumulation: the weights' codes are those of the step's "
                         "first micro-batch (quantised before the timed region), re-used by every timed step")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import paper_2501_17116_b200 as fp4
    from paper_2501_17116_b200 import harness, workloads as WL

    rank, local_rank, world = harness.rank_info()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    harness.init_process_group("nccl")
    peaks = load_peaks()
    cfg = WL.CONFIGS[args.config]
    alpha = cfg.alphas[0]
    M = cfg.M
    kind = args.gemm_kind
    fmt_a = fp4.FP4_FORMAT_E4M3 if args.precision == "w4a8" else fp4.FP4_FORMAT_E2M1
    fmt_w = fp4.FP4_FORMAT_E4M3 if args.precision == "w8a4" else fp4.FP4_FORMAT_E2M1
    dy8 = {"w4a4-dy8": fp4.FP4_FORMAT_E4M3, "w4a4-dy8e5m2": fp4.FP4_FORMAT_E5M2}.get(args.precision, fp4.FP4_FORMAT_E2M1)
    if args.precision != "w4a4":
        assert kind == 1, "E4M3 operands need the byte-container GEMM: pass --gemm-kind 1"
    if fmt_a == fp4.FP4_FORMAT_E4M3:
        alpha = 1.0                              # outlier clamping belongs to 4-bit activations

    # ------------------------------------------------------------------ inputs ------------
    def pinned(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()

    layers = []
    ws_bytes = 0
    lib = fp4.load_library()
    share = not args.no_share_activations
    owner = {}                                   # id of the host activation array -> first layer that reads it
    inputs = layer_inputs(cfg, WL, seed=rank)
    if args.fuse_shared:
        inputs = fuse_shared(inputs)
    pinned_a = {}                                # one pinned copy of an activation that several linears read
    while inputs:
        name, K, N, a_bits, w_bits, dy_bits = inputs.pop(0)      # the unpinned copies are dropped as we go
        if id(a_bits) not in pinned_a:
            pinned_a[id(a_bits)] = pinned(a_bits)
        hA, hW, hG = pinned_a[id(a_bits)], pinned(w_bits), pinned(dy_bits)
        first = owner.setdefault(id(a_bits), len(layers)) if share else len(layers)
        shared = first != len(layers)
        L = dict(name=name, K=K, N=N, hA=hA, hW=hW, hG=hG, W=hW.to(dev), G=hG.to(dev),
                 A=layers[first]["A"] if shared else hA.to(dev), reuse_a=shared, keep=a_bits,
                 Y=torch.empty((M, N), dtype=torch.bfloat16, device=dev),
                 dA=torch.empty((M, K), dtype=torch.bfloat16, device=dev),
                 dW=torch.empty((K, N), dtype=torch.bfloat16, device=dev),
                 sa=layers[first]["sa"] if shared else fp4.QTensor(M, K, 0, dev, fp4.tail_capacity(M, K, alpha), fmt=fmt_a),
                 sw=fp4.QTensor(K, N, 1, dev, fmt=fmt_w))
        del w_bits, dy_bits
        layers.append(L)
        ws_bytes = max(ws_bytes, int(lib.fp4_step_host_workspace_bytes(M, K, N, alpha)))
    for L in layers:
        L.pop("keep")                            # (held only so that ids of activation arrays stayed unique)
    # pinned host outputs of the end-to-end measurement: one set, as large as the largest linear
    # needs, written by every linear in turn (the copies back are ordered on one stream)
    def host_out(n_elems):
        return torch.empty(n_elems, dtype=torch.bfloat16).pin_memory()
    hY_all = host_out(max(M * L["N"] for L in layers))
    hdA_all = host_out(max(M * L["K"] for L in layers))
    hdW_all = host_out(max(L["K"] * L["N"] for L in layers))
    for L in layers:
        L["hY"] = hY_all[:M * L["N"]].view(M, L["N"])
        L["hdA"] = hdA_all[:M * L["K"]].view(M, L["K"])
        L["hdW"] = hdW_all[:L["K"] * L["N"]].view(L["K"], L["N"])
    ctx = fp4.Context(local_rank, ws_bytes)
    flop_step = sum(6.0 * M * L["K"] * L["N"] for L in layers)
    resident_bytes = sum(2 * (M * L["K"] + L["K"] * L["N"] + M * L["N"]) * 2 for L in layers)

    def step():
        for L in layers:
            fp4.fp4_linear_fwd(ctx, L["A"], L["W"], alpha, L["sa"], L["sw"], gemm_kind=kind, out=L["Y"],
                               reuse_a=L["reuse_a"], reuse_w=cached_w[0])
            fp4.fp4_linear_bwd(ctx, L["G"], L["W"], L["sa"], L["sw"], gemm_kind=kind, dA=L["dA"], dW=L["dW"],
                               dy_fmt=dy8)

    cached_w = [False]                           # --cache-weights: set after the first (untimed) step

    def step_host():
        for L in layers:
            fp4.fp4_linear_step_host(ctx, L["hA"], L["hW"], L["hG"], alpha, L["hY"], L["hdA"], L["hdW"],
                                     gemm_kind=kind, read_status=False)

    # ------------------------------------------------------------------ device-resident ---
    # The step is captured once into a CUDA graph (the library's side streams fork from and
    # rejoin the capturing stream) and replayed: the timed region is K replays back to back.
    for _ in range(args.warmup):
        step()
        cached_w[0] = args.cache_weights
    torch.cuda.synchronize()
    assert ctx.read_status() == 0, "device status word is set"
    ctx.profile_reset()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    launches_per_step = ctx.launch_count()
    for _ in range(args.warmup):
        graph.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    harness.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    harness.barrier()
    ms = e0.elapsed_time(e1)
    launches = launches_per_step * args.steps
    assert ctx.read_status() == 0, "device status word is set"

    # Per-kernel-class device times: the same K steps again, launched plainly with a CUDA event
    # pair around every kernel class on its launching stream (events cannot sit inside a graph).
    ctx.profile_reset()
    ctx.profile_enable(True)
    ctx.set_overlap(False)              # one kernel at a time: durations are not inflated by SM sharing
    torch.cuda.synchronize()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for _ in range(args.steps):
        step()
    p1.record()
    torch.cuda.synchronize()
    ms_profiled = p0.elapsed_time(p1)
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    ctx.set_overlap(True)
    ctx.profile_reset()
    nnz = [int(L["sa"].nnz.item()) if L["sa"].nnz is not None else 0 for L in layers]

    # Residual entries that are gathered per entry (one row of the dense matrix each): all but those
    # of the dense columns (at least max(M / 4, 512) entries, the first 128 of them), which go through
    # the tensor cores -- in the weight gradient always, in the forward with a heavy residual.
    def scattered_entries(L, forward):
        sa = L["sa"]
        if sa.nnz is None:
            return 0
        total = int(sa.nnz.item())
        if forward and not (sa.sparse_cap * 100 >= M * L["K"]):
            return total
        counts = (sa.csc_colptr[1:] - sa.csc_colptr[:-1]).cpu().numpy()
        dense = np.nonzero(counts >= max(M // 4, 512))[0][:128]
        return total - int(counts[dense].sum())

    gathered_fwd = sum(scattered_entries(L, True) * L["N"] * 2.0 for L in layers)
    gathered_bwd = sum(scattered_entries(L, False) * L["N"] * 2.0 for L in layers)

    # L2 read bandwidth, measured here: the bound of those gathers
    l2_gbs = None
    if alpha < 1.0:
        probe = torch.empty(32 << 20, dtype=torch.uint8, device=dev)
        sink = torch.zeros(1, dtype=torch.int32, device=dev)
        blocks, reps = 16 * SM_COUNT, 1             # enough blocks that launch ramp and tail do not show
        best = None
        for _ in range(4):
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record()
            fp4.fp4_l2_read_probe(probe, reps, blocks, sink)
            q1.record()
            torch.cuda.synchronize()
            t = q0.elapsed_time(q1)
            best = t if best is None else min(best, t)
        l2_gbs = blocks * reps * probe.numel() / (best / 1e3) / 1e9
        del probe

    # ------------------------------------------------------------------ end to end ---------
    # (the host-buffer entry point takes the method's own formats only)
    ms_e2e = None
    if args.precision == "w4a4" and not args.no_e2e:
        for _ in range(3):
            step_host()
        torch.cuda.synchronize()
        harness.barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(args.steps):
            step_host()
        t1.record()
        torch.cuda.synchronize()
        harness.barrier()
        ms_e2e = t0.elapsed_time(t1)
    clocks = sampler.stop()

    sec = harness.max_over_ranks(ms / 1e3, dev)
    sec_e2e = harness.max_over_ranks(ms_e2e / 1e3, dev) if ms_e2e is not None else None
    total_flop = harness.sum_over_ranks(flop_step * args.steps, dev)
    value = total_flop / sec / 1e12
    value_e2e = total_flop / sec_e2e / 1e12 if sec_e2e else None
    h2d = sum((M * L["K"] + L["K"] * L["N"] + M * L["N"]) * 2 for L in layers)
    d2h = h2d

    # ------------------------------------------------------------------ rooflines ----------
    # Tensor peak: 4 x the measured BF16 cuBLAS rate (nominal dense FP4 : BF16 = 9 : 2.25); the
    # byte-container kind runs at the FP8 rate (K = 32 per instruction), half of that.  The burst
    # figure applies to a class whose timed region is short, the sustained one to a seconds-long one.
    ratio = FP4_OVER_BF16 if kind == 0 else FP4_OVER_BF16 / 2
    region_seconds = ms_profiled / 1e3
    use_burst = region_seconds < BURST_SECONDS
    fp4_peak = ratio * (peaks["bf16_burst"] if use_burst else peaks["bf16_sustained"])
    alu_peak = SM_COUNT * FMA_LANES * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    steps = args.steps
    elems_a = sum(M * L["K"] for L in layers if not L["reuse_a"])      # activations actually quantised
    elems_w = sum(L["K"] * L["N"] for L in layers)
    elems_g = sum(M * L["N"] for L in layers)
    nnz_total = sum(nnz)
    nnz_quantised = sum(z for z, L in zip(nnz, layers) if not L["reuse_a"])
    work = {
        # class: (bound, algorithmic work per step, unit of the rate).  Bytes are what the method
        # itself has to move: every tensor read once per kernel class that needs it, codes written
        # once per layout (A: 2 + 0.5 + 0.5 + 1/8 mask; W: 2 + 1; dY: 2 + 0.5 + 0.5, both backward
        # copies from one read).
        "gemm": ("tensor", flop_step, "TFLOP/s"),
        "select": ("hbm", 2.0 * elems_a, "GB/s"),
        "encode": ("hbm", 3.125 * elems_a + 3.0 * elems_w + 3.0 * elems_g, "GB/s"),
        "absmax": ("hbm", 2.0 * elems_w + 2.0 * elems_g, "GB/s"),
        "sparse": ("hbm", 2 * 8.0 * nnz_quantised + 3 * elems_a / 8.0, "GB/s"),       # entries + 3 mask sweeps
        # compensation: 2 nnz N flop on the plain ALUs by the method's own count; what bounds the
        # kernels is the L2 traffic of the per-entry gathers (one BF16 row of the dense matrix per
        # scattered entry), reported against the L2 read bandwidth measured above
        "comp_fwd": ("l2", gathered_fwd, "GB/s"),
        "comp_wgrad_dge": ("l2", gathered_bwd, "GB/s"),
    }
    alu_flop = {"comp_fwd": sum(2.0 * z * L["N"] for z, L in zip(nnz, layers)),
                "comp_wgrad_dge": sum(2.0 * z * L["N"] + 8.0 * L["K"] * L["N"] for z, L in zip(nnz, layers))}
    src = "of measured" if peaks["source"] == "measured" else "of fallback"
    peak_text = {
        "tensor": f"{src}: {ratio:g} x {'burst' if use_burst else 'sustained'} bf16 cuBLAS "
                  f"(classes timed inside a {region_seconds:.2f} s region)",
        "hbm": f"{src}: copy bandwidth",
        "l2": "of measured: L2 read bandwidth by fp4_l2_read_probe in this run (32 MB buffer, 16-byte loads)",
    }
    kernels = {}
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    for name, (t_ms, n) in prof.items():
        bound, w_step, unit = work[name]
        peak = {"tensor": fp4_peak, "hbm": peaks["hbm_gbs"], "l2": l2_gbs or 1.0}[bound]
        scale = 1e12 if unit == "TFLOP/s" else 1e9
        achieved = (w_step * steps / (t_ms / 1e3) / scale) if t_ms > 0 else 0.0
        kernels[name] = {"bound": bound, "achieved": round(achieved, 2), "peak": round(peak, 1), "unit": unit,
                         "frac": round(achieved / peak, 4), "ms_per_step": round(t_ms / steps, 4),
                         "share": round(t_ms / total_ms, 4), "launches_per_step": n // steps}
        if bound == "l2":
            # the method's own flop count against the plain fp32 pipe (148 SMs x 128 FMA x 2 x max clock)
            tf = alu_flop[name] * steps / (t_ms / 1e3) / 1e12 if t_ms > 0 else 0.0
            kernels[name]["alu_tflops"] = round(tf, 2)
            kernels[name]["alu_frac"] = round(tf / alu_peak, 4)
        if bound == "tensor":
            kernels[name]["frac_of_burst"] = round(achieved / (ratio * peaks["bf16_burst"]), 4)
            kernels[name]["frac_of_sustained"] = round(achieved / (ratio * peaks["bf16_sustained"]), 4)
    dominant = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    dk = kernels[dominant]
    traffic = NCU_TRAFFIC_PER_LAUNCH.get(cfg.name, {}).get(dominant) if args.precision == "w4a4" and kind == 0 else None
    roofline = {"kernel": dominant, "bound": dk["bound"], "achieved": dk["achieved"], "peak": dk["peak"],
                "unit": dk["unit"], "frac": dk["frac"], "traffic": traffic, "peak_source": peak_text[dk["bound"]]}

    # ------------------------------------------------------------------ single kernels -----
    kernels_isolated = None
    if not args.no_isolated and args.precision == "w4a4":
        kernels_isolated = isolated_kernels(fp4, WL, cfg, dev, local_rank, kind, peaks)

    # ------------------------------------------------------------------ CPU baseline -------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        m_rows = min(ORACLE_SAMPLE_TOKENS, M)
        tf, times = oracle_sample_tflops(cfg, WL, 3, m_rows)
        cpu_baseline = {"value": tf / min(times), "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                        "sample": oracle_sample_text(cfg, m_rows) + ", best of 3",
                        "seconds": round(min(times), 3)}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "fp4_e2m1" if args.precision == "w4a4" else ("fp4_e2m1+fp8_e5m2" if args.precision.endswith("e5m2") else "fp4_e2m1+fp8_e4m3"), "data": "synthetic",
            "config": {"workload": cfg.name, "tokens": M, "linears": [f"{L['name']}:{L['K']}x{L['N']}" for L in layers],
                       "alpha": alpha, "dge": True, "gemm_kind": "mxf4" if kind == 0 else "f8f6f4",
                       "precision": args.precision,
                       "l2": f"inputs exceed L2: {resident_bytes / 1e6:.0f} MB touched per step",
                       "launch": "one CUDA graph per step, replayed",
                       "shared_activations": ("q|k|v and gate|up run as one linear each (weights side by side)"
                                              if args.fuse_shared else
                                              "q/k/v and gate/up read one activation tensor: quantised once, re-used"
                                              if share else "every linear quantises its activation"),
                       "weights": ("codes of the weights cached across the timed steps (micro-batches of one "
                                   "optimizer step)" if args.cache_weights else "quantised in every step"),
                       "kernel_timing": f"CUDA events per kernel class over {args.steps} plainly launched steps, side "
                                        f"streams off ({ms_profiled / args.steps:.3f} ms/step that way)",
                       "replicas": world},
            "e2e": ({"value": value_e2e, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                     "ms_per_step": 1e3 * sec_e2e / args.steps} if sec_e2e else None),
            "gpu_launches": launches,
            "roofline": roofline, "kernels": kernels, "kernels_isolated": kernels_isolated,
            "cpu_baseline": cpu_baseline, "clocks": clocks,
            "residual_nnz": nnz_total,
        }))
    ctx.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
