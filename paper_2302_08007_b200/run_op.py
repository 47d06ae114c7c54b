"""Run one operation of the library a few times on a seeded synthetic tensor (for profilers and
quick timing):  python -m paper_2302_08007_b200.run_op --op pack --fmt MX6 --axis 1 --dtype bf16"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as bdr
from . import synth

FORMATS = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}


def _timed(fn, reps):
    fn()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev[0].record()
    for _ in range(reps):
        fn()
    ev[1].record()
    torch.cuda.synchronize()
    return ev[0].elapsed_time(ev[1]) / reps


def run_gemm(a, cfg):
    """C[rows, rows] = A[rows, cols] * B[rows, cols]^T with both operands packed in --fmt along K = cols."""
    M = N = a.rows
    K = a.cols
    A = torch.from_numpy(synth.normal_matrix(M, K, seed=0, stream=10)).cuda()
    B = torch.from_numpy(synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)).cuda()
    pa, pb = bdr.alloc_planes(cfg, M, K), bdr.alloc_planes(cfg, N, K)
    bdr.bdr_pack(cfg, A, pa)
    bdr.bdr_pack(cfg, B, pb)
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    if a.f8:
        ws = torch.empty(bdr.mx_gemm_f8_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
        ms = _timed(lambda: bdr.mx_gemm_f8(cfg, pa, cfg, pb, M, N, K, c, ws), a.reps)
    elif a.ws:
        ws = torch.empty(bdr.mx_gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
        ms = _timed(lambda: bdr.mx_gemm_ws(cfg, pa, cfg, pb, M, N, K, c, ws), a.reps)
    else:
        ms = _timed(lambda: bdr.mx_gemm(cfg, pa, cfg, pb, M, N, K, c), a.reps)
    print("%s %s %dx%dx%d: %.4f ms per launch, %.1f TFLOP/s, status %d" % (
        "mx_gemm_f8" if a.f8 else "mx_gemm_ws" if a.ws else "mx_gemm", a.fmt, M, N, K, ms, 2.0 * M * N * K / ms / 1e9, bdr.mx_gemm_status()))


def run_sweep(a):
    """The 457-configuration QSNR sweep over rows*cols fp32 values ~ N(0,1) (one row)."""
    from . import sweep
    cfgs = [c for _, c in sweep.sweep_configs()]
    x = torch.from_numpy(synth.normal(a.rows * a.cols, seed=0)).cuda().reshape(1, -1)
    out = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
    ms = _timed(lambda: bdr.bdr_qsnr(cfgs, x, out, ws), a.reps)
    print("bdr_qsnr %d configs x %d values: %.4f ms per call, %.0f configs/s" % (len(cfgs), x.numel(), ms, len(cfgs) / ms * 1e3))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="pack", choices=["quant_dequant", "pack", "unpack", "gemm", "sweep"])
    ap.add_argument("--fmt", default="MX6", choices=list(FORMATS))
    ap.add_argument("--axis", type=int, default=1)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--cols", type=int, default=8192)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--no-sums", action="store_true")
    ap.add_argument("--ws", action="store_true", help="gemm: the two-phase entry point (mx_gemm_ws)")
    ap.add_argument("--f8", action="store_true", help="gemm: the block-scaled 8-bit entry point (mx_gemm_f8; MX4 / MX6)")
    ap.add_argument("--no-y", action="store_true", help="quant_dequant: only the QSNR sums")
    a = ap.parse_args()
    cfg = FORMATS[a.fmt]
    if a.op == "gemm":
        return run_gemm(a, cfg)
    if a.op == "sweep":
        return run_sweep(a)
    x = torch.from_numpy(synth.outlier_channel_matrix(a.rows, a.cols, seed=0, stream=3)).cuda()
    if a.dtype == "bf16":
        x = x.to(torch.bfloat16)
    y = torch.empty_like(x)
    planes = bdr.alloc_planes(cfg, a.rows, a.cols, a.axis)
    sums = None if a.no_sums else torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_pack(cfg, x, planes, axis=a.axis)

    def once():
        if a.op == "quant_dequant":
            bdr.bdr_quant_dequant(cfg, x, None if a.no_y else y, axis=a.axis, qsnr_sums=sums)
        elif a.op == "pack":
            bdr.bdr_pack(cfg, x, planes, axis=a.axis, qsnr_sums=sums)
        else:
            bdr.bdr_unpack(cfg, planes, y, axis=a.axis)

    once()  # first call of this kernel variant: attribute set-up
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev[0].record()
    for _ in range(a.reps):
        once()
    ev[1].record()
    torch.cuda.synchronize()
    print("%s %s axis=%d %s %dx%d: %.4f ms per launch" % (a.op, a.fmt, a.axis, a.dtype, a.rows, a.cols,
                                                          ev[0].elapsed_time(ev[1]) / a.reps))


if __name__ == "__main__":
    main()
