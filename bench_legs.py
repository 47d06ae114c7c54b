"""Secondary benchmark legs (argument marshalling + CUDA-event timing only): the design-space sweep
(configs/s), the MX GEMM (TFLOP/s), the linear-layer step, the small-vector latency case, and the single-operation
runner behind `bench.py --only` (one operation a few times on a seeded tensor, for profilers and quick timing).
bench.py calls these after its timed steps."""
from __future__ import annotations

import os
import time

import numpy as np
import torch

from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import linear, sweep, synth

SWEEP_N = 1 << 24


def _time(fn, reps: int, warmup: int = 1) -> float:
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def sweep_leg(args) -> dict:
    """QSNR of 2^24 fp32 values per distribution under the 457-configuration sweep."""
    named = sweep.sweep_configs()
    cfgs = [c for _, c in named]
    names = [n for n, _ in named]
    out = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
    per_dist = {}
    total_ms = 0.0
    show = {"MX9": "bdr_k1=16_k2=2_d2=1_m=7", "MX6": "bdr_k1=16_k2=2_d2=1_m=4", "MX4": "bdr_k1=16_k2=2_d2=1_m=2",
            "MSFP16": "bdr_k1=16_k2=1_d2=0_m=7", "INT8": "int8", "INT4": "int4", "FP8_E4M3": "fp8_e4m3",
            "FP8_E5M2": "fp8_e5m2", "VSQ_INT4_d2=6": "vsq_int4_d2=6"}
    for dist in synth.SWEEP_DISTRIBUTIONS:
        x = torch.from_numpy(synth.sweep_distribution(dist, SWEEP_N, seed=0)).cuda().reshape(1, -1)
        ms = _time(lambda: bdr.bdr_qsnr(cfgs, x, out, ws), reps=3)
        q = out.cpu().numpy()
        per_dist[dist] = {"ms": ms, "qsnr_db": {k: float(q[names.index(v)]) for k, v in show.items()}}
        total_ms += ms
        del x
    n_eval = len(cfgs) * len(synth.SWEEP_DISTRIBUTIONS)
    value = n_eval / (total_ms * 1e-3)
    elem_cfg = n_eval * SWEEP_N / (total_ms * 1e-3)
    peaks = getattr(args, "peaks", {})
    hbm = float(peaks.get("hbm_gbs", 6650.0))
    # Two bounds.  (1) Issue: 148 SMs x 4 schedulers x 32 lanes x 1.965 GHz = 37.2 T lane-instructions/s; the kernel
    # executes kSweepInstr lane-instructions per element-configuration (ncu smsp__inst_executed on the 457-configuration
    # sweep), so `frac` is an issue-slot utilisation of THIS kernel's instruction stream, not a statement about the
    # fewest instructions the method needs.  (2) What a one-configuration-per-pass implementation could reach at the
    # HBM roofline: peak / (4 bytes x 2^24 values) configs/s; the fused kernel reads the tensor once per 16 families.
    issue_peak = 148 * 4 * 32 * 1.965e9
    single_pass = hbm * 1e9 / (4.0 * SWEEP_N)
    roofline = {"bound": "alu", "achieved": elem_cfg * kSweepInstr / 1e12, "peak": issue_peak / 1e12,
                "unit": "T lane-instr/s", "frac": elem_cfg * kSweepInstr / issue_peak,
                "kind": "issue-slot utilisation with the kernel's own %.1f instructions per element-configuration (ncu)" % kSweepInstr,
                "peak_source": "148 SMs x 4 schedulers x 32 lanes x 1.965 GHz", "traffic": None,
                "single_pass_hbm_bound_configs_per_s": single_pass, "vs_single_pass_hbm_bound": value / single_pass}
    out_leg = {"metric": "BDR-sweep configs/s", "value": value, "unit": "configs/s",
               "configs": len(cfgs), "distributions": list(synth.SWEEP_DISTRIBUTIONS),
               "elements_per_distribution": SWEEP_N, "ms_total": total_ms,
               "element_configs_per_s": elem_cfg, "bound": "alu", "roofline": roofline,
               "per_distribution": per_dist}
    if getattr(args, "cpu_legs", False):
        out_leg["cpu_baseline"] = sweep_oracle_sample()
    return {"sweep": out_leg}


kSweepInstr = 7.8  # lane-instructions per element-configuration of sweep_kernel (ncu, profiles/sweep_457cfg_4m.md)


def sweep_oracle_sample() -> dict:
    """The oracle on a stated subset of the sweep: 16 configurations (every 32nd grid point + INT8, FP8 E4M3, VSQ) over
    the 2^24 values of the N(0,1) distribution, all host cores."""
    from oracle import oracle as orc
    cores = len(os.sched_getaffinity(0))
    named = sweep.sweep_configs()
    pick = list(range(0, 441, 32))[:13] + [442, 443, 446]
    x = synth.sweep_distribution("normal", SWEEP_N, seed=0).reshape(1024, -1)   # rows are lines: threads split rows
    t0 = time.perf_counter()
    for i in pick:
        c = named[i][1]
        orc.qsnr(orc.Config(c.k1, c.d1, c.k2, c.d2, c.m, c.scale_kind, c.rounding), x, nthreads=cores)
    sec = time.perf_counter() - t0
    return {"value": len(pick) / (sec * (SWEEP_N / x.size)), "unit": "configs/s", "cores": cores, "kind": "oracle",
            "sample": "%d of 457 configurations on the 2^24 N(0,1) values as 1024 rows (%.1f s)" % (len(pick), sec)}


def gemm_leg(args) -> dict:
    """C[4096,4096] = A * B^T with MX6 operands packed along K (fp32 accumulate and output)."""
    M = N = K = 4096
    a = torch.from_numpy(synth.normal_matrix(M, K, seed=0, stream=10)).cuda()
    b = torch.from_numpy(synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)).cuda()
    pa, pb = bdr.alloc_planes(bdr.MX6, M, K), bdr.alloc_planes(bdr.MX6, N, K)
    bdr.bdr_pack(bdr.MX6, a, pa)
    bdr.bdr_pack(bdr.MX6, b, pb)
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    ws = torch.empty(bdr.mx_gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    ms = _time(lambda: bdr.mx_gemm_ws(bdr.MX6, pa, bdr.MX6, pb, M, N, K, c, ws), reps=20, warmup=3)
    ms_fused = _time(lambda: bdr.mx_gemm(bdr.MX6, pa, bdr.MX6, pb, M, N, K, c), reps=20, warmup=3)
    ws8 = torch.empty(bdr.mx_gemm_f8_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    ms_f8 = _time(lambda: bdr.mx_gemm_f8(bdr.MX6, pa, bdr.MX6, pb, M, N, K, c, ws8), reps=20, warmup=3)
    f8_exact = int(ws8[-256:-252].view(torch.int32).item()) == 0
    # the same product from operands re-encoded ahead of time (what a caller with static weights would do)
    enc = []
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    for planes, rows in ((pa, M), (pb, N)):
        e8 = torch.empty((rows, K), dtype=torch.uint8, device="cuda")
        sf = torch.empty(rows * K // 32, dtype=torch.uint8, device="cuda")
        bdr.bdr_reencode_e4m3(bdr.MX6, planes, rows, K, e8, sf, flag)
        enc += [e8, sf]
    ms_pre = _time(lambda: bdr.mx_gemm_e4m3(enc[0], enc[1], enc[2], enc[3], M, N, K, c), reps=20, warmup=3)
    # the plain mx_gemm call while scratch memory is lent to the library (it then takes the 8-bit path itself)
    bdr.bdr_set_workspace(ws8)
    try:
        ms_lent = _time(lambda: bdr.mx_gemm(bdr.MX6, pa, bdr.MX6, pb, M, N, K, c), reps=20, warmup=3)
    finally:
        bdr.bdr_set_workspace(None)
    ms_hw = _time(lambda: bdr.mx_gemm_hw(bdr.MX6, pa, bdr.MX6, pb, M, N, K, c, r=64, f=25), reps=2, warmup=1)
    cpu = gemm_oracle_sample(M, N, K) if getattr(args, "cpu_legs", False) else None
    tf = lambda t: 2.0 * M * N * K / (t * 1e-3) / 1e12
    ws_name = ("mx_gemm_ws (both operands decoded once to a bf16 workspace, then a TMA-fed tcgen05 GEMM; the time "
               "covers both phases)")
    f8_name = ("mx_gemm_f8 (both operands re-encoded exactly to E4M3 with one E8M0 scale per 32 elements, then a "
               "block-scaled tcgen05 GEMM; the time covers both phases and the gated fall-back launch)")
    best_f8 = f8_exact and ms_f8 < ms
    return {"mx_gemm": {"metric": "MX-GEMM TFLOP/s", "value": tf(ms_f8 if best_f8 else ms), "unit": "TFLOP/s",
                        "ms": ms_f8 if best_f8 else ms, "shape": [M, N, K], "format": "MX6 x MX6", "bound": "tensor",
                        "entry_point": f8_name if best_f8 else ws_name,
                        "mx_gemm_ws": {"value": tf(ms), "unit": "TFLOP/s", "ms": ms},
                        "mx_gemm_f8": {"value": tf(ms_f8), "unit": "TFLOP/s", "ms": ms_f8, "ran_on_8bit_path": f8_exact},
                        "fused_mx_gemm": {"value": tf(ms_fused), "unit": "TFLOP/s", "ms": ms_fused,
                                          "note": "mx_gemm without scratch memory (decode inside the GEMM)"},
                        "mx_gemm_with_lent_workspace": {"value": tf(ms_lent), "unit": "TFLOP/s", "ms": ms_lent},
                        "mx_gemm_e4m3": {"value": tf(ms_pre), "unit": "TFLOP/s", "ms": ms_pre,
                                         "note": "operands re-encoded ahead of time (not the headline: the re-encoding is not timed)",
                                         "exact": int(flag.item()) == 0},
                        "mx_gemm_hw": {"value": tf(ms_hw), "unit": "TFLOP/s", "ms": ms_hw, "bound": "alu",
                                       "note": "the product as the dot-product pipeline of Section IV-B computes it (r = 64, f = 25): integer "
                                               "block sums, truncating alignment per block and output; ordinary arithmetic units, bit-exact "
                                               "with the oracle"},
                        "cpu_baseline": cpu, "status": bdr.mx_gemm_status()}}


def gemm_oracle_sample(M: int, N: int, K: int) -> dict:
    """The fp64 oracle product on sampled outputs of the C4 problem (operands quantized by the oracle first)."""
    from oracle import oracle as orc
    cores = len(os.sched_getaffinity(0))
    rows = 1024
    a = synth.normal_matrix(M, K, seed=0, stream=10)[:rows]
    b = synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)[:rows]
    t0 = time.perf_counter()
    qa, _ = orc.quant_dequant(orc.MX6, a, nthreads=cores)
    qb, _ = orc.quant_dequant(orc.MX6, b, nthreads=cores)
    orc.gemm_nt_f64(qa, qb, nthreads=cores)
    sec = time.perf_counter() - t0
    return {"value": 2.0 * rows * rows * K / sec / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
            "sample": "the %d x %d corner of C (first %d rows of A and of B, K = %d), quantization included (%.2f s)" % (rows, rows, rows, K, sec)}


def linear_leg(args) -> dict:
    """One transformer linear layer in MX9 training form: X[8192x4096], W[16384x4096], dY[8192x16384]
    (bf16); six quantizations with fused QSNR and three MX GEMMs (forward, dX, dW)."""
    tokens, d_in, d_out = 8192, 4096, 16384
    bf = lambda a: torch.from_numpy(synth.f32_to_bf16_bits(a).view(np.int16)).view(torch.bfloat16).cuda()
    x = bf(synth.outlier_channel_matrix(tokens, d_in, seed=0, stream=1, frac=0.01, gain=20.0))
    w = bf(synth.normal_matrix(d_out, d_in, seed=0, stream=2, sigma=0.02))
    dy = bf(synth.normal_matrix(tokens, d_out, seed=0, stream=3, sigma=1e-3))
    buf = linear.alloc(bdr.MX9, tokens, d_in, d_out)
    ms = _time(lambda: linear.step(bdr.MX9, x, w, dy, buf), reps=3)
    flops = 3 * 2.0 * tokens * d_in * d_out
    peaks = getattr(args, "peaks", {})
    hbm = float(peaks.get("hbm_gbs", 6650.0))
    tensor = float(peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops", 1590.0)))   # a kernel inside a long step

    def roofline(m_bits, t_ms, tensor_peak, what):
        # the step's floor: every operand read once and both its packed copies written (2 + 2 bits/8 bytes per element:
        # bdr_pack2) at the HBM peak, plus the three products at the tensor peak
        n_el = tokens * d_in + d_out * d_in + tokens * d_out
        qbytes = n_el * (2.0 + 2.0 * (m_bits + 2) / 8.0)
        floor_ms = qbytes / (hbm * 1e9) * 1e3 + flops / (tensor_peak * 1e12) * 1e3
        return {"bound": "tensor", "achieved": flops / (t_ms * 1e-3) / 1e12, "peak": tensor_peak, "unit": "TFLOP/s",
                "frac": floor_ms / t_ms, "floor_ms": floor_ms, "quantization_bytes": qbytes, "flops": flops,
                "kind": "floor = quantization bytes / HBM peak + 3 GEMMs / tensor peak; frac = floor / measured",
                "peak_source": what, "traffic": None}

    out = {"linear_layer": {"workload": "MX9 linear layer fwd+bwd: 6 quantize+pack (+QSNR), 3 mx_gemm", "ms": ms,
                            "gemm_tflops_incl_quantization": flops / (ms * 1e-3) / 1e12,
                            "roofline": roofline(7, ms, tensor, "measured sustained bf16 and HBM copy" if peaks else "fallback"),
                            "qsnr_db": linear.qsnr_db(buf), "mx_gemm_status": bdr.mx_gemm_status()}}
    del buf
    # the same step in MX6 (the paper's inference / fine-tuning format): the three products take the 8-bit path
    buf6 = linear.alloc(bdr.MX6, tokens, d_in, d_out)
    ms6 = _time(lambda: linear.step(bdr.MX6, x, w, dy, buf6), reps=3)
    nb = bdr.mx_gemm_f8_workspace_bytes(d_out, d_in, tokens)   # the flag word of the step's last product (dW)
    out["linear_layer"]["mx6"] = {"ms": ms6, "gemm_tflops_incl_quantization": flops / (ms6 * 1e-3) / 1e12,
                                  "roofline": roofline(4, ms6, 2.0 * tensor, "measured sustained bf16 x 2 (nominal 8-bit ratio) and HBM copy"),
                                  "ran_on_8bit_path": int(buf6.workspace[nb - 256:nb - 252].view(torch.int32).item()) == 0,
                                  "qsnr_db": linear.qsnr_db(buf6)}
    return out


def c1_leg(args) -> dict:
    """C1: MX6 of one fp32 vector of 65,536 values ~ N(0,1): dequantized tensor, packed planes and QSNR sums from one
    bdr_pack call.  0.57 MB that live in L2: the call is bound by launch latency, so it is reported in microseconds."""
    n = 65536
    xh = synth.normal(n, seed=0)
    x = torch.from_numpy(xh).cuda().reshape(1, n)
    y = torch.empty_like(x)
    planes = bdr.alloc_planes(bdr.MX6, 1, n, 1)
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    call = lambda: bdr.bdr_pack(bdr.MX6, x, planes, axis=1, y_dq=y, qsnr_sums=sums)
    call()
    torch.cuda.synchronize()
    us_stream = _time(call, reps=200, warmup=20) * 1e3          # back-to-back calls from Python
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call()
    us_graph = _time(g.replay, reps=200, warmup=20) * 1e3       # the launch alone, replayed
    lat = []
    for _ in range(50):                                         # one call, then wait for it: what a lone caller sees
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        call()
        torch.cuda.synchronize()
        lat.append((time.perf_counter() - t0) * 1e6)
    sums.zero_()
    call()
    db = bdr.bdr_qsnr_from_sums(sums, torch.empty(1, dtype=torch.float64, device="cuda")).item()
    out = {"workload": "C1: MX6 quantize + pack + dequantize + QSNR sums of 65,536 fp32 values ~ N(0,1), one bdr_pack call",
           "us_per_call_back_to_back": us_stream, "us_per_call_graph_replay": us_graph,
           "us_call_plus_sync_median": float(np.median(lat)), "bound": "launch latency (0.57 MB, served by L2)",
           "algorithmic_bytes": n * (4 + 4 + 0.75), "qsnr_db": db}
    if getattr(args, "cpu_legs", False):
        from oracle import oracle as orc
        t0 = time.perf_counter()
        for _ in range(20):
            orc.quant_dequant(orc.MX6, xh)
            orc.pack(orc.MX6, xh)
        out["cpu_baseline"] = {"value": (time.perf_counter() - t0) / 20 * 1e6, "unit": "us per call", "cores": 1, "kind": "oracle",
                               "sample": "the whole vector, quant-dequant + pack, 20 repetitions"}
    return {"c1_vector": out}


def embedding_leg(args) -> dict:
    """Lookups in an MX6-packed embedding table (Section V, inferencing): 2^20 rows of 128 elements, 2^20 random indices,
    bf16 output.  Algorithmic bytes per lookup: the row's packed bytes (128 x 6 / 8), the 8-byte index and the 256 output bytes."""
    n_rows, dim, n_idx = 1 << 20, 128, 1 << 20
    g = torch.Generator(device="cuda").manual_seed(0)
    table = (torch.randn((n_rows, dim), device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    planes = bdr.alloc_planes(bdr.MX6, n_rows, dim, 1)
    bdr.bdr_pack(bdr.MX6, table, planes, axis=1)
    idx = torch.randint(0, n_rows, (n_idx,), device="cuda", dtype=torch.int64, generator=g)
    out = torch.empty((n_idx, dim), dtype=torch.bfloat16, device="cuda")
    ms = _time(lambda: bdr.bdr_gather_rows(bdr.MX6, planes, n_rows, idx, out), reps=10, warmup=2)
    nbytes = n_idx * (dim * 6 / 8 + 8 + dim * 2)
    peaks = getattr(args, "peaks", {})
    hbm = float(peaks.get("hbm_gbs", 6650.0))
    res = {"workload": "2^20 random lookups in a 2^20 x 128 MX6-packed table, bf16 output", "ms": ms, "value": nbytes / (ms * 1e-3) / 1e9,
           "unit": "GB/s", "lookups_per_s": n_idx / (ms * 1e-3),
           "roofline": {"bound": "hbm", "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s", "frac": nbytes / (ms * 1e-3) / 1e9 / hbm,
                        "peak_source": "measured" if peaks else "fallback", "traffic": None,
                        "kind": "algorithmic bytes (packed row + index + output row) / CUDA-event time; random 96 + 8 + 8 byte reads"},
           "status": bdr.bdr_device_status()}
    if getattr(args, "cpu_legs", False):
        from oracle import oracle as orc
        sample = 4096
        host = tuple(t[:sample].cpu().numpy() for t in (planes.exps, planes.micro, planes.elems))
        t0 = time.perf_counter()
        orc.unpack(orc.MX6, host, sample, dim)
        sec = time.perf_counter() - t0
        res["cpu_baseline"] = {"value": sample / sec, "unit": "lookups/s", "cores": 1, "kind": "oracle",
                               "sample": "decoding %d rows of the table (%.3f s)" % (sample, sec)}
    return {"embedding_lookup": res}


# ---------------------------------------------------------------------------------------------------------------------
# bench.py --only <op>: one operation, a few launches, for profilers and quick timing
# ---------------------------------------------------------------------------------------------------------------------
FORMATS = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}


def run_only(a) -> None:
    cfg = FORMATS[a.fmt]
    reps = a.reps
    if a.only in ("gemm", "gemm_ws", "gemm_f8", "gemm_hw"):
        M = N = a.rows
        K = a.cols
        A = torch.from_numpy(synth.normal_matrix(M, K, seed=0, stream=10)).cuda()
        B = torch.from_numpy(synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)).cuda()
        pa, pb = bdr.alloc_planes(cfg, M, K), bdr.alloc_planes(cfg, N, K)
        bdr.bdr_pack(cfg, A, pa)
        bdr.bdr_pack(cfg, B, pb)
        c = torch.empty((M, N), dtype=torch.float32, device="cuda")
        if a.only == "gemm_f8":
            ws = torch.empty(bdr.mx_gemm_f8_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
            ms = _time(lambda: bdr.mx_gemm_f8(cfg, pa, cfg, pb, M, N, K, c, ws), reps)
        elif a.only == "gemm_ws":
            ws = torch.empty(bdr.mx_gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
            ms = _time(lambda: bdr.mx_gemm_ws(cfg, pa, cfg, pb, M, N, K, c, ws), reps)
        elif a.only == "gemm_hw":
            ms = _time(lambda: bdr.mx_gemm_hw(cfg, pa, cfg, pb, M, N, K, c, r=64, f=25), reps)
        else:
            ms = _time(lambda: bdr.mx_gemm(cfg, pa, cfg, pb, M, N, K, c), reps)
        print("%s %s %dx%dx%d: %.4f ms per call, %.1f TFLOP/s, status %d" % (a.only, a.fmt, M, N, K, ms, 2.0 * M * N * K / ms / 1e9,
                                                                          bdr.mx_gemm_status()))
        return
    if a.only == "sweep":
        cfgs = [c for _, c in sweep.sweep_configs()]
        x = torch.from_numpy(synth.normal(a.rows * a.cols, seed=0)).cuda().reshape(1, -1)
        out = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
        ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
        ms = _time(lambda: bdr.bdr_qsnr(cfgs, x, out, ws), reps)
        print("bdr_qsnr %d configs x %d values: %.4f ms per call, %.0f configs/s" % (len(cfgs), x.numel(), ms, len(cfgs) / ms * 1e3))
        return
    x = torch.from_numpy(synth.outlier_channel_matrix(a.rows, a.cols, seed=0, stream=3)).cuda()
    if a.dtype == "bf16":
        x = x.to(torch.bfloat16)
    y = torch.empty_like(x)
    planes = bdr.alloc_planes(cfg, a.rows, a.cols, a.axis)
    planes2 = bdr.alloc_planes(cfg, a.rows, a.cols, 1 - a.axis) if a.only == "pack2" else None
    sums = None if a.no_sums else torch.zeros(2, dtype=torch.float64, device="cuda")
    sums2 = None if a.no_sums else torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_pack(cfg, x, planes, axis=a.axis)

    def once():
        if a.only == "quant_dequant":
            bdr.bdr_quant_dequant(cfg, x, None if a.no_y else y, axis=a.axis, qsnr_sums=sums)
        elif a.only == "pack":
            bdr.bdr_pack(cfg, x, planes, axis=a.axis, qsnr_sums=sums)
        elif a.only == "pack2":
            bdr.bdr_pack2(cfg, x, planes if a.axis == 1 else planes2, planes2 if a.axis == 1 else planes, sums, sums2)
        else:
            bdr.bdr_unpack(cfg, planes, y, axis=a.axis)

    ms = _time(once, reps)
    print("%s %s axis=%d %s %dx%d: %.4f ms per launch, status %d" % (a.only, a.fmt, a.axis, a.dtype, a.rows, a.cols, ms,
                                                                   bdr.bdr_device_status()))


def paper_sweep_leg(args) -> dict:
    """Section IV-B/C as the paper sets it up: 16,384 vectors of 1,024 values ~ N(0, |N(0,1)|) (one variance per vector),
    the 457 configurations, the FP32 kinds scaled by the maximum over a window of past chunks (delayed scaling), and the
    QSNR-versus-cost frontier with cost = bits per element / packing efficiency of a 256-element tile in 64-byte lines."""
    n_vec, length, chunks, window = 16384, 1024, 8, 4
    named = sweep.sweep_configs()
    cfgs = [c for _, c in named]
    x = torch.from_numpy(synth.variable_variance_vectors(n_vec, length, seed=0)).cuda()
    out = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
    ms = _time(lambda: bdr.bdr_qsnr(cfgs, x, out, ws), reps=3)
    q_now = out.cpu().numpy().copy()
    # delayed scaling: chunk t is quantized with the largest maximum of chunks t - window .. t - 1
    per = n_vec // chunks
    hist = torch.zeros(chunks, dtype=torch.float32, device="cuda")
    for t in range(chunks):
        bdr.bdr_amax(x[t * per:(t + 1) * per], hist[t:t + 1])
    comp = [c for _, c in sweep.comparators()]
    outc = torch.empty(len(comp), dtype=torch.float64, device="cuda")
    wsc = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(comp)), dtype=torch.uint8, device="cuda")
    delayed = np.zeros(len(comp))
    for t in range(1, chunks):
        bdr.bdr_qsnr_delayed(comp, x[t * per:(t + 1) * per], hist[max(0, t - window):t], outc, wsc)
        delayed += outc.cpu().numpy()
    delayed /= chunks - 1                                  # mean of per-chunk dB, as the paper averages per-vector QSNR
    q = q_now.copy()
    q[441:] = delayed
    pts = [(n, sweep.bits_per_element(c) / bdr.bdr_tile_packing_efficiency(c), float(v)) for (n, c), v in zip(named, q)]
    front = sweep.pareto_frontier(pts)
    names = [n for n, _ in named]
    show = {"MX9": "bdr_k1=16_k2=2_d2=1_m=7", "MX6": "bdr_k1=16_k2=2_d2=1_m=4", "MX4": "bdr_k1=16_k2=2_d2=1_m=2",
            "MSFP16": "bdr_k1=16_k2=1_d2=0_m=7", "MSFP12": "bdr_k1=16_k2=1_d2=0_m=3", "INT8": "int8", "FP8_E4M3": "fp8_e4m3",
            "FP8_E5M2": "fp8_e5m2"}
    return {"paper_sweep": {"workload": "16,384 x 1,024 fp32 ~ N(0,|N(0,1)|), 457 configurations in one bdr_qsnr call",
                            "ms": ms, "configs_per_s": len(cfgs) / (ms * 1e-3),
                            "qsnr_db": {k: float(q[names.index(v)]) for k, v in show.items()},
                            "qsnr_db_current_amax": {k: float(q_now[names.index(v)]) for k, v in show.items() if names.index(v) >= 441},
                            "delayed_scaling": "FP32 kinds: maximum over the %d previous chunks of %d vectors, mean of per-chunk dB" % (window, per),
                            "packing_efficiency_256_in_64B": {k: bdr.bdr_tile_packing_efficiency(cfgs[names.index(v)]) for k, v in show.items()},
                            "frontier": [{"name": n, "bits_over_packing_efficiency": c, "qsnr_db": v} for n, c, v in front]}}
