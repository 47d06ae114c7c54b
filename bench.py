#!/usr/bin/env python
"""Benchmark of the BDR/MX hot path on B200.

One "step" = one pass of the whole quantization path over one 8192 x 8192 bf16 activation tensor
(Laplace(0,1), 1% outlier columns x50): for each of MX4 / MX6 / MX9 and each direction (row-wise,
column-wise) a quantize-dequantize with fused QSNR sums, a quantize+pack, and an unpack+dequantize
-- 18 kernel launches.  `value` is the algorithmic bytes those 18 operations
must move divided by the device time (GB/s); the MX-GEMM, design-sweep, linear-layer and small-vector legs are
measured separately after the timed steps and reported in the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --only pack --fmt MX6 --axis 0 [--rows R --cols C --reps N]     # one operation, for profilers
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

ROWS, COLS = 8192, 8192
FORMATS = (("MX4", 2), ("MX6", 4), ("MX9", 7))  # name, m  (k1=16, d1=8, k2=2, d2=1: Table II)
METRIC = "MX quant-dequant GB/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of each of the step's kernels on the
# bench workload itself (8192 x 8192 bf16), from the committed ncu capture
# profiles/step_kernels_dram_traffic.md.  Writes that still sit in L2 when a kernel ends are not
# counted by those counters, which is why some figures are below the algorithmic bytes.
NCU_TRAFFIC_BYTES: dict[str, float | None] = {
    "quant_dequant_MX4_row": 216465664, "quant_dequant_MX4_col": 216645888,
    "quant_dequant_MX6_row": 216837632, "quant_dequant_MX6_col": 215354368,
    "quant_dequant_MX9_row": 216819712, "quant_dequant_MX9_col": 216272128,
    "pack_MX4_row": 149406720, "pack_MX4_col": 146448384,
    "pack_MX6_row": 157472768, "pack_MX6_col": 154535680,
    "pack_MX9_row": 173253888, "pack_MX9_col": 168492800,
    "unpack_MX4_row": 111284224, "unpack_MX4_col": 109175808,
    "unpack_MX6_row": 128216832, "unpack_MX6_col": 127134464,
    "unpack_MX9_row": 154121472, "unpack_MX9_col": 151977728,
}


def bits_per_element(m: int) -> float:
    return (m + 1) + 8 / 16 + 1 / 2


def op_bytes(op: str, m: int, n_elems: int) -> float:
    """Algorithmic bytes of one operation on bf16 data: what the method itself must move."""
    packed = bits_per_element(m) / 8.0
    per_elem = {"quant_dequant": 2.0 + 2.0, "pack": 2.0 + packed, "unpack": packed + 2.0}[op]
    return per_elem * n_elems


def step_bytes(n_elems: int) -> float:
    return sum(op_bytes(op, m, n_elems) for _, m in FORMATS for _axis in (1, 0) for op in ("quant_dequant", "pack", "unpack"))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured", d
    except Exception:
        return FALLBACK_HBM_GBS, "fallback", {}


def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """The job's time is the slowest rank's time (all-reduce MAX); identity for one rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job GB/s of `world` independent replicas that each move bytes_per_rank per step."""
    return bytes_per_rank * world / (ms_per_step * 1e-3) / 1e9


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines: list[str] = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded sample of the same workload
# ---------------------------------------------------------------------------------------------------
def oracle_step(x_f32: np.ndarray, nthreads: int) -> float:
    """Runs the step's 18 operations with the oracle on x_f32 (rows split over threads for axis 1,
    columns for axis 0; ctypes releases the GIL).  Returns seconds."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle as orc

    rows, cols = x_f32.shape

    def one(cfg, axis, part):
        xs = np.ascontiguousarray(x_f32[part, :] if axis == 1 else x_f32[:, part])
        r, c = xs.shape
        orc.quant_dequant(cfg, xs, axis=axis)
        planes = orc.pack(cfg, xs, axis=axis)
        orc.unpack(cfg, planes, r, c, axis=axis)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=nthreads) as ex:
        for _, m in FORMATS:
            cfg = orc.Config(16, 8, 2, 1, m)
            for axis in (1, 0):
                n = rows if axis == 1 else cols
                chunk = -(-n // nthreads)
                chunk = -(-chunk // 16) * 16
                parts = [slice(i, min(n, i + chunk)) for i in range(0, n, chunk)]
                list(ex.map(lambda p: one(cfg, axis, p), parts))
    return time.perf_counter() - t0


def cpu_sample(x_bits: np.ndarray, sample_rows: int) -> np.ndarray:
    from paper_2302_08007_b200 import synth
    return synth.bf16_bits_to_f32(x_bits[:sample_rows]).reshape(sample_rows, -1)


def run_reference(args):
    """--impl reference: the oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    from paper_2302_08007_b200 import synth
    orc.build()
    cores = len(os.sched_getaffinity(0))
    sample_rows = 1024
    x = synth.outlier_channel_matrix(sample_rows, COLS, seed=0, stream=3, frac=0.01, gain=50.0)
    xs = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x)).reshape(sample_rows, COLS)
    for _ in range(args.warmup):
        oracle_step(xs, cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(xs, cores)
    dt = time.perf_counter() - t0
    gbs = step_bytes(xs.size) * args.steps / dt / 1e9
    sample = "%d x %d slice of the 8192 x 8192 tensor per step, all 18 operations" % (sample_rows, COLS)
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "C3: 8192x8192 bf16 Laplace(0,1), 1% outlier columns x50; MX4/MX6/MX9 x row/column x "
                                   "(quant-dequant, pack, unpack); CPU oracle on a bounded sample"},
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------------
N_SETS = 3   # buffer sets rotated so that no launch finds its input in L2 (126 MB)
REPEATS = 10  # the K-step timed region is measured this many times; the headline is the median


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2302_08007_b200 import binding as bdr
    from paper_2302_08007_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    bdr.lib()  # fail loudly if the CUDA library is missing

    # every rank quantizes its own tensor (independent replicas of the path: no data-path collective)
    x_host = synth.outlier_channel_matrix(ROWS, COLS, seed=rank, stream=3, frac=0.01, gain=50.0)
    x_bits = synth.f32_to_bf16_bits(x_host)
    del x_host
    x_pinned = torch.from_numpy(x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    n_elems = x_pinned.numel()

    cfgs = {name: bdr.Config(16, 8, 2, 1, m) for name, m in FORMATS}
    # N_SETS copies of (x, y, planes).  Operation j of step s reads x[(s + j) % N_SETS] and writes y[(s + j) % N_SETS];
    # the packs of step s write plane set s % N_SETS and its unpacks read plane set (s + 1) % N_SETS, which was
    # written two steps (7.7 GB of traffic) earlier.  So no launch reads what one of the two launches before it
    # read or wrote, and every byte a kernel reads comes from HBM, not from the 126 MB L2.
    xs = [x_pinned.cuda() for _ in range(N_SETS)]
    ys = [torch.empty_like(xs[0]) for _ in range(N_SETS)]
    plane_sets = [{(name, axis): bdr.alloc_planes(cfgs[name], ROWS, COLS, axis) for name, _ in FORMATS for axis in (1, 0)}
                  for _ in range(N_SETS)]
    ops = [(name, m, axis, op) for op in ("quant_dequant", "pack", "unpack") for name, m in FORMATS for axis in (1, 0)]
    sums = torch.zeros((len(ops), 2), dtype=torch.float64, device="cuda")
    sum_views = [sums[i] for i in range(len(ops))]  # made once: no tensor indexing on the launch path

    def run_op(j, s, x_override=None, y_override=None, planes_override=None):
        name, _m, axis, op = ops[j]
        k = (s + j) % N_SETS
        src = xs[k] if x_override is None else x_override
        dst = ys[k] if y_override is None else y_override
        if op == "quant_dequant":
            bdr.bdr_quant_dequant(cfgs[name], src, dst, axis=axis, qsnr_sums=sum_views[j])
        elif op == "pack":
            pl = plane_sets[s % N_SETS] if planes_override is None else planes_override
            bdr.bdr_pack(cfgs[name], src, pl[(name, axis)], axis=axis)
        else:
            pl = plane_sets[(s + 1) % N_SETS] if planes_override is None else planes_override
            bdr.bdr_unpack(cfgs[name], pl[(name, axis)], dst, axis=axis)

    def step_direct(s):
        for j in range(len(ops)):
            run_op(j, s)

    def capture(fn):
        """One CUDA graph of fn's launches (the library allocates nothing and never synchronises, so its
        calls can be captured); the launches then replay without the Python/ctypes cost per call."""
        fn()  # first calls outside capture: function attributes, symbol look-ups
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g.replay

    for s in range(N_SETS):   # every plane set is filled before anything reads it
        step_direct(s)
    torch.cuda.synchronize()
    use_graph = not args.no_graph
    if use_graph:
        graphs = [capture(lambda s=s: step_direct(s)) for s in range(N_SETS)]
        step = lambda s: graphs[s % N_SETS]()
    else:
        step = step_direct

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for s in range(args.warmup):
        step(s)
    barrier()
    if args.step_only:   # for a profiler's launch list: nothing but the step's launches
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for s in range(args.steps):
            step(s)
        ev1.record()
        barrier()
        if rank == 0:
            print("step only: %d steps of %d launches, %.4f ms per step" % (args.steps, len(ops), ev0.elapsed_time(ev1) / args.steps))
        if world > 1:
            dist.destroy_process_group()
        return

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    times = []
    for _rep in range(REPEATS):   # each repetition: exactly K steps between barrier + synchronize
        sums.zero_()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for s in range(args.steps):
            step(s)
        ev1.record()
        barrier()
        times.append(max_over_ranks(ev0.elapsed_time(ev1), world) / args.steps)
    clocks = sampler.stop() if rank == 0 else {}
    ms_per_step = float(np.median(times))
    ms_best = float(min(times))
    value = aggregate_value(step_bytes(n_elems), world, ms_per_step)
    db = bdr.bdr_qsnr_from_sums(sums, torch.empty(len(ops), dtype=torch.float64, device="cuda")).cpu().numpy()
    qsnr = {"%s_axis%d" % (name, axis): float(db[j]) for j, (name, _m, axis, op) in enumerate(ops) if op == "quant_dequant"}

    # ---- per-kernel timing on the launching stream (roofline of the dominant kernel) ----
    # one graph of ROUNDS x N_SETS launches of the operation, cycling through the buffer sets, replayed: consecutive
    # launches never touch the same buffers, so inputs (also the 34-76 MB of planes an unpack reads) come from HBM,
    # and the gap between two graph replays is spread over a dozen launches
    kernels = {}
    reps = max(5, min(args.steps, 20))
    ROUNDS = 4
    for j, (name, m, axis, op) in enumerate(ops):
        def rot(j=j):
            for _r in range(ROUNDS if use_graph else 1):
                for s in range(N_SETS):
                    run_op(j, s, planes_override=plane_sets[s])
        launch = capture(rot) if use_graph else rot
        launch()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            launch()
        b.record()
        torch.cuda.synchronize()
        dur_ms = a.elapsed_time(b) / (reps * N_SETS * (ROUNDS if use_graph else 1))
        key = "%s_%s_%s" % (op, name, "row" if axis == 1 else "col")
        kernels[key] = {"ms": dur_ms, "GBps": op_bytes(op, m, n_elems) / (dur_ms * 1e-3) / 1e9}
    peak, peak_kind, peaks = measured_peaks()
    dom = max(kernels, key=lambda k: kernels[k]["ms"])
    for k in kernels.values():
        k["frac"] = k["GBps"] / peak
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak, "unit": "GB/s",
                "frac": kernels[dom]["GBps"] / peak, "peak_source": peak_kind,
                "traffic": NCU_TRAFFIC_BYTES.get(dom),
                "achieved_kind": "algorithmic bytes / CUDA-event time, rotating %d buffer sets" % N_SETS}

    # ---- end to end through the C ABI with host buffers ----
    # Every step copies its input from pinned host memory, runs the 18 C-ABI calls, and copies back to pinned host
    # memory what the caller of each call receives: the dequantized tensor of every quantize-dequantize and unpack,
    # the three planes of every pack, and the QSNR sums.  Copy streams in both directions overlap the kernels.
    e2e_steps = max(2, min(args.steps, 3))
    xin = [torch.empty_like(xs[0]) for _ in range(2)]
    y_dev = [torch.empty_like(xs[0]) for _ in range(len(ops))]            # one output tensor per operation
    y_host = [torch.empty((ROWS, COLS), dtype=torch.bfloat16).pin_memory() if ops[j][3] != "pack" else None for j in range(len(ops))]
    e2e_planes = plane_sets[0]
    planes_host = {k: tuple(torch.empty(t.shape, dtype=torch.uint8).pin_memory() for t in (p.exps, p.micro, p.elems))
                   for k, p in e2e_planes.items()}
    sums_host = torch.empty((len(ops), 2), dtype=torch.float64).pin_memory()
    h2d, d2h = torch.cuda.Stream(), torch.cuda.Stream()
    main_stream = torch.cuda.current_stream()
    copied = [torch.cuda.Event() for _ in range(e2e_steps)]
    consumed = [torch.cuda.Event() for _ in range(e2e_steps)]
    drained = [torch.cuda.Event() for _ in range(e2e_steps)]
    d2h_bytes = 0
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    h2d.wait_event(e0)
    d2h.wait_event(e0)

    def enqueue_copy(i):
        with torch.cuda.stream(h2d):
            if i >= 2:
                h2d.wait_event(consumed[i - 2])  # the buffer's previous contents have been used
            xin[i % 2].copy_(x_pinned, non_blocking=True)
            copied[i].record(h2d)

    enqueue_copy(0)
    for i in range(e2e_steps):
        if i + 1 < e2e_steps:
            enqueue_copy(i + 1)
        main_stream.wait_event(copied[i])
        if i >= 1:
            main_stream.wait_event(drained[i - 1])   # the previous step's results have left the output buffers
        for j, (name, _m, axis, op) in enumerate(ops):   # the calls a user makes, one C-ABI call per operation
            run_op(j, 0, x_override=xin[i % 2], y_override=y_dev[j], planes_override=e2e_planes)
            done = torch.cuda.Event()
            done.record(main_stream)
            with torch.cuda.stream(d2h):
                d2h.wait_event(done)
                if op == "pack":
                    p = e2e_planes[(name, axis)]
                    for src_t, dst_t in zip((p.exps, p.micro, p.elems), planes_host[(name, axis)]):
                        dst_t.copy_(src_t, non_blocking=True)
                        d2h_bytes += src_t.numel() if i == 0 else 0
                else:
                    y_host[j].copy_(y_dev[j], non_blocking=True)
                    d2h_bytes += y_dev[j].numel() * 2 if i == 0 else 0
        consumed[i].record(main_stream)
        with torch.cuda.stream(d2h):
            d2h.wait_event(consumed[i])
            sums_host.copy_(sums, non_blocking=True)
            drained[i].record(d2h)
    main_stream.wait_event(drained[e2e_steps - 1])
    e1.record()
    barrier()
    d2h_bytes += sums.numel() * 8
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world)
    e2e = {"value": aggregate_value(step_bytes(n_elems), world, e2e_ms / e2e_steps), "unit": "GB/s",
           "h2d_bytes_per_step": n_elems * 2, "d2h_bytes_per_step": d2h_bytes, "ms_per_step": e2e_ms / e2e_steps,
           "steps": e2e_steps,
           "returns": "dequantized tensor of each quantize-dequantize and unpack, three planes of each pack, QSNR sums",
           "overlap": "host-to-device copy of the next step and device-to-host copies of finished operations on their own streams",
           "bound": "PCIe: %.2f GB cross the bus per step" % ((n_elems * 2 + d2h_bytes) / 1e9)}
    del y_dev, y_host, planes_host, xin

    extra = {}
    if rank == 0:
        args.peaks = peaks
        args.cpu_legs = world == 1
        extra = secondary_legs(args, bdr, synth, torch)

    cpu_baseline = None
    if rank == 0 and world == 1:
        from oracle import oracle as orc
        orc.build()
        cores = len(os.sched_getaffinity(0))
        sample_rows = 4096
        xs_cpu = cpu_sample(x_bits, sample_rows)
        sec = oracle_step(xs_cpu, cores)
        cpu_baseline = {"value": step_bytes(xs_cpu.size) / sec / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                        "sample": "first %d of %d rows, all 18 operations once (%.1f s)" % (sample_rows, ROWS, sec)}
        one_rows = 512   # the same oracle on one thread, on a sample an eighth as large
        xs_one = cpu_sample(x_bits, one_rows)
        sec1 = oracle_step(xs_one, 1)
        cpu_baseline["single_thread"] = {"value": step_bytes(xs_one.size) / sec1 / 1e9, "unit": "GB/s", "cores": 1,
                                         "sample": "first %d of %d rows, all 18 operations once (%.1f s)" % (one_rows, ROWS, sec1)}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "C3: 8192x8192 bf16 Laplace(0,1), 1% outlier columns x50; MX4/MX6/MX9 x "
                                       "row/column x (quant-dequant+QSNR, pack, unpack)",
                           "l2": "inputs larger than L2 and rotated: %d sets of (x, y, planes); no launch reads what either "
                                 "of the two launches before it read or wrote" % N_SETS,
                           "launch": "direct" if args.no_graph else "one CUDA graph of the 18 launches per step",
                           "replicas": "independent tensor per rank, no collective"},
                "repeats": REPEATS, "ms_per_step_best": ms_best, "ms_per_step_all": times,
                "value_kind": "median of %d repetitions of the %d-step timed region" % (REPEATS, args.steps),
                "frac_of_hbm_peak": value / world / peak, "roofline": roofline, "kernels": kernels,
                "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": len(ops) * args.steps, "clocks": clocks,
                "qsnr_db": qsnr}
        line.update(extra)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def secondary_legs(args, bdr, synth, torch) -> dict:
    """MX-GEMM TFLOP/s, design-sweep configs/s, the linear-layer step and the small-vector latency case."""
    import bench_legs as legs
    out = {}
    for fn in (legs.c1_leg, legs.gemm_leg, legs.sweep_leg, legs.paper_sweep_leg, legs.embedding_leg, legs.linear_leg):
        try:
            out.update(fn(args))
        except bdr.BdrError as e:
            out[fn.__name__] = {"unavailable": str(e)}
    # tensor roofline of the GEMM line: the measured cuBLAS bf16 burst figure (the call is timed alone); an 8-bit
    # contraction takes that figure times the nominal 8-bit : bf16 ratio of 2
    g = out.get("mx_gemm")
    if isinstance(g, dict) and "value" in g:
        _, src, peaks = measured_peaks()
        bf16_peak = float(peaks.get("bf16_tflops", FALLBACK_BF16_TFLOPS))
        f8 = g["entry_point"].startswith("mx_gemm_f8")
        peak = bf16_peak * (2.0 if f8 else 1.0)
        g["roofline"] = {"bound": "tensor", "dtype": "e4m3 x e4m3, e8m0 block scales, fp32 accumulate" if f8 else "bf16, fp32 accumulate",
                         "achieved": g["value"], "peak": peak, "unit": "TFLOP/s", "frac": g["value"] / peak,
                         "peak_source": ("measured bf16" if "bf16_tflops" in peaks else "fallback bf16") + (" x 2 (nominal 8-bit ratio)" if f8 else ""),
                         "frac_of_bf16_peak": g["value"] / bf16_peak}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from Python instead of replaying a CUDA graph of the step")
    ap.add_argument("--only", default=None, choices=["quant_dequant", "pack", "unpack", "pack2", "gemm", "gemm_ws", "gemm_f8", "gemm_hw", "sweep"],
                    help="run one operation a few times on a seeded tensor and print its time (for profilers); no JSON line")
    ap.add_argument("--step-only", action="store_true", help="run only the warm-up and the timed steps (18 launches each) and print the time; no JSON line")
    ap.add_argument("--fmt", default="MX6", choices=["MX4", "MX6", "MX9"])
    ap.add_argument("--axis", type=int, default=1)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--cols", type=int, default=8192)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--no-sums", action="store_true", help="--only quant_dequant / pack: without the fused QSNR sums")
    ap.add_argument("--no-y", action="store_true", help="--only quant_dequant: only the QSNR sums")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.only:
        import bench_legs
        return bench_legs.run_only(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
