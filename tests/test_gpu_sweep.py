"""GPU parity of bdr_qsnr (the design-space sweep) against the oracle: QSNR within 1e-6 dB relative."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import sweep, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def run_sweep(cfgs, x_host, dtype="f32", ld=None, axis=1):
    x = H.host_to_device(x_host, dtype, ld)
    out = torch.full((len(cfgs),), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
    bdr.bdr_qsnr(cfgs, x, out, ws, axis=axis)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def check(cfgs, got, x, what="", axis=1):
    for cfg, g in zip(cfgs, got):
        want = orc.qsnr(H.to_orc(cfg), x, axis=axis)
        if math.isnan(want) or math.isinf(want):
            assert (math.isnan(g) and math.isnan(want)) or g == want, (what, cfg, g, want)
        else:
            assert abs(g - want) <= H.QSNR_REL_TOL * max(abs(want), 1e-3), (what, cfg, g, want)


def test_sweep_workload_has_the_documented_size():
    names = [n for n, _ in sweep.sweep_configs()]
    assert len(sweep.bdr_grid()) == 441 and len(names) == 457 and len(set(names)) == 457


@pytest.mark.parametrize("dist", synth.SWEEP_DISTRIBUTIONS)
def test_full_sweep_on_each_distribution(dist):
    cfgs = [c for _, c in sweep.sweep_configs()]
    x = synth.sweep_distribution(dist, 1 << 16, seed=1).reshape(1, -1)
    check(cfgs, run_sweep(cfgs, x), x, dist)


def test_sweep_ragged_rows_pitch_and_bf16():
    cfgs = [c for _, c in sweep.sweep_configs()][::5] + [c for _, c in sweep.comparators()]
    x = synth.normal_with_outliers(7 * 5000, seed=3).reshape(7, 5000)      # rows are lines; 5000 is not a multiple of 16
    check(cfgs, run_sweep(cfgs, x, ld=5008), x, "ragged")
    xb = H.make_input("laplace_outliers", 3, 4096 + 512, "bf16", seed=4)
    check(cfgs, run_sweep(cfgs, xb, dtype="bf16"), xb, "bf16")


def test_sweep_along_columns():
    # axis 0: the lines are columns (the reduction dimension of half of a training step's operands, Section V);
    # blocks, sub-blocks and VSQ vectors run down a column.  Every configuration against the oracle on a
    # matrix whose outlier channels are columns, then ragged shapes with a pitch, bf16, and columns longer
    # than one 4096-element tile.
    cfgs = [c for _, c in sweep.sweep_configs()]
    x = synth.outlier_channel_matrix(1024, 64, seed=11, gain=50.0)
    got = run_sweep(cfgs, x, axis=0)
    check(cfgs, got, x, "columns", axis=0)
    rows_dir = run_sweep(cfgs, x, axis=1)
    assert np.abs(got[:441] - rows_dir[:441]).max() > 0.1       # the direction matters on this input
    some = cfgs[::7] + [c for _, c in sweep.comparators()]
    xr = synth.normal_with_outliers(5000 * 7, seed=12).reshape(5000, 7)   # 5000 is not a multiple of 16; 2 tiles per column
    check(some, run_sweep(some, xr, ld=12, axis=0), xr, "ragged columns", axis=0)
    xb = H.make_input("laplace_outliers", 4096 + 512, 6, "bf16", seed=13)
    check(some, run_sweep(some, xb, dtype="bf16", axis=0), xb, "bf16 columns", axis=0)
    one = synth.normal(777, 14).reshape(777, 1)
    check(some, run_sweep(some, one, axis=0), one, "single column", axis=0)
    check(some, run_sweep(some, one.reshape(1, 777), axis=0), one.reshape(1, 777), "columns of one element", axis=0)


def test_sweep_extra_configs_edge_values_and_ties_away():
    C = bdr.Config
    cfgs = [C(1, 8, 1, 0, 8), C(2, 8, 1, 1, 3), C(4, 8, 2, 2, 5), C(16, 8, 16, 1, 4), C(512, 8, 4, 3, 6),
            C(16, 8, 2, 1, 4, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY), C(0, 32, 1, 0, 7, bdr.SCALE_FP32_INT, bdr.ROUND_NEAREST_AWAY),
            C(0, 32, 1, 4, 3, bdr.SCALE_FP32_FP, bdr.ROUND_NEAREST_AWAY), C(0, 32, 16, 6, 3, bdr.SCALE_FP32_VSQ, bdr.ROUND_NEAREST_AWAY),
            C(0, 32, 1, 3, 2, bdr.SCALE_FP32_FP), C(0, 32, 1, 0, 1, bdr.SCALE_FP32_INT)]
    for kind in ("edge", "tiny", "normal"):
        x = H.make_input(kind, 2, 8192, "f32", seed=6)
        if kind == "edge":
            x = np.clip(x, -1e30, 1e30).astype(np.float32)       # keep x/s finite for the FP32-scaled kinds
        check(cfgs, run_sweep(cfgs, x), x, kind)


def test_sweep_degenerate_tensors_and_errors():
    cfgs = [bdr.MX6, bdr.Config(0, 32, 1, 0, 7, bdr.SCALE_FP32_INT)]
    z = np.zeros((1, 4096), dtype=np.float32)
    got = run_sweep(cfgs, z)
    assert np.isnan(got).all()                                  # no signal: QSNR undefined
    exact = np.tile(np.array([1.0, 0.5, -0.25, 1.75], dtype=np.float32), 1024).reshape(1, -1)
    assert math.isinf(run_sweep([bdr.MX6], exact)[0])           # representable input: no noise
    x = torch.zeros((4, 64), device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_qsnr([bdr.MX6], x, out, ws)
    assert e.value.status == -6
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(1), dtype=torch.uint8, device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_qsnr([bdr.MX6], x, out, ws, axis=2)
    assert e.value.status == -2
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_qsnr([bdr.Config(16, 8, 3, 1, 4)], x, out, ws)
    assert e.value.status == -2
    torch.cuda.synchronize()


def test_full_size_sweep_on_sampled_configurations():
    # the benchmark's sweep workload itself: all 457 configurations over 2^24 values in one call (the launch
    # bench.py times); the oracle recomputes every 12th configuration and all comparators one by one
    cfgs = [c for _, c in sweep.sweep_configs()]
    x = synth.sweep_distribution("normal_outliers", 1 << 24, seed=0).reshape(1, -1)
    got = run_sweep(cfgs, x)
    picked = list(range(0, 441, 12)) + list(range(441, 457))
    for i in picked:
        want = orc.qsnr(H.to_orc(cfgs[i]), x, nthreads=16)
        assert abs(got[i] - want) <= H.QSNR_REL_TOL * max(abs(want), 1e-3), (i, cfgs[i], got[i], want)
    assert np.isfinite(got).all()


def test_first_level_maximum_from_a_window_of_past_tensors():
    # Fig. 7 caption: INT / FP / VSQ take their FP32 scale from the maximum over a window of past vectors.  bdr_amax
    # gives each past tensor's maximum (checked against numpy), bdr_qsnr_delayed uses the largest of the window; the
    # oracle is handed that maximum.  Windows above, equal to and below the current tensor's own maximum (then
    # values saturate); the power-of-two formats do not depend on it.
    cfgs = [c for _, c in sweep.comparators()] + [bdr.MX6, bdr.MX9,
            bdr.Config(0, 32, 1, 0, 7, bdr.SCALE_FP32_INT, bdr.ROUND_NEAREST_AWAY), bdr.Config(0, 32, 16, 6, 3, bdr.SCALE_FP32_VSQ, bdr.ROUND_NEAREST_AWAY)]
    x = synth.variable_variance_vectors(512, 1024, seed=21)
    xd = torch.from_numpy(x).cuda()
    cur = float(np.abs(x).max())
    past = [synth.variable_variance_vectors(64, 1024, seed=22 + i) * np.float32(sc) for i, sc in enumerate((0.5, 1.5, 0.25))]
    window = torch.zeros(len(past), dtype=torch.float32, device="cuda")
    for i, t in enumerate(past):
        bdr.bdr_amax(torch.from_numpy(t).cuda(), window[i:i + 1])
    bb = torch.from_numpy(synth.f32_to_bf16_bits(past[0]).view(np.int16)).view(torch.bfloat16).cuda().reshape(64, 1024)
    a16 = torch.zeros(1, dtype=torch.float32, device="cuda")
    bdr.bdr_amax(bb[:, :1000], a16)                                    # bf16, a pitch: 1000 of 1024 columns
    torch.cuda.synchronize()
    assert window.cpu().tolist() == [float(np.abs(t).max()) for t in past]
    assert a16.item() == float(np.abs(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(past[0])).reshape(64, 1024)[:, :1000]).max())
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
    out = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
    for win in (window, window[:1], window[2:], torch.tensor([cur], dtype=torch.float32, device="cuda"),
                torch.tensor([cur * 0.01, 0.0], dtype=torch.float32, device="cuda")):
        amax = float(win.max().item())
        bdr.bdr_qsnr_delayed(cfgs, xd, win, out, ws)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        for cfg, g in zip(cfgs, got):
            o = H.to_orc(cfg)
            want = orc.qsnr(o, x, amax=None if cfg.scale_kind == bdr.SCALE_POW2 else amax)
            assert abs(g - want) <= H.QSNR_REL_TOL * max(abs(want), 1e-3), (cfg, amax, g, want)
    same = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
    bdr.bdr_qsnr(cfgs, xd, same, ws)                                   # window = the tensor's own maximum: plain bdr_qsnr
    bdr.bdr_qsnr_delayed(cfgs, xd, torch.tensor([cur], dtype=torch.float32, device="cuda"), out, ws)
    torch.cuda.synchronize()
    assert torch.allclose(same, out, rtol=1e-12, atol=0)               # the same arithmetic; only the order of the fp64 atomics differs
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_qsnr_delayed(cfgs, xd, window[:0], out, ws)
    assert e.value.status == -5
    torch.cuda.synchronize()


def test_qsnr_from_sums_is_eq3_on_pairs():
    pairs = np.array([[1.0, 100.0], [3.5e-7, 2.25], [0.0, 4.0], [1.0, 0.0], [0.0, 0.0], [7.0, 7.0], [1e-300, 1e300]], dtype=np.float64)
    sums = torch.from_numpy(pairs).cuda()
    out = torch.full((len(pairs),), -1.0, dtype=torch.float64, device="cuda")
    bdr.bdr_qsnr_from_sums(sums, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for (e, s_), g in zip(pairs, got):
        want = orc.qsnr_db(e, s_)
        if math.isnan(want) or math.isinf(want):
            assert (math.isnan(g) and math.isnan(want)) or g == want, (e, s_, g, want)
        else:
            assert abs(g - want) <= 1e-12 * max(abs(want), 1.0), (e, s_, g, want)
    assert torch.equal(sums.cpu(), torch.from_numpy(pairs))          # the sums are only read


def test_short_contiguous_rows_are_swept_as_one_long_line_without_changing_the_result():
    # 1,024-element vectors (the paper's sweep workload): every block size of the grid divides the row, so the kernel treats the
    # contiguous tensor as one long row; a pitch, or a row length some block size does not divide, keeps the rows apart
    cfgs = [c for _, c in sweep.sweep_configs()]
    x = synth.variable_variance_vectors(48, 1024, seed=31)
    check(cfgs, run_sweep(cfgs, x), x, "merged rows")
    check(cfgs[::9], run_sweep(cfgs[::9], x, ld=1040), x, "pitched rows")
    x2 = synth.variable_variance_vectors(40, 1536, seed=32)          # 1536 is not a multiple of 1024: blocks of 1024 are ragged per row
    check(cfgs[::9] + cfgs[430:457], run_sweep(cfgs[::9] + cfgs[430:457], x2), x2, "rows kept apart")
