"""The allocation-free sweep entry point, bdr_qsnr_static.

Some callers may not allocate device memory at all -- code that runs inside another framework's
step, where that framework's pool owns the GPU's memory and a cudaMalloc would both risk failing and
stall the device.  For them the library carries its own small scratch array.  This test calls the
entry point through the C ABI twice in a row (the scratch keeps the previous call's contents, so the
second call proves it is cleared) and checks both results against the ordinary bdr_qsnr, within the
QSNR tolerance the other tests use, and a sample of them (every 12th grid point and every comparator) against
the CPU oracle, so that the expected values do not come from the library alone.  A further call uses exactly
as many configurations as the scratch holds.  It lives in a file that pytest collects last.
"""
import math

import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import sweep, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _close(a, b):
    if math.isnan(a) or math.isnan(b) or math.isinf(a) or math.isinf(b):
        return (math.isnan(a) and math.isnan(b)) or a == b
    return abs(a - b) <= H.QSNR_REL_TOL * max(abs(b), 1e-3)


def test_static_scratch_sweep_matches_workspace_sweep_twice_in_a_row():
    cfgs = [c for _, c in sweep.sweep_configs()]
    assert len(cfgs) <= bdr.bdr_qsnr_static_max_cfgs()
    inputs = [torch.from_numpy(synth.sweep_distribution("laplace", 3 * 40000, seed=7)).cuda().reshape(3, 40000),
              torch.from_numpy(synth.sweep_distribution("normal_outliers", 1 << 16, seed=8)).cuda().reshape(1, -1)]
    ws = torch.empty(bdr.bdr_qsnr_workspace_bytes(len(cfgs)), dtype=torch.uint8, device="cuda")
    for x in inputs:                                  # two calls in a row share the built-in scratch
        want = torch.empty(len(cfgs), dtype=torch.float64, device="cuda")
        got = torch.full((len(cfgs),), -1.0, dtype=torch.float64, device="cuda")
        bdr.bdr_qsnr(cfgs, x, want, ws)
        bdr.bdr_qsnr_static(cfgs, x, got)
        torch.cuda.synchronize()
        got_h = got.cpu().tolist()
        for cfg, g, w in zip(cfgs, got_h, want.cpu().tolist()):
            assert _close(g, w), (cfg, g, w)
        x_h = x.cpu().numpy()
        for i in list(range(0, 441, 12)) + list(range(441, len(cfgs))):
            w = orc.qsnr(H.to_orc(cfgs[i]), x_h)
            assert _close(got_h[i], w), ("oracle", cfgs[i], got_h[i], w)


def test_static_scratch_sweep_with_exactly_as_many_configurations_as_it_holds():
    n = bdr.bdr_qsnr_static_max_cfgs()
    base = [c for _, c in sweep.sweep_configs()]
    cfgs = (base + base)[:n]                           # repeats are legal: every entry has its own accumulators
    assert len(cfgs) == n
    x_h = synth.sweep_distribution("student_t3", 1 << 15, seed=9).reshape(1, -1)
    x = torch.from_numpy(x_h).cuda()
    got = torch.full((n,), -1.0, dtype=torch.float64, device="cuda")
    bdr.bdr_qsnr_static(cfgs, x, got)
    torch.cuda.synchronize()
    got_h = got.cpu().tolist()
    for i in (0, 5, 440, 441, 456, 457, n - 1):         # first, last and the entries around the repeat
        w = orc.qsnr(H.to_orc(cfgs[i]), x_h)
        assert _close(got_h[i], w), (i, cfgs[i], got_h[i], w)
    assert got_h[457:n] == got_h[:n - 457]              # the second copy of a configuration gives the same number


def test_static_scratch_sweep_rejects_more_configurations_than_it_holds():
    x = torch.zeros((1, 256), device="cuda")
    n = bdr.bdr_qsnr_static_max_cfgs() + 1
    out = torch.empty(n, dtype=torch.float64, device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_qsnr_static([bdr.MX6] * n, x, out)
    assert e.value.status == -5
    torch.cuda.synchronize()
