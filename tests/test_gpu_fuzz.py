"""Randomised dispatch test: shapes, pitches and base-pointer offsets chosen so that every kernel family
(packed-arithmetic bf16 kernels, generic row / column kernels, general kernels) and the fall-backs between
them are reached; every result is compared bit for bit with the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

CONFIGS = [bdr.MX4, bdr.MX6, bdr.MX9, bdr.Config(16, 8, 2, 1, 5), bdr.Config(32, 8, 4, 2, 4), bdr.Config(16, 8, 16, 0, 7),
           bdr.Config(64, 8, 2, 1, 3), bdr.Config(16, 8, 2, 1, 4, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY)]
ROWS = [1, 3, 16, 32, 100, 256, 512]
COLS = [16, 48, 100, 128, 512, 1024, 2048, 4096]


def _device_view(x_f32, dtype, ld, offset):
    """x on the device as a [rows, cols] view with row pitch ld that starts `offset` elements into its buffer."""
    rows, cols = x_f32.shape
    t = torch.from_numpy(np.ascontiguousarray(x_f32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    buf = torch.zeros(offset + rows * ld, dtype=t.dtype, device="cuda")
    view = buf[offset:offset + rows * ld].view(rows, ld)[:, :cols]
    view.copy_(t.cuda())
    return view


@pytest.mark.parametrize("seed", range(48))
def test_random_shapes_pitches_and_offsets(seed):
    rng = np.random.default_rng(1000 + seed)
    cfg = CONFIGS[int(rng.integers(len(CONFIGS)))]
    dtype = "bf16" if rng.random() < 0.7 else "f32"
    axis = int(rng.integers(2))
    rows, cols = int(ROWS[rng.integers(len(ROWS))]), int(COLS[rng.integers(len(COLS))])
    pad = int(rng.choice([0, 0, 0, 8, 16, 24, 3]))
    offset = int(rng.choice([0, 0, 0, 8, 16, 1]))
    ld = cols + pad
    kind = ["normal", "edge", "laplace_outliers"][int(rng.integers(3))]
    x = H.make_input(kind, rows, cols, dtype, seed=seed)
    what = "seed %d: %s %s axis=%d %dx%d ld=%d offset=%d %s" % (seed, cfg, dtype, axis, rows, cols, ld, offset, kind)
    ocfg = H.to_orc(cfg)
    want, so = orc.quant_dequant(ocfg, x, axis=axis)

    xd = _device_view(x, dtype, ld, offset)
    yd = _device_view(np.zeros_like(x), dtype, ld, offset)
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_quant_dequant(cfg, xd, yd, axis=axis, qsnr_sums=sums)
    torch.cuda.synchronize()
    H.assert_bits_equal(H.device_to_host_f32(yd), want, what + " quant_dequant")
    H.assert_qsnr_close(sums.cpu().numpy(), so, what)

    planes = bdr.alloc_planes(cfg, rows, cols, axis)
    with_y = bool(rng.integers(2))
    yq = _device_view(np.zeros_like(x), dtype, ld, offset) if with_y else None
    bdr.bdr_pack(cfg, xd, planes, axis=axis, y_dq=yq)
    back = _device_view(np.full_like(x, 7.0), dtype, ld, offset)
    bdr.bdr_unpack(cfg, planes, back, axis=axis)
    torch.cuda.synchronize()
    H.assert_planes_equal(H.planes_to_host(planes), orc.pack(ocfg, x, axis=axis), what)
    if with_y:
        H.assert_bits_equal(H.device_to_host_f32(yq), want, what + " y_dq")
    H.assert_bits_equal(H.device_to_host_f32(back), want, what + " unpack")
    assert bdr.bdr_device_status() == 0
