"""GPU parity of bdr_quant_dequant_parent (FP32 parent scale above the two-level quantizer, the extension sketched at the
end of Section III): dequantized values bit for bit against the oracle, the sums within the QSNR tolerance."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

C_ = bdr.Config


@pytest.mark.parametrize("cfg", [bdr.MX4, bdr.MX6, bdr.MX9, C_(16, 8, 4, 2, 5), C_(8, 8, 1, 1, 3), C_(1, 8, 1, 0, 8),
                                 C_(16, 8, 2, 1, 4, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY)], ids=str)
def test_parent_scale_matches_oracle(cfg):
    o = H.to_orc(cfg)
    for kind, rows, cols, kp, axis, ld in (("laplace_outliers", 16, 2048, 1024, 1, None), ("normal", 7, 1000, 256, 1, 1003),
                                           ("edge", 4, 512, 64, 1, None), ("normal", 300, 24, 128, 0, None), ("tiny", 3, 96, 32, 1, None)):
        x = H.make_input(kind, rows, cols, "f32", seed=61)
        if kind == "edge":
            x = np.clip(x, -1e30, 1e30).astype(np.float32)
            x[1, :] = 0.0
            x[1, 5] = -0.0
        xd = H.host_to_device(x, "f32", ld)
        y = torch.zeros_like(xd) if ld is None else H.host_to_device(np.zeros_like(x), "f32", ld)
        sums = torch.zeros(2, dtype=torch.float64, device="cuda")
        bdr.bdr_quant_dequant_parent(cfg, kp, xd, y, axis=axis, qsnr_sums=sums)
        torch.cuda.synchronize()
        want, so = orc.quant_dequant_parent(o, kp, x, axis=axis)
        H.assert_bits_equal(H.device_to_host_f32(y), want, "%s %s k_parent=%d axis=%d" % (cfg, kind, kp, axis))
        H.assert_qsnr_close(sums.cpu().numpy(), so, "%s %s" % (cfg, kind))


def test_parent_scale_argument_checks_and_sums_only():
    x = torch.randn(4, 256, device="cuda")
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_quant_dequant_parent(bdr.MX6, 256, x, None, qsnr_sums=sums)          # sums only
    torch.cuda.synchronize()
    _, so = orc.quant_dequant_parent(orc.MX6, 256, x.cpu().numpy())
    H.assert_qsnr_close(sums.cpu().numpy(), so)
    for cfg, kp, status in ((bdr.MX6, 24, -2), (bdr.MX6, 2048, -3), (C_(32, 8, 2, 1, 4), 64, -3), (C_(16, 8, 3, 1, 4), 64, -2)):
        with pytest.raises(bdr.BdrError) as e:
            bdr.bdr_quant_dequant_parent(cfg, kp, x, torch.empty_like(x))
        assert e.value.status == status
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_quant_dequant_parent(bdr.MX6, 64, x.to(torch.bfloat16), torch.empty_like(x, dtype=torch.bfloat16))
    assert e.value.status == -3
    torch.cuda.synchronize()


@pytest.mark.parametrize("kp", [16, 64, 256, 512, 1024])
def test_parent_scale_row_kernel_on_groups_with_a_wide_dynamic_range(kp):
    # whole groups along contiguous rows (the fast kernel): every block of a group scaled by a random power of two over 80
    # binades, so that the quotients x / s run from about 1 down to far below the block unit, plus zero and tiny groups
    rng = np.random.default_rng(62 + kp)
    rows, cols = 33, 4096
    x = (synth.normal_matrix(rows, cols, seed=63) * np.repeat(2.0 ** rng.integers(-70, 11, (rows, cols // 16)), 16, axis=1)).astype(np.float32)
    x[3, :kp] = 0.0
    x[4, :kp] = synth.normal(kp, 64) * np.float32(1e-37)
    x[5, :kp] = synth.normal(kp, 65) * np.float32(1e30)
    for cfg in (bdr.MX4, bdr.MX9, C_(16, 8, 8, 2, 5), C_(16, 8, 1, 3, 6)):
        xd = H.host_to_device(x, "f32")
        y = torch.zeros_like(xd)
        sums = torch.zeros(2, dtype=torch.float64, device="cuda")
        bdr.bdr_quant_dequant_parent(cfg, kp, xd, y, axis=1, qsnr_sums=sums)
        torch.cuda.synchronize()
        want, so = orc.quant_dequant_parent(H.to_orc(cfg), kp, x, axis=1)
        H.assert_bits_equal(H.device_to_host_f32(y), want, "%s k_parent=%d" % (cfg, kp))
        H.assert_qsnr_close(sums.cpu().numpy(), so, "%s k_parent=%d" % (cfg, kp))
