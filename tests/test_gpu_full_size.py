"""The benchmark's own workload at full size: the 8192 x 8192 bf16 tensor bench.py generates, through the
18 operations of its step (MX4 / MX6 / MX9 x row / column x quantize-dequantize with sums, pack, unpack),
every output compared with the oracle in full -- values and packed bytes bit for bit, the Eq. 3 sums
within 1e-6 relative.  The kernels' launch configuration depends only on the shape and the format, so
these are the launches bench.py times (there replayed from a CUDA graph)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

ROWS = COLS = 8192
MX = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}


@pytest.fixture(scope="module")
def tensor():
    x = synth.outlier_channel_matrix(ROWS, COLS, seed=0, stream=3, frac=0.01, gain=50.0)
    bits = synth.f32_to_bf16_bits(x)
    host = synth.bf16_bits_to_f32(bits).reshape(ROWS, COLS)
    dev = torch.from_numpy(bits.view(np.int16).reshape(ROWS, COLS)).view(torch.bfloat16).cuda()
    return host, dev


@pytest.mark.parametrize("axis", [1, 0])
@pytest.mark.parametrize("name", list(MX))
def test_benchmark_step_at_full_size(tensor, name, axis):
    host, x = tensor
    cfg, ocfg = MX[name], H.to_orc(MX[name])
    want, so = orc.quant_dequant(ocfg, host, axis=axis, nthreads=16)
    want_bits = synth.f32_to_bf16_bits(want).reshape(ROWS, COLS)

    def bits_of(t):
        return t.view(torch.int16).cpu().numpy().view(np.uint16)

    y = torch.empty_like(x)
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_quant_dequant(cfg, x, y, axis=axis, qsnr_sums=sums)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(y), want_bits), "%s axis=%d quant_dequant" % (name, axis)
    H.assert_qsnr_close(sums.cpu().numpy(), so, "%s axis=%d" % (name, axis))

    planes = bdr.alloc_planes(cfg, ROWS, COLS, axis)
    bdr.bdr_pack(cfg, x, planes, axis=axis)
    torch.cuda.synchronize()
    H.assert_planes_equal(H.planes_to_host(planes), orc.pack(ocfg, host, axis=axis), "%s axis=%d pack" % (name, axis))

    back = torch.empty_like(x)
    bdr.bdr_unpack(cfg, planes, back, axis=axis)
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(back), want_bits), "%s axis=%d unpack" % (name, axis)
    assert bdr.bdr_device_status() == 0
