"""GPU parity of bdr_pack2 (both packed copies of a tensor from one read, Section V / Fig. 8): the row-direction
planes must equal the oracle's pack along axis 1 and the column-direction planes its pack along axis 0 -- i.e. the
planes of the transposed tensor -- byte for byte; the fused sums give the oracle's QSNR for both directions."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

MX = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}


def _canary_planes(cfg, rows, cols, axis):
    p = bdr.alloc_planes(cfg, rows, cols, axis)
    for t in (p.exps, p.micro, p.elems):
        t.fill_(0xA5)                      # every byte must be written by the call
    return p


def run_pack2(cfg, x_host, dtype, with_sums, ld=None):
    rows, cols = x_host.shape
    x = H.host_to_device(x_host, dtype, ld)
    pr, pc = _canary_planes(cfg, rows, cols, 1), _canary_planes(cfg, rows, cols, 0)
    sr = torch.zeros(2, dtype=torch.float64, device="cuda") if with_sums else None
    sc = torch.zeros(2, dtype=torch.float64, device="cuda") if with_sums else None
    bdr.bdr_pack2(cfg, x, pr, pc, sr, sc)
    torch.cuda.synchronize()
    return pr, pc, sr, sc


def check(cfg, x_host, dtype, with_sums, what, ld=None):
    o = H.to_orc(cfg)
    pr, pc, sr, sc = run_pack2(cfg, x_host, dtype, with_sums, ld)
    H.assert_planes_equal(H.planes_to_host(pr), orc.pack(o, x_host, axis=1), what + " rows")
    H.assert_planes_equal(H.planes_to_host(pc), orc.pack(o, x_host, axis=0), what + " columns")
    if with_sums:
        H.assert_qsnr_close(sr.cpu().numpy(), orc.quant_dequant(o, x_host, axis=1)[1], what + " rows")
        H.assert_qsnr_close(sc.cpu().numpy(), orc.quant_dequant(o, x_host, axis=0)[1], what + " columns")
    assert bdr.bdr_device_status() == 0


@pytest.mark.parametrize("with_sums", [False, True], ids=["planes", "planes+sums"])
@pytest.mark.parametrize("name", list(MX))
def test_single_read_kernel_matches_oracle_in_both_directions(name, with_sums):
    # 768 x 512: three tiles down, four across (several tiles per CTA column, a ragged number of tiles per wave)
    for kind, seed in (("laplace_outliers", 31), ("normal", 32)):
        x = H.make_input(kind, 768, 512, "bf16", seed=seed)
        check(MX[name], x, "bf16", with_sums, "%s %s" % (name, kind))


@pytest.mark.parametrize("name", list(MX))
def test_blocks_outside_the_fast_exponent_range(name):
    # tiny / huge / edge values send blocks to the out-of-line formulation in either direction
    for kind in ("tiny", "huge", "edge"):
        x = H.make_input(kind, 256, 256, "bf16", seed=33)
        check(MX[name], x, "bf16", True, "%s %s" % (name, kind))
    # a block whose exponent differs by direction: one huge element makes its row block and its column block slow
    x = H.make_input("normal", 256, 256, "bf16", seed=34)
    x[37, 101] = np.float32(2.0 ** 125)
    x[200, 5] = np.float32(2.0 ** -125)
    check(MX[name], x, "bf16", False, name + " mixed")   # planes only: 2^250 of signal energy puts QSNR near 700 dB, where
    #                                                       the fp32 partial sums of small blocks underflow (stated limit: ~400 dB)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_shapes_dtypes_and_configurations_served_by_one_pass_per_direction(dtype):
    cfgs = [bdr.MX6, bdr.Config(32, 8, 4, 2, 5), bdr.Config(16, 8, 2, 1, 4, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY)]
    for rows, cols, ld in ((256, 128, None), (100, 36, None), (512, 256, 264), (7, 1000, 1003), (16, 16, None), (1, 33, None)):
        x = H.make_input("normal", rows, cols, dtype, seed=rows + cols)
        for cfg in cfgs:
            check(cfg, x, dtype, True, "%s %s %dx%d" % (cfg, dtype, rows, cols), ld=ld)


def test_pack2_is_byte_identical_to_two_bdr_pack_calls_and_validates_on_the_host():
    cfg = bdr.MX9
    x_host = H.make_input("laplace_outliers", 512, 768, "bf16", seed=35)
    x = H.host_to_device(x_host, "bf16")
    pr, pc, _, _ = run_pack2(cfg, x_host, "bf16", False)
    for axis, got in ((1, pr), (0, pc)):
        ref = bdr.alloc_planes(cfg, 512, 768, axis)
        bdr.bdr_pack(cfg, x, ref, axis=axis)
        torch.cuda.synchronize()
        for a, b in zip((got.exps, got.micro, got.elems), (ref.exps, ref.micro, ref.elems)):
            assert torch.equal(a, b)
    small = bdr.alloc_planes(cfg, 256, 768, 0)              # column planes sized for fewer rows: lines too short
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_pack2(cfg, x, pr, small)
    assert e.value.status == -5
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_pack2(bdr.Config(16, 8, 3, 1, 4), x, pr, pc)
    assert e.value.status == -2
    empty = torch.empty((0, 768), dtype=torch.bfloat16, device="cuda")
    bdr.bdr_pack2(cfg, empty, pr, pc)                       # nothing to do
    torch.cuda.synchronize()


def test_full_size_activation_tensor():
    # the linear-layer configuration's activation tensor: 8192 x 4096 bf16, outlier channels along the columns
    rows, cols = 8192, 4096
    xh = synth.outlier_channel_matrix(rows, cols, seed=0, stream=1, frac=0.01, gain=20.0)
    bits = synth.f32_to_bf16_bits(xh)
    host = synth.bf16_bits_to_f32(bits).reshape(rows, cols)
    for name in ("MX9", "MX6"):
        cfg, o = MX[name], H.to_orc(MX[name])
        pr, pc, sr, sc = run_pack2(cfg, host, "bf16", True)
        H.assert_planes_equal(H.planes_to_host(pr), orc.pack(o, host, axis=1), name + " rows")
        H.assert_planes_equal(H.planes_to_host(pc), orc.pack(o, host, axis=0), name + " columns")
        H.assert_qsnr_close(sr.cpu().numpy(), orc.quant_dequant(o, host, axis=1, nthreads=16)[1], name + " rows")
        H.assert_qsnr_close(sc.cpu().numpy(), orc.quant_dequant(o, host, axis=0, nthreads=16)[1], name + " columns")
    assert bdr.bdr_device_status() == 0
