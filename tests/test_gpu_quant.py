"""GPU parity: the CUDA path through the C ABI against the oracle, element by element.

Bit-exact for dequantized tensors and packed bytes; QSNR within 1e-6 dB relative.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

Cfg = bdr.Config

# every (k1, k2, d2) family the sweep uses plus the degenerate corners, a few m each
ROW_CONFIGS = [Cfg(k1, 8, k2, d2, m) for (k1, k2, d2) in
               [(1, 1, 0), (2, 1, 1), (2, 2, 2), (4, 2, 1), (8, 1, 2), (8, 8, 1), (16, 2, 1), (16, 1, 0), (16, 4, 2),
                (16, 8, 3), (16, 16, 1), (32, 2, 1), (64, 8, 2), (128, 1, 1), (256, 4, 2), (512, 2, 1), (1024, 8, 1),
                (1024, 1, 2)]
               for m in (1, 4, 8)]
MX = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}


def run_quant(cfg, x_host, dtype, axis=1, ld=None, want_y=True, inplace=False):
    x = H.host_to_device(x_host, dtype, ld)
    y = x if inplace else (torch.empty_like(x) if ld is None else H.host_to_device(np.zeros_like(x_host), dtype, ld))
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_quant_dequant(cfg, x, y if want_y else None, axis=axis, qsnr_sums=sums)
    torch.cuda.synchronize()
    return (H.device_to_host_f32(y) if want_y else None), sums.cpu().numpy()


@pytest.mark.parametrize("cfg", ROW_CONFIGS, ids=str)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rowwise_quant_dequant_matches_oracle(cfg, dtype):
    # 3 rows x 2560 columns spans several CTAs' worth of slices; 2560 is a multiple of every k1 <= 512
    for kind, rows, cols in (("normal", 3, 2560), ("edge", 5, 2048), ("laplace_outliers", 2, 1024)):
        x = H.make_input(kind, rows, cols, dtype, seed=11)
        y, sums = run_quant(cfg, x, dtype)
        want, so = orc.quant_dequant(H.to_orc(cfg), x)
        H.assert_bits_equal(y, want, "%s %s %s" % (cfg, dtype, kind))
        H.assert_qsnr_close(sums, so, "%s %s %s" % (cfg, dtype, kind))


@pytest.mark.parametrize("cfg", [bdr.MX6, bdr.MX9, Cfg(64, 8, 4, 2, 3), Cfg(1024, 8, 2, 1, 5), Cfg(8, 8, 2, 1, 4)], ids=str)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rowwise_ragged_shapes_and_pitches(cfg, dtype):
    for rows, cols, ld in ((1, 1, None), (7, 100, None), (4, 1000, 1003), (3, 16, 24), (2, 1037, 1040), (1, 5000, None)):
        x = H.make_input("normal", rows, cols, dtype, seed=rows * 1000 + cols)
        y, sums = run_quant(cfg, x, dtype, ld=ld)
        want, so = orc.quant_dequant(H.to_orc(cfg), x)
        H.assert_bits_equal(y, want, "%s %s %dx%d ld=%s" % (cfg, dtype, rows, cols, ld))
        H.assert_qsnr_close(sums, so)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_extreme_exponents_signed_zeros_and_ties_away(dtype):
    for kind in ("tiny", "huge", "edge"):
        x = H.make_input(kind, 4, 1024, dtype, seed=5)
        for cfg in (bdr.MX4, bdr.MX9, Cfg(16, 8, 2, 3, 8), Cfg(32, 8, 1, 2, 6, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY),
                    Cfg(16, 8, 2, 1, 4, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY)):
            y, sums = run_quant(cfg, x, dtype)
            want, so = orc.quant_dequant(H.to_orc(cfg), x)
            H.assert_bits_equal(y, want, "%s %s %s" % (cfg, dtype, kind))
            H.assert_qsnr_close(sums, so, "%s %s %s" % (cfg, dtype, kind))


def test_nonfinite_inputs_poison_only_their_block():
    x = H.make_input("normal", 2, 512, "f32", seed=9)
    x[0, 37] = np.inf
    x[1, 300] = np.nan
    for cfg in (bdr.MX6, Cfg(64, 8, 2, 1, 4)):
        y, sums = run_quant(cfg, x, "f32")
        want, _ = orc.quant_dequant(H.to_orc(cfg), x)
        assert np.array_equal(np.isnan(y), np.isnan(want))
        ok = ~np.isnan(want)
        H.assert_bits_equal(y[ok], want[ok])
        assert np.isnan(sums).any()


def test_in_place_and_sums_only():
    x = H.make_input("normal", 8, 2048, "f32", seed=3)
    want, so = orc.quant_dequant(H.to_orc(bdr.MX6), x)
    y, sums = run_quant(bdr.MX6, x, "f32", inplace=True)
    H.assert_bits_equal(y, want)
    _, sums2 = run_quant(bdr.MX6, x, "f32", want_y=False)
    H.assert_qsnr_close(sums2, so)
    assert np.array_equal(sums, sums2) or np.allclose(sums, sums2, rtol=1e-12)


def test_empty_tensors_are_no_ops():
    for rows, cols in ((0, 64), (4, 0)):
        x = torch.empty((rows, cols), device="cuda")
        bdr.bdr_quant_dequant(bdr.MX6, x, torch.empty_like(x))
    torch.cuda.synchronize()


# ---- the first BASELINE configuration, complete -------------------------------------------------------
def test_config1_mx6_vector_of_65536():
    x = synth.normal(65536, seed=0).reshape(1, -1)
    xd = torch.from_numpy(x).cuda()
    planes = bdr.alloc_planes(bdr.MX6, 1, 65536)
    assert [p.shape[1] for p in (planes.exps, planes.micro, planes.elems)] == [4096, 4096, 40960]
    y = torch.empty_like(xd)
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_pack(bdr.MX6, xd, planes, y_dq=y, qsnr_sums=sums)
    torch.cuda.synchronize()
    want, so = orc.quant_dequant(orc.MX6, x)
    H.assert_bits_equal(y.cpu().numpy(), want)
    H.assert_planes_equal(H.planes_to_host(planes), orc.pack(orc.MX6, x))
    H.assert_qsnr_close(sums.cpu().numpy(), so)
    assert abs(orc.qsnr_db(*sums.cpu().numpy()) - 28.3) < 0.1


# ---- pack / unpack -----------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", list(MX))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("axis", [1, 0])
def test_pack_and_unpack_mx_formats(name, dtype, axis):
    cfg = MX[name]
    # fast-path shapes (multiples of 512) and shapes that force the general kernels
    for kind, rows, cols in (("laplace_outliers", 512, 1024), ("edge", 1024, 512), ("normal", 40, 100), ("normal", 33, 512),
                             ("edge", 64, 2048)):
        x = H.make_input(kind, rows, cols, dtype, seed=21)
        xd = H.host_to_device(x, dtype)
        planes = bdr.alloc_planes(cfg, rows, cols, axis)
        y = torch.empty_like(xd)
        sums = torch.zeros(2, dtype=torch.float64, device="cuda")
        bdr.bdr_pack(cfg, xd, planes, axis=axis, y_dq=y, qsnr_sums=sums)
        back = torch.full_like(xd, 7.0)
        bdr.bdr_unpack(cfg, planes, back, axis=axis)
        torch.cuda.synchronize()
        what = "%s %s axis=%d %s %dx%d" % (name, dtype, axis, kind, rows, cols)
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=axis)
        H.assert_bits_equal(H.device_to_host_f32(y), want, what + " y_dq")
        H.assert_planes_equal(H.planes_to_host(planes), orc.pack(H.to_orc(cfg), x, axis=axis), what)
        H.assert_bits_equal(H.device_to_host_f32(back), want, what + " unpack")
        H.assert_qsnr_close(sums.cpu().numpy(), so, what)


@pytest.mark.parametrize("cfg", [Cfg(8, 8, 4, 2, 3), Cfg(32, 8, 1, 3, 6), Cfg(16, 8, 16, 0, 7), Cfg(16, 8, 2, 2, 8),
                                 Cfg(16, 8, 2, 0, 3), Cfg(1024, 8, 8, 1, 1), Cfg(1, 8, 1, 0, 8)], ids=str)
def test_pack_and_unpack_general_configs(cfg):
    for axis in (1, 0):
        for rows, cols in ((6, 200), (512, 512)):
            x = H.make_input("edge", rows, cols, "f32", seed=31)
            xd = H.host_to_device(x, "f32")
            planes = bdr.alloc_planes(cfg, rows, cols, axis)
            for t in (planes.exps, planes.micro, planes.elems):
                t.fill_(0xAB)                                   # every byte up to the pitch must be rewritten
            bdr.bdr_pack(cfg, xd, planes, axis=axis)
            back = torch.empty_like(xd)
            bdr.bdr_unpack(cfg, planes, back, axis=axis)
            torch.cuda.synchronize()
            want, _ = orc.quant_dequant(H.to_orc(cfg), x, axis=axis)
            H.assert_planes_equal(H.planes_to_host(planes), orc.pack(H.to_orc(cfg), x, axis=axis), str(cfg))
            H.assert_bits_equal(back.cpu().numpy(), want, str(cfg))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_columnwise_quant_dequant(dtype):
    for cfg in (bdr.MX6, bdr.MX9, Cfg(32, 8, 4, 2, 3), Cfg(8, 8, 1, 1, 5)):
        for rows, cols, ld in ((512, 256, None), (100, 72, None), (64, 200, 208)):
            x = H.make_input("laplace_outliers", rows, cols, dtype, seed=41)
            y, sums = run_quant(cfg, x, dtype, axis=0, ld=ld)
            want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=0)
            H.assert_bits_equal(y, want, "%s %s %dx%d" % (cfg, dtype, rows, cols))
            H.assert_qsnr_close(sums, so)


@pytest.mark.parametrize("cfg", ROW_CONFIGS + [Cfg(16, 8, 2, 1, 4, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY),
                                             Cfg(64, 8, 4, 2, 6, bdr.SCALE_POW2, bdr.ROUND_NEAREST_AWAY)], ids=str)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_columnwise_quant_dequant_of_every_configuration(cfg, dtype):
    # blocks run down the columns; every (k1, k2, d2) family of the sweep: block sizes from 1 to 1024 rows, several blocks
    # per column, a ragged last block (rows not a multiple of k1), ragged column groups, a pitch, in place, sums only
    for kind, rows, cols, ld in (("laplace_outliers", 2048 + 40, 96, None), ("edge", 1100, 70, 72), ("normal", 48, 130, None)):
        x = H.make_input(kind, rows, cols, dtype, seed=43)
        y, sums = run_quant(cfg, x, dtype, axis=0, ld=ld)
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=0)
        H.assert_bits_equal(y, want, "%s %s %s %dx%d" % (cfg, dtype, kind, rows, cols))
        H.assert_qsnr_close(sums, so, "%s %s %s" % (cfg, dtype, kind))
    x = H.make_input("normal", 300, 64, dtype, seed=44)
    want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=0)
    y, _ = run_quant(cfg, x, dtype, axis=0, inplace=True)
    H.assert_bits_equal(y, want, "%s %s in place" % (cfg, dtype))
    _, sums = run_quant(cfg, x, dtype, axis=0, want_y=False)
    H.assert_qsnr_close(sums, so, "%s %s sums only" % (cfg, dtype))
    for kind in ("tiny", "huge"):
        x = H.make_input(kind, 260, 34, dtype, seed=45)
        y, sums = run_quant(cfg, x, dtype, axis=0)
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=0)
        H.assert_bits_equal(y, want, "%s %s %s" % (cfg, dtype, kind))
        H.assert_qsnr_close(sums, so, "%s %s %s" % (cfg, dtype, kind))


# ---- host-side error paths: nothing is launched -----------------------------------------------------------
def test_argument_errors_are_reported_not_launched():
    x = torch.zeros((4, 64), device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_quant_dequant(Cfg(16, 8, 3, 1, 4), x, x)                 # k2 does not divide k1
    assert e.value.status == -2
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_quant_dequant(Cfg(16, 7, 2, 1, 4), x, x)                 # d1 must be 8
    assert e.value.status == -2
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_quant_dequant(Cfg(24, 8, 2, 1, 4), x, x)                 # legal BDR, no kernel
    assert e.value.status == -3
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_quant_dequant(bdr.MX6, x, None)                          # nothing to produce
    assert e.value.status == -1
    planes = bdr.alloc_planes(bdr.MX6, 4, 64)
    small = bdr.Planes(planes.exps, planes.micro, torch.empty((4, 16), dtype=torch.uint8, device="cuda"))
    with pytest.raises(bdr.BdrError) as e:
        bdr.bdr_pack(bdr.MX6, x, small)
    assert e.value.status == -5
    torch.cuda.synchronize()


@pytest.mark.gpu
def test_bounded_waits_never_ran_out():
    # bulk-copy kernels (1024-element runs of bf16) report a wait that ran out through a sticky status word
    cfg = bdr.MX6
    x = H.make_input("normal", 64, 4096, "bf16", seed=5)
    xd = H.host_to_device(x, "bf16")
    y = torch.empty_like(xd)
    bdr.bdr_quant_dequant(cfg, xd, y)
    planes = bdr.alloc_planes(cfg, 64, 4096, 1)
    bdr.bdr_pack(cfg, xd, planes, y_dq=y)
    torch.cuda.synchronize()
    assert bdr.bdr_device_status() == 0


# ---- bf16 fast paths (packed bf16x2 arithmetic): every output combination, exponent-range boundaries ----
def _boundary_input(rows, cols, seed):
    """bf16-exact values whose 16-element blocks (in both directions: the tile is constant over 16 x 16
    patches) have their largest exponent field at and around the limits of the packed-arithmetic range."""
    rng = np.random.default_rng(seed)
    fields = np.array([1, 8, 14, 15, 16, 17, 18, 100, 127, 200, 238, 239, 240, 241, 242, 248, 249, 250, 251, 252, 254])
    pr, pc = rows // 16, cols // 16
    f = fields[rng.integers(0, len(fields), (pr, pc))]
    scale = np.ldexp(1.0, (f - 127).astype(np.int64)).astype(np.float64)       # 2^(F-127) per patch
    scale = np.kron(scale, np.ones((16, 16)))
    mant = 1.0 + rng.integers(0, 128, (rows, cols)) / 128.0                         # 8-bit significands in [1, 2)
    down = np.ldexp(1.0, -rng.integers(0, 12, (rows, cols)).astype(np.int64))        # most elements below the block maximum
    sign = np.where(rng.random((rows, cols)) < 0.5, -1.0, 1.0)
    x = sign * mant * down * scale
    x[::16, ::16] = np.abs(mant[::16, ::16] * scale[::16, ::16])                       # one element per patch carries the exponent
    x[1::16, 3::16] = 0.0
    x[2::16, 5::16] = -0.0
    x = x.astype(np.float32)
    x = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x)).reshape(rows, cols)
    return np.where(np.isfinite(x), x, np.float32(1.0)).astype(np.float32)


@pytest.mark.parametrize("axis", [1, 0])
@pytest.mark.parametrize("name", list(MX))
def test_bf16_fast_paths_every_output_combination(name, axis):
    cfg = MX[name]
    rows, cols = 256, 2048
    for kind in ("laplace_outliers", "boundary", "edge"):
        x = _boundary_input(rows, cols, seed=77) if kind == "boundary" else H.make_input(kind, rows, cols, "bf16", seed=33)
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=axis)
        want_planes = orc.pack(H.to_orc(cfg), x, axis=axis)
        xd = H.host_to_device(x, "bf16")
        for with_y in (False, True):
            for with_sums in (False, True):
                what = "%s axis=%d %s y=%s sums=%s" % (name, axis, kind, with_y, with_sums)
                y = torch.full_like(xd, 5.0) if with_y else None
                sums = torch.zeros(2, dtype=torch.float64, device="cuda") if with_sums else None
                planes = bdr.alloc_planes(cfg, rows, cols, axis)
                for p in (planes.exps, planes.micro, planes.elems):
                    p.fill_(0xA5)
                bdr.bdr_pack(cfg, xd, planes, axis=axis, y_dq=y, qsnr_sums=sums)
                torch.cuda.synchronize()
                H.assert_planes_equal(H.planes_to_host(planes), want_planes, what)
                if with_y:
                    H.assert_bits_equal(H.device_to_host_f32(y), want, what + " y_dq")
                if with_sums:
                    H.assert_qsnr_close(sums.cpu().numpy(), so, what)
                if with_y or with_sums:
                    y2 = torch.full_like(xd, 5.0) if with_y else None
                    s2 = torch.zeros(2, dtype=torch.float64, device="cuda") if with_sums else None
                    bdr.bdr_quant_dequant(cfg, xd, y2, axis=axis, qsnr_sums=s2)
                    torch.cuda.synchronize()
                    if with_y:
                        H.assert_bits_equal(H.device_to_host_f32(y2), want, what + " quant_dequant")
                    if with_sums:
                        H.assert_qsnr_close(s2.cpu().numpy(), so, what + " quant_dequant")
        back = torch.full_like(xd, 7.0)
        bdr.bdr_unpack(cfg, planes, back, axis=axis)
        torch.cuda.synchronize()
        H.assert_bits_equal(H.device_to_host_f32(back), want, "%s axis=%d %s unpack" % (name, axis, kind))
    assert bdr.bdr_device_status() == 0


@pytest.mark.parametrize("m", [1, 3, 5, 6])
def test_bf16_quant_dequant_other_mantissa_widths(m):
    # the packed-arithmetic quantize-dequantize kernels take any m <= 7 of the k1 = 16, k2 = 2, d2 = 1 family
    cfg = Cfg(16, 8, 2, 1, m)
    x = _boundary_input(256, 2048, seed=m)
    for axis in (1, 0):
        y, sums = run_quant(cfg, x, "bf16", axis=axis)
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=axis)
        H.assert_bits_equal(y, want, "%s axis=%d" % (cfg, axis))
        H.assert_qsnr_close(sums, so, "%s axis=%d" % (cfg, axis))


@pytest.mark.parametrize("k1", [16, 32, 64, 256, 1024])
@pytest.mark.parametrize("k2,d2", [(2, 1), (1, 0), (8, 0)])
def test_bf16_rowwise_wider_blocks_and_no_shifts(k1, k2, d2):
    # the packed-arithmetic row kernel also takes blocks of up to 1024 elements (the exponent is a maximum over
    # the lanes that share the block) and formats without microexponents (BFP / MSFP)
    for m in (1, 4, 7):
        cfg = Cfg(k1, 8, k2, d2, m)
        cases = [("boundary", _boundary_input(64, 2048, seed=k1 + m), None),
                 ("laplace_outliers", H.make_input("laplace_outliers", 6, 4096, "bf16", seed=k1), None),
                 ("normal pitch", H.make_input("normal", 3, 2048, "bf16", seed=m), 2080),
                 ("edge", H.make_input("edge", 4, 1024, "bf16", seed=3), None)]
        for what, x, ld in cases:
            y, sums = run_quant(cfg, x, "bf16", ld=ld)
            want, so = orc.quant_dequant(H.to_orc(cfg), x)
            H.assert_bits_equal(y, want, "%s %s" % (cfg, what))
            H.assert_qsnr_close(sums, so, "%s %s" % (cfg, what))
            _, sums_only = run_quant(cfg, x, "bf16", ld=ld, want_y=False)
            H.assert_qsnr_close(sums_only, so, "%s %s sums only" % (cfg, what))
    assert bdr.bdr_device_status() == 0


def test_bf16_fast_paths_with_a_row_pitch():
    # rows of 2048 elements that are 2112 elements apart: the run index splits into (row, position)
    rows, cols, ld = 5, 2048, 2112
    x = H.make_input("laplace_outliers", rows, cols, "bf16", seed=12)
    for cfg in (bdr.MX4, bdr.MX9):
        y, sums = run_quant(cfg, x, "bf16", ld=ld)
        want, so = orc.quant_dequant(H.to_orc(cfg), x)
        H.assert_bits_equal(y, want, "%s pitch" % (cfg,))
        H.assert_qsnr_close(sums, so)
        xd = H.host_to_device(x, "bf16", ld)
        planes = bdr.alloc_planes(cfg, rows, cols, 1)
        bdr.bdr_pack(cfg, xd, planes)
        back = H.host_to_device(np.zeros_like(x), "bf16", ld)
        bdr.bdr_unpack(cfg, planes, back)
        torch.cuda.synchronize()
        H.assert_planes_equal(H.planes_to_host(planes), orc.pack(H.to_orc(cfg), x), "%s pitch" % (cfg,))
        H.assert_bits_equal(H.device_to_host_f32(back), want, "%s pitch unpack" % (cfg,))


def test_bf16_column_fast_paths_with_a_row_pitch():
    # the tile kernels of the column direction address the tensor through tensor maps built with the caller's pitch
    rows, cols, ld = 512, 384, 448
    x = H.make_input("laplace_outliers", rows, cols, "bf16", seed=13)
    for cfg in (bdr.MX4, bdr.MX6, bdr.MX9):
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=0)
        y, sums = run_quant(cfg, x, "bf16", axis=0, ld=ld)
        H.assert_bits_equal(y, want, "%s pitch" % (cfg,))
        H.assert_qsnr_close(sums, so)
        xd = H.host_to_device(x, "bf16", ld)
        planes = bdr.alloc_planes(cfg, rows, cols, 0)
        bdr.bdr_pack(cfg, xd, planes, axis=0)
        back = H.host_to_device(np.full_like(x, 3.0), "bf16", ld)
        bdr.bdr_unpack(cfg, planes, back, axis=0)
        torch.cuda.synchronize()
        H.assert_planes_equal(H.planes_to_host(planes), orc.pack(H.to_orc(cfg), x, axis=0), "%s pitch" % (cfg,))
        H.assert_bits_equal(H.device_to_host_f32(back), want, "%s pitch unpack" % (cfg,))
    assert bdr.bdr_device_status() == 0


@pytest.mark.parametrize("axis", [1, 0])
def test_bf16_fast_paths_in_place(axis):
    # y may alias x: the run (row direction) or the box (column direction) is loaded whole before it is written back
    x = H.make_input("laplace_outliers", 512, 2048, "bf16", seed=8)
    for cfg in (bdr.MX4, bdr.MX9):
        want, so = orc.quant_dequant(H.to_orc(cfg), x, axis=axis)
        xd = H.host_to_device(x, "bf16")
        sums = torch.zeros(2, dtype=torch.float64, device="cuda")
        bdr.bdr_quant_dequant(cfg, xd, xd, axis=axis, qsnr_sums=sums)
        torch.cuda.synchronize()
        H.assert_bits_equal(H.device_to_host_f32(xd), want, "%s axis=%d in place" % (cfg, axis))
        H.assert_qsnr_close(sums.cpu().numpy(), so)
