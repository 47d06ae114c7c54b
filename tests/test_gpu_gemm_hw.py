"""GPU parity of mx_gemm_hw, the product as the hardware dot-product pipeline of Section IV-B computes it: the result is
unique (integer block sums, truncating alignment, one fp32 rounding per pass, fp32 accumulation in a fixed order), so the
kernel must match the oracle bit for bit."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

MX = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}


def run_hw(cfg_a, a, cfg_b, b, r, f):
    M, K = a.shape
    N = b.shape[0]
    pa, pb = bdr.alloc_planes(cfg_a, M, K), bdr.alloc_planes(cfg_b, N, K)
    bdr.bdr_pack(cfg_a, torch.from_numpy(a).cuda(), pa)
    bdr.bdr_pack(cfg_b, torch.from_numpy(b).cuda(), pb)
    c = torch.full((M, N), -7.0, dtype=torch.float32, device="cuda")
    bdr.mx_gemm_hw(cfg_a, pa, cfg_b, pb, M, N, K, c, r=r, f=f)
    torch.cuda.synchronize()
    return c.cpu().numpy()


def spread(rows, K, seed, lo=-6, hi=7):
    """N(0,1) values with a random power of two per 16-block: the block exponents of a pass differ."""
    rng = np.random.default_rng(seed)
    return (synth.normal_matrix(rows, K, seed=seed) * np.repeat(2.0 ** rng.integers(lo, hi, (rows, K // 16)), 16, axis=1)).astype(np.float32)


@pytest.mark.parametrize("fa,fb", [("MX9", "MX9"), ("MX6", "MX6"), ("MX4", "MX4"), ("MX9", "MX4"), ("MX6", "MX9")])
def test_bit_exact_against_the_oracle(fa, fb):
    a, b = spread(128, 256, 41), spread(192, 256, 42)
    for r, f in ((64, 25), (64, 10), (32, 14), (16, 25), (64, 1), (128, 25), (256, 9)):
        got = run_hw(MX[fa], a, MX[fb], b, r, f)
        want = orc.gemm_hw(H.to_orc(MX[fa]), a, H.to_orc(MX[fb]), b, r=r, f=f)
        H.assert_bits_equal(got, want, "%s x %s r=%d f=%d" % (fa, fb, r, f))


def test_wide_exponent_spread_tiny_huge_and_nonfinite_blocks():
    a, b = spread(64, 128, 43, -60, 60), spread(64, 128, 44, -60, 60)
    a[3, 16:32] = 0.0                                   # an all-zero block still takes part in the exponent maximum
    a[2, :] = synth.normal(128, 48) * np.float32(2.0 ** -70)   # a result deep in the subnormal range of fp32 (row 2 x row 5)
    b[5, :] = synth.normal(128, 49) * np.float32(2.0 ** -65)
    a[7, :] *= np.float32(2.0 ** 60)                    # and beyond its largest value
    b[9, :] *= np.float32(2.0 ** 60)
    for r, f in ((64, 25), (32, 8)):
        got = run_hw(bdr.MX6, a, bdr.MX9, b, r, f)
        want = orc.gemm_hw(orc.MX6, a, orc.MX9, b, r=r, f=f)
        nan = np.isnan(want)                        # +inf from one pass and -inf from another: NaN, whose payload is not compared
        assert np.array_equal(np.isnan(got), nan)
        H.assert_bits_equal(got[~nan], want[~nan], "spread r=%d f=%d" % (r, f))
        fin = want[np.isfinite(want)]
        assert (~np.isfinite(want)).any() and ((np.abs(fin) < 1e-38) & (fin != 0)).any() if f == 25 else True
    a[11, 70] = np.inf
    b[13, 3] = np.nan
    got = run_hw(bdr.MX6, a, bdr.MX9, b, 64, 25)
    want = orc.gemm_hw(orc.MX6, a, orc.MX9, b, r=64, f=25)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.isnan(got[11]).all() and np.isnan(got[:, 13]).all()
    ok = ~np.isnan(want)
    H.assert_bits_equal(got[ok], want[ok], "beside the NaN row and column")


def test_wide_frame_reproduces_the_exact_product_and_narrow_frames_lose_accuracy_gradually():
    # ordinary operands (the GEMM configuration's distributions): with f = 25 the pipeline agrees with the fp64 product
    # of the dequantized operands to fp32 accuracy; every bit taken from the frame costs about 6 dB
    a = synth.normal_matrix(256, 512, seed=45)
    b = synth.normal_matrix(256, 512, seed=46, sigma=0.02)
    ref = orc.gemm_nt_f64(orc.quant_dequant(orc.MX6, a)[0], orc.quant_dequant(orc.MX6, b)[0], nthreads=8)
    errs = []
    for f in (25, 16, 12, 8):
        got = run_hw(bdr.MX6, a, bdr.MX6, b, 64, f)
        H.assert_bits_equal(got, orc.gemm_hw(orc.MX6, a, orc.MX6, b, r=64, f=f), "f=%d" % f)
        errs.append(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    assert errs[0] <= 1e-6 and errs == sorted(errs) and errs[-1] > 1e-3


def test_argument_checks():
    a = synth.normal_matrix(64, 64, seed=47)
    pa = bdr.alloc_planes(bdr.MX6, 64, 64)
    bdr.bdr_pack(bdr.MX6, torch.from_numpy(a).cuda(), pa)
    c = torch.empty((64, 64), dtype=torch.float32, device="cuda")
    for kw, status in ((dict(r=48), -3), (dict(r=128), -3), (dict(r=2048), -3), (dict(f=0), -5), (dict(f=26), -5)):   # K = 64: r = 128 does not divide it
        with pytest.raises(bdr.BdrError) as e:
            bdr.mx_gemm_hw(bdr.MX6, pa, bdr.MX6, pa, 64, 64, 64, c, **kw)
        assert e.value.status == status
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_hw(bdr.MX6, pa, bdr.Config(16, 8, 2, 1, 5), pa, 64, 64, 64, c)
    assert e.value.status == -3
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_hw(bdr.MX6, pa, bdr.MX6, pa, 32, 64, 64, c)
    assert e.value.status == -3
    torch.cuda.synchronize()


def test_passes_longer_than_a_step():
    # r = 512 and 1024: the blocks of a pass are aligned to a maximum taken over up to 64 blocks
    a, b = spread(64, 2048, 48, -20, 21), spread(128, 2048, 49, -20, 21)
    for r, f in ((512, 25), (1024, 16), (1024, 25)):
        got = run_hw(bdr.MX9, a, bdr.MX6, b, r, f)
        H.assert_bits_equal(got, orc.gemm_hw(orc.MX9, a, orc.MX6, b, r=r, f=f), "r=%d f=%d" % (r, f))
