"""GPU parity of mx_gemm against the fp64 oracle product of the dequantized operands.

Target: relative Frobenius error <= 1e-3.  The decoded operands are exact in bf16 and their products
exact in fp32, so only the fp32 summation order separates the two; the observed error is ~1e-6.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

FMT = {"MX4": bdr.MX4, "MX6": bdr.MX6, "MX9": bdr.MX9}
REL_FROB_TOL = 1e-3


def gpu_gemm(cfg_a, a_host, cfg_b, b_host):
    M, K = a_host.shape
    N = b_host.shape[0]
    a, b = torch.from_numpy(a_host).cuda(), torch.from_numpy(b_host).cuda()
    pa, pb = bdr.alloc_planes(cfg_a, M, K), bdr.alloc_planes(cfg_b, N, K)
    bdr.bdr_pack(cfg_a, a, pa)
    bdr.bdr_pack(cfg_b, b, pb)
    c = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    bdr.mx_gemm(cfg_a, pa, cfg_b, pb, M, N, K, c)
    torch.cuda.synchronize()
    assert bdr.mx_gemm_status() == 0
    return c.cpu().numpy()


def oracle_gemm(cfg_a, a_host, cfg_b, b_host):
    aq, _ = orc.quant_dequant(H.to_orc(cfg_a), a_host)
    bq, _ = orc.quant_dequant(H.to_orc(cfg_b), b_host)
    return orc.gemm_nt_f64(aq, bq, nthreads=8)


def rel_frob(c, ref):
    return float(np.linalg.norm(c.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


def test_exact_case_small_integers():
    # operands that are representable in MX9 and whose dot products are small integers: any
    # summation order gives the same fp32 result, so the match must be bit for bit
    rng = np.random.default_rng(0)
    a = rng.integers(-8, 9, (128, 64)).astype(np.float32)
    b = rng.integers(-8, 9, (256, 64)).astype(np.float32)
    a[:, ::16] = 8.0      # pin every block's shared exponent so all of -8..8 stay representable
    b[:, ::16] = -8.0
    c = gpu_gemm(bdr.MX9, a, bdr.MX9, b)
    ref = oracle_gemm(bdr.MX9, a, bdr.MX9, b)
    assert np.array_equal(ref, (a.astype(np.int64) @ b.astype(np.int64).T).astype(np.float64))
    assert np.array_equal(c.astype(np.float64), ref)


@pytest.mark.parametrize("fa,fb", [("MX6", "MX6"), ("MX9", "MX4"), ("MX4", "MX9"), ("MX9", "MX9"), ("MX4", "MX4")])
def test_random_operands_match_the_oracle(fa, fb):
    M, N, K = 256, 512, 320                              # several tiles in M and N, 5 K steps
    a = synth.normal_matrix(M, K, seed=1, stream=1)
    b = synth.normal_matrix(N, K, seed=1, stream=2, sigma=0.02)
    c = gpu_gemm(FMT[fa], a, FMT[fb], b)
    ref = oracle_gemm(FMT[fa], a, FMT[fb], b)
    err = rel_frob(c, ref)
    assert err <= REL_FROB_TOL, err
    assert err <= 1e-5, err                              # what exact decoding should deliver


@pytest.mark.parametrize("fa,fb", [("MX6", "MX6"), ("MX9", "MX4"), ("MX4", "MX6"), ("MX9", "MX9")])
def test_two_cta_kernel_shapes(fa, fb):
    # M a multiple of 256 and K a multiple of 256 select the 2-CTA (cta_group::2) kernel
    M, N, K = 512, 768, 1024
    a = synth.normal_matrix(M, K, seed=6, stream=1)
    b = synth.outlier_channel_matrix(N, K, seed=6, stream=2, gain=20.0, dist="normal", sigma=0.02)
    c = gpu_gemm(FMT[fa], a, FMT[fb], b)
    ref = oracle_gemm(FMT[fa], a, FMT[fb], b)
    assert rel_frob(c, ref) <= 1e-5


def test_outlier_channels_and_extreme_scales():
    M, N, K = 128, 256, 512
    a = synth.outlier_channel_matrix(M, K, seed=2, gain=50.0)
    for scale in (1.0, 1e-30, 1e25):
        b = synth.normal_matrix(N, K, seed=3, sigma=0.02) * np.float32(scale)
        c = gpu_gemm(bdr.MX6, a, bdr.MX9, b)
        ref = oracle_gemm(bdr.MX6, a, bdr.MX9, b)
        assert rel_frob(c, ref) <= 1e-5, scale
    z = np.zeros((N, K), dtype=np.float32)
    assert not gpu_gemm(bdr.MX6, a, bdr.MX6, z).any()


def test_config4_shape_on_sampled_entries():
    M = N = K = 4096
    a = synth.normal_matrix(M, K, seed=0, stream=10)
    b = synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)
    c = gpu_gemm(bdr.MX6, a, bdr.MX6, b)
    aq, _ = orc.quant_dequant(orc.MX6, a, nthreads=8)
    bq, _ = orc.quant_dequant(orc.MX6, b, nthreads=8)
    rng = np.random.default_rng(4)
    ri, ci = rng.integers(0, M, 4096), rng.integers(0, N, 4096)
    ref = orc.gemm_nt_f64_sampled(aq, bq, ri, ci)
    got = c[ri, ci].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert np.isfinite(c).all()
    # a full row and a full column of tiles as well
    assert rel_frob(c[:128], orc.gemm_nt_f64(aq[:128], bq, nthreads=8)) <= 1e-5


def test_gemm_argument_errors():
    pa, pb = bdr.alloc_planes(bdr.MX6, 128, 64), bdr.alloc_planes(bdr.MX6, 256, 64)
    c = torch.empty((128, 256), device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm(bdr.Config(16, 8, 2, 1, 3), pa, bdr.MX6, pb, 128, 256, 64, c)     # m = 3 has no gemm kernel
    assert e.value.status == -3
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm(bdr.MX6, pa, bdr.MX6, pb, 100, 256, 64, c)
    assert e.value.status == -3
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm(bdr.MX6, pa, bdr.MX6, pb, 128, 256, 128, c)                       # planes too narrow for K
    assert e.value.status == -5
    torch.cuda.synchronize()


# ---- two-phase entry point (decode once into a workspace, then a TMA-fed tensor-core GEMM) ----------------
def gpu_gemm_ws(cfg_a, a_host, cfg_b, b_host):
    M, K = a_host.shape
    N = b_host.shape[0]
    a, b = torch.from_numpy(a_host).cuda(), torch.from_numpy(b_host).cuda()
    pa, pb = bdr.alloc_planes(cfg_a, M, K), bdr.alloc_planes(cfg_b, N, K)
    bdr.bdr_pack(cfg_a, a, pa)
    bdr.bdr_pack(cfg_b, b, pb)
    ws = torch.empty(bdr.mx_gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    c = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    bdr.mx_gemm_ws(cfg_a, pa, cfg_b, pb, M, N, K, c, ws)
    torch.cuda.synchronize()
    assert bdr.mx_gemm_status() == 0 and bdr.bdr_device_status() == 0
    return c.cpu().numpy()


def test_ws_exact_case_small_integers():
    rng = np.random.default_rng(1)
    a = rng.integers(-8, 9, (256, 128)).astype(np.float32)
    b = rng.integers(-8, 9, (256, 128)).astype(np.float32)
    a[:, ::16] = 8.0
    b[:, ::16] = -8.0
    c = gpu_gemm_ws(bdr.MX9, a, bdr.MX9, b)
    assert np.array_equal(c.astype(np.int64), a.astype(np.int64) @ b.astype(np.int64).T)


@pytest.mark.parametrize("fa,fb", [("MX6", "MX6"), ("MX9", "MX4"), ("MX4", "MX9")])
def test_ws_random_operands_match_the_oracle(fa, fb):
    M, N, K = 512, 768, 1088                             # six tiles, 17 K steps (ring wraps several times)
    a = synth.normal_matrix(M, K, seed=7, stream=1)
    b = synth.outlier_channel_matrix(N, K, seed=7, stream=2, gain=20.0, dist="normal", sigma=0.02)
    c = gpu_gemm_ws(FMT[fa], a, FMT[fb], b)
    ref = oracle_gemm(FMT[fa], a, FMT[fb], b)
    assert rel_frob(c, ref) <= 1e-5


def test_ws_more_tiles_than_clusters_and_extreme_scales():
    # 24 x 16 = 384 tiles: every cluster walks over several tiles and both accumulator buffers are reused
    M, N, K = 6144, 4096, 64
    a = synth.normal_matrix(M, K, seed=8, stream=1)
    b = synth.normal_matrix(N, K, seed=8, stream=2, sigma=0.02)
    c = gpu_gemm_ws(bdr.MX6, a, bdr.MX6, b)
    ref = oracle_gemm(bdr.MX6, a, bdr.MX6, b)
    assert rel_frob(c, ref) <= 1e-5
    for scale in (1e-30, 1e25):
        b2 = synth.normal_matrix(256, 128, seed=3, sigma=0.02) * np.float32(scale)
        a2 = synth.outlier_channel_matrix(256, 128, seed=2, gain=50.0)
        c2 = gpu_gemm_ws(bdr.MX6, a2, bdr.MX9, b2)
        assert rel_frob(c2, oracle_gemm(bdr.MX6, a2, bdr.MX9, b2)) <= 1e-5, scale


def test_ws_config4_shape_on_sampled_entries():
    M = N = K = 4096
    a = synth.normal_matrix(M, K, seed=0, stream=10)
    b = synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)
    c = gpu_gemm_ws(bdr.MX6, a, bdr.MX6, b)
    aq, _ = orc.quant_dequant(orc.MX6, a, nthreads=8)
    bq, _ = orc.quant_dequant(orc.MX6, b, nthreads=8)
    rng = np.random.default_rng(5)
    ri, ci = rng.integers(0, M, 4096), rng.integers(0, N, 4096)
    ref = orc.gemm_nt_f64_sampled(aq, bq, ri, ci)
    got = c[ri, ci].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert np.isfinite(c).all()
    assert rel_frob(c[-256:], orc.gemm_nt_f64(aq[-256:], bq, nthreads=8)) <= 1e-5


def test_ws_split_tiles_with_a_padded_output_pitch_and_whole_rounds():
    # two tiles on 74 clusters: both are computed as two halves of K that add into tiles cleared beforehand, with the
    # pitch of the view C is; the columns beside the view stay untouched.  Called twice: the clearing is per call.
    M, N, K = 512, 256, 512
    a = synth.normal_matrix(M, K, seed=23, stream=1)
    b = synth.normal_matrix(N, K, seed=23, stream=2, sigma=0.02)
    ta, tb = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    pa, pb = bdr.alloc_planes(bdr.MX9, M, K), bdr.alloc_planes(bdr.MX9, N, K)
    bdr.bdr_pack(bdr.MX9, ta, pa)
    bdr.bdr_pack(bdr.MX9, tb, pb)
    ws = torch.empty(bdr.mx_gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    wide = torch.full((M, N + 64), 7.0, dtype=torch.float32, device="cuda")
    ref = oracle_gemm(bdr.MX9, a, bdr.MX9, b)
    for _ in range(2):
        bdr.mx_gemm_ws(bdr.MX9, pa, bdr.MX9, pb, M, N, K, wide[:, :N], ws)
        torch.cuda.synchronize()
        assert bdr.mx_gemm_status() == 0
        got = wide.cpu().numpy()
        assert (got[:, N:] == 7.0).all()
        assert rel_frob(got[:, :N], ref) <= 1e-5
    # an odd number of K steps cannot be halved: whole tiles, plain stores
    K2 = 192
    a2, b2 = synth.normal_matrix(M, K2, seed=24, stream=1), synth.normal_matrix(N, K2, seed=24, stream=2, sigma=0.02)
    assert rel_frob(gpu_gemm_ws(bdr.MX6, a2, bdr.MX6, b2), oracle_gemm(bdr.MX6, a2, bdr.MX6, b2)) <= 1e-5


def test_ws_tiles_walked_in_bands():
    # operands above 64 MiB: the clusters walk the 9 x 10 tiles in bands of eight tile rows (the last band has one row)
    # and most clusters take a second tile; every tile must land where it belongs
    M, N, K = 2304, 2560, 8192
    a = synth.normal_matrix(M, K, seed=21, stream=1)
    b = synth.normal_matrix(N, K, seed=21, stream=2, sigma=0.02)
    c = gpu_gemm_ws(bdr.MX9, a, bdr.MX9, b)
    assert np.isfinite(c).all()
    aq, _ = orc.quant_dequant(orc.MX9, a, nthreads=8)
    bq, _ = orc.quant_dequant(orc.MX9, b, nthreads=8)
    rng = np.random.default_rng(6)
    ri, ci = rng.integers(0, M, 8192), rng.integers(0, N, 8192)
    ref = orc.gemm_nt_f64_sampled(aq, bq, ri, ci)
    got = c[ri, ci].astype(np.float64)
    assert np.max(np.abs(got - ref)) <= 1e-4 * np.max(np.abs(ref))      # a misplaced tile is off by the size of an entry
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert rel_frob(c[-256:], orc.gemm_nt_f64(aq[-256:], bq, nthreads=8)) <= 1e-5   # the one-row band


def test_ws_argument_errors():
    pa, pb = bdr.alloc_planes(bdr.MX6, 256, 64), bdr.alloc_planes(bdr.MX6, 256, 64)
    c = torch.empty((256, 256), device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_ws(bdr.MX6, pa, bdr.MX6, pb, 256, 256, 64, c, small)               # workspace too small
    assert e.value.status == -6
    ws = torch.empty(bdr.mx_gemm_workspace_bytes(256, 256, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_ws(bdr.MX6, pa, bdr.MX6, pb, 128, 256, 64, c, ws)                  # M must be a multiple of 256
    assert e.value.status == -3
    torch.cuda.synchronize()


def test_padded_plane_pitches_unpack_and_ws_gemm():
    # planes whose line pitch exceeds the natural bytes: the general pack kernel fills them, the bf16 row unpack
    # reads them run by run, and the two-phase GEMM decodes from them
    M, N, K = 256, 256, 2048
    a = synth.normal_matrix(M, K, seed=11, stream=1)
    b = synth.normal_matrix(N, K, seed=11, stream=2, sigma=0.02)

    def padded(cfg, rows):
        p = bdr.alloc_planes(cfg, rows, K)
        wide = lambda t: torch.zeros((rows, t.shape[1] + 32), dtype=torch.uint8, device="cuda")[:, :t.shape[1]]
        return bdr.Planes(wide(p.exps), wide(p.micro), wide(p.elems))

    pa, pb = padded(bdr.MX6, M), padded(bdr.MX9, N)
    ad, bd = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    bdr.bdr_pack(bdr.MX6, ad, pa)
    bdr.bdr_pack(bdr.MX9, bd, pb)
    back = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    bdr.bdr_unpack(bdr.MX6, pa, back)
    aq, _ = orc.quant_dequant(orc.MX6, a)
    H.assert_bits_equal(H.device_to_host_f32(back), aq, "unpack from padded planes")
    ws = torch.empty(bdr.mx_gemm_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    bdr.mx_gemm_ws(bdr.MX6, pa, bdr.MX9, pb, M, N, K, c, ws)
    torch.cuda.synchronize()
    assert rel_frob(c.cpu().numpy(), oracle_gemm(bdr.MX6, a, bdr.MX9, b)) <= 1e-5
    assert bdr.mx_gemm_status() == 0 and bdr.bdr_device_status() == 0


def test_mx_gemm_uses_a_lent_workspace_and_gives_it_back():
    # the same call, with and without scratch memory lent to the library: same product (up to summation order);
    # the scratch is touched only while it is lent
    M, N, K = 512, 256, 768
    a = synth.normal_matrix(M, K, seed=13, stream=1)
    b = synth.normal_matrix(N, K, seed=13, stream=2, sigma=0.02)
    nbytes = max(bdr.mx_gemm_f8_workspace_bytes(M, N, K), bdr.mx_gemm_workspace_bytes(M, N, K))
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    try:
        for fa, fb in ((bdr.MX6, bdr.MX4), (bdr.MX9, bdr.MX6)):
            ref = oracle_gemm(fa, a, fb, b)
            ws.fill_(0xAB)
            bdr.bdr_set_workspace(ws)
            c = gpu_gemm(fa, a, fb, b)
            assert rel_frob(c, ref) <= 1e-5
            assert int((ws != 0xAB).sum().item()) > M * K // 2           # the two-phase kernels ran
            ws.fill_(0xAB)
            bdr.bdr_set_workspace(None)
            c = gpu_gemm(fa, a, fb, b)
            assert rel_frob(c, ref) <= 1e-5
            assert int((ws != 0xAB).sum().item()) == 0                    # back to the kernel without scratch
        bdr.bdr_set_workspace(ws[:1024])                                 # too small: the call still works
        assert rel_frob(gpu_gemm(bdr.MX6, a, bdr.MX6, b), oracle_gemm(bdr.MX6, a, bdr.MX6, b)) <= 1e-5
    finally:
        bdr.bdr_set_workspace(None)
