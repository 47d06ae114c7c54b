"""MX4 / MX6 operands on the block-scaled 8-bit tensor-core path: the re-encoding (E4M3 elements, one
power-of-two scale per 32 elements) must reproduce the oracle's decoded operand exactly, and the product
must match the oracle's fp64 product of the decoded operands like the bf16 kernels do."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from oracle import reencode as orc_re
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

FMT = {"MX4": bdr.MX4, "MX6": bdr.MX6}


def _pack(cfg, x_host):
    rows, K = x_host.shape
    p = bdr.alloc_planes(cfg, rows, K)
    bdr.bdr_pack(cfg, torch.from_numpy(x_host).cuda(), p)
    return p


def _reencode(cfg, x_host):
    rows, K = x_host.shape
    p = _pack(cfg, x_host)
    out = torch.full((rows, K), 0x7F, dtype=torch.uint8, device="cuda")
    sf = torch.full((rows * K // 32,), 0xEE, dtype=torch.uint8, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    bdr.bdr_reencode_e4m3(cfg, p, rows, K, out, sf, flag)
    torch.cuda.synchronize()
    # bytes, scale bytes and the flag against the oracle's re-encoding (bytes are unspecified once the flag is up)
    want_out, want_sf, want_flag = orc_re.reencode_e4m3(H.to_orc(cfg), x_host)
    assert int(flag.item()) == int(want_flag)
    if not want_flag:
        assert np.array_equal(out.cpu().numpy(), want_out)
    assert np.array_equal(sf.cpu().numpy(), want_sf)
    vals = out.view(torch.float8_e4m3fn).to(torch.float32).cpu().numpy().astype(np.float64)
    # scale of (row r, group g): atom [g // 4][r // 128], byte (r % 32) * 16 + ((r % 128) // 32) * 4 + g % 4
    sfh = sf.cpu().numpy().reshape(K // 128, rows // 128, 32, 4, 4)          # [chunk][row tile][r % 32][(r % 128) // 32][g % 4]
    per = sfh.transpose(1, 3, 2, 0, 4).reshape(rows, K // 32).astype(np.int64)  # [row tile, r // 32, r % 32] -> row; [chunk, g % 4] -> group
    scale = np.ldexp(1.0, per - 127)
    return vals * np.repeat(scale, 32, axis=1), int(flag.item()), out.cpu().numpy(), per


@pytest.mark.parametrize("name", list(FMT))
def test_reencoding_is_exact(name):
    cfg = FMT[name]
    for kind, rows, K in (("normal", 256, 640), ("laplace_outliers", 128, 1024), ("normal", 384, 128)):
        x = H.make_input(kind, rows, K, "f32", seed=rows + K)
        want, _ = orc.quant_dequant(H.to_orc(cfg), x)
        got, flag, _, _ = _reencode(cfg, x)
        assert flag == 0, (name, kind)
        assert np.array_equal(got, want.astype(np.float64)), (name, kind)
        assert np.array_equal(np.signbit(got), np.signbit(want)), (name, kind)   # signed zeros too


def test_reencoding_exponent_gaps_between_neighbouring_blocks():
    # block pairs whose exponents are d binades apart: exact while the smaller block's elements keep their low
    # bits above 2^-9 of the group scale, flagged beyond that; an all-zero neighbour is always fine
    rng = np.random.default_rng(3)
    rows, K = 128, 512
    for cfg, m in ((bdr.MX6, 4), (bdr.MX4, 2)):
        limit = 9 + 7 - (m - 1)          # t = 7 - (m-1) - d - tau >= -9; every pair holds a value in [1, 2) * 2^F, so tau = 0
        for d in (0, 1, 5, limit, limit + 1, limit + 4, 30):
            mant = 1.0 + rng.integers(0, 8, (rows, K)) / 8.0
            x = (mant * np.where(rng.random((rows, K)) < 0.5, -1.0, 1.0)).astype(np.float32)
            x[:, 16:32] *= np.float32(2.0 ** -d)                 # second block of the first group of every row
            x[:, 48:64] = 0.0                                    # an all-zero block beside a normal one
            want, _ = orc.quant_dequant(H.to_orc(cfg), x)
            got, flag, _, _ = _reencode(cfg, x)
            exact = np.array_equal(got, want.astype(np.float64))
            if d <= limit:
                assert flag == 0 and exact, (m, d)
            else:
                assert flag == 1, (m, d)                          # never silently inexact
                assert np.array_equal(got[:, 32:], want[:, 32:].astype(np.float64)), (m, d)   # other groups unaffected
    # tiny and non-finite blocks raise the flag as well
    for bad in (np.float32(1e-38), np.float32(np.inf)):
        x = H.make_input("normal", rows, K, "f32", seed=5)
        x[7, 96:112] = bad                                       # a whole block: its exponent is 1 or 255
        _, flag, _, _ = _reencode(bdr.MX6, x)
        assert flag == 1


def gpu_gemm_f8(cfg_a, a_host, cfg_b, b_host):
    M, K = a_host.shape
    N = b_host.shape[0]
    pa, pb = _pack(cfg_a, a_host), _pack(cfg_b, b_host)
    ws = torch.empty(bdr.mx_gemm_f8_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    c = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    bdr.mx_gemm_f8(cfg_a, pa, cfg_b, pb, M, N, K, c, ws)
    torch.cuda.synchronize()
    assert bdr.mx_gemm_status() == 0 and bdr.bdr_device_status() == 0
    flag = int(ws[-256:-252].view(torch.int32).item())
    return c.cpu().numpy(), flag


def oracle_gemm(cfg_a, a_host, cfg_b, b_host):
    aq, _ = orc.quant_dequant(H.to_orc(cfg_a), a_host)
    bq, _ = orc.quant_dequant(H.to_orc(cfg_b), b_host)
    return orc.gemm_nt_f64(aq, bq, nthreads=8)


def rel_frob(c, ref):
    return float(np.linalg.norm(c.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


def test_f8_exact_case_small_integers():
    # products and sums are small integers: every summation order gives the same fp32 result
    rng = np.random.default_rng(2)
    a = rng.integers(-8, 9, (256, 256)).astype(np.float32)
    b = rng.integers(-8, 9, (512, 256)).astype(np.float32)
    a[:, ::16] = 8.0
    b[:, ::16] = -8.0
    c, flag = gpu_gemm_f8(bdr.MX6, a, bdr.MX6, b)
    assert flag == 0
    assert np.array_equal(c.astype(np.int64), a.astype(np.int64) @ b.astype(np.int64).T)


def test_f8_scales_of_every_row_and_group_reach_the_product():
    # one non-zero element per row of A at a K position that walks over every 32-element group, each row with its own
    # power of two; B = rows of ones scaled per row: C[i, j] = 2^(ea_i + eb_j) exactly, so a scale read from the
    # wrong row, group, CTA or column shows up
    M, N, K = 512, 512, 512
    a = np.zeros((M, K), np.float32)
    ea = (np.arange(M) * 7) % 23 - 11
    a[np.arange(M), (np.arange(M) * 37) % K] = np.ldexp(1.0, ea).astype(np.float32)
    eb = (np.arange(N) * 5) % 19 - 9
    b = np.ones((N, K), np.float32) * np.ldexp(1.0, eb).astype(np.float32)[:, None]
    c, flag = gpu_gemm_f8(bdr.MX6, a, bdr.MX4, b)
    assert flag == 0
    assert np.array_equal(c.astype(np.float64), np.ldexp(1.0, ea[:, None] + eb[None, :]))


@pytest.mark.parametrize("fa,fb", [("MX6", "MX6"), ("MX6", "MX4"), ("MX4", "MX6"), ("MX4", "MX4")])
def test_f8_random_operands_match_the_oracle(fa, fb):
    M, N, K = 512, 768, 1280                             # six tiles, 10 K steps (the ring wraps)
    a = synth.normal_matrix(M, K, seed=7, stream=1)
    b = synth.outlier_channel_matrix(N, K, seed=7, stream=2, gain=20.0, dist="normal", sigma=0.02)
    c, flag = gpu_gemm_f8(FMT[fa], a, FMT[fb], b)
    assert flag == 0
    assert rel_frob(c, oracle_gemm(FMT[fa], a, FMT[fb], b)) <= 1e-5


def test_f8_more_tiles_than_clusters():
    M, N, K = 6144, 4096, 256                            # 384 tiles: every cluster walks over several tiles
    a = synth.normal_matrix(M, K, seed=8, stream=1)
    b = synth.normal_matrix(N, K, seed=8, stream=2, sigma=0.02)
    c, flag = gpu_gemm_f8(bdr.MX6, a, bdr.MX6, b)
    assert flag == 0
    assert rel_frob(c, oracle_gemm(bdr.MX6, a, bdr.MX6, b)) <= 1e-5


def test_f8_padded_output_pitch_keeps_the_padding():
    # C is a view of a wider buffer: the split tiles are cleared and accumulated with the view's pitch, and the
    # columns beside the view stay untouched
    M, N, K = 512, 256, 512
    a = synth.normal_matrix(M, K, seed=21, stream=1)
    b = synth.normal_matrix(N, K, seed=21, stream=2, sigma=0.02)
    pa, pb = _pack(bdr.MX6, a), _pack(bdr.MX6, b)
    ws = torch.empty(bdr.mx_gemm_f8_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    wide = torch.full((M, N + 64), 7.0, dtype=torch.float32, device="cuda")
    bdr.mx_gemm_f8(bdr.MX6, pa, bdr.MX6, pb, M, N, K, wide[:, :N], ws)
    torch.cuda.synchronize()
    assert bdr.mx_gemm_status() == 0
    got = wide.cpu().numpy()
    assert (got[:, N:] == 7.0).all()
    assert rel_frob(got[:, :N], oracle_gemm(bdr.MX6, a, bdr.MX6, b)) <= 1e-5


def test_gemm_from_operands_re_encoded_earlier():
    # weights re-encoded once, activations per call: the GEMM kernel on its own
    M, N, K = 512, 1024, 768
    a = synth.outlier_channel_matrix(M, K, seed=31, stream=1, gain=20.0)
    b = synth.normal_matrix(N, K, seed=31, stream=2, sigma=0.02)
    enc = []
    for cfg, x in ((bdr.MX6, a), (bdr.MX4, b)):
        rows = x.shape[0]
        out = torch.empty((rows, K), dtype=torch.uint8, device="cuda")
        sf = torch.empty(rows * K // 32, dtype=torch.uint8, device="cuda")
        flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        bdr.bdr_reencode_e4m3(cfg, _pack(cfg, x), rows, K, out, sf, flag)
        assert int(flag.item()) == 0
        enc += [out, sf]
    for _ in range(2):                                       # the second call finds C full of the first call's result
        c = torch.full((M, N), 3.0, dtype=torch.float32, device="cuda")
        bdr.mx_gemm_e4m3(enc[0], enc[1], enc[2], enc[3], M, N, K, c)
        torch.cuda.synchronize()
        assert bdr.mx_gemm_status() == 0
        assert rel_frob(c.cpu().numpy(), oracle_gemm(bdr.MX6, a, bdr.MX4, b)) <= 1e-5


def test_f8_whole_rounds_only():
    # 64 tiles on 74 clusters: more than half of the clusters are busy in the only round, so no tile's K range is
    # split in two (the other tests have few tiles, or a sparse last round, and take the split path)
    M, N, K = 2048, 2048, 256
    a = synth.normal_matrix(M, K, seed=11, stream=1)
    b = synth.normal_matrix(N, K, seed=11, stream=2, sigma=0.02)
    c, flag = gpu_gemm_f8(bdr.MX4, a, bdr.MX6, b)
    assert flag == 0
    assert rel_frob(c, oracle_gemm(bdr.MX4, a, bdr.MX6, b)) <= 1e-5


def test_f8_falls_back_when_the_operands_are_not_representable():
    M, N, K = 256, 256, 512
    a = synth.normal_matrix(M, K, seed=9, stream=1)
    b = synth.normal_matrix(N, K, seed=9, stream=2, sigma=0.02)
    a[:, 16:32] *= np.float32(2.0 ** -20)                # neighbouring blocks twenty binades apart
    c, flag = gpu_gemm_f8(bdr.MX6, a, bdr.MX6, b)
    assert flag == 1
    assert rel_frob(c, oracle_gemm(bdr.MX6, a, bdr.MX6, b)) <= 1e-5
    b[3, 0:16] = np.float32(1e-38)                       # a block exponent below the supported range
    c, flag = gpu_gemm_f8(bdr.MX6, synth.normal_matrix(M, K, seed=1), bdr.MX6, b)
    assert flag == 1
    assert rel_frob(c, oracle_gemm(bdr.MX6, synth.normal_matrix(M, K, seed=1), bdr.MX6, b)) <= 1e-5


def test_f8_config4_shape_on_sampled_entries():
    M = N = K = 4096
    a = synth.normal_matrix(M, K, seed=0, stream=10)
    b = synth.normal_matrix(N, K, seed=0, stream=11, sigma=0.02)
    c, flag = gpu_gemm_f8(bdr.MX6, a, bdr.MX6, b)
    assert flag == 0
    aq, _ = orc.quant_dequant(orc.MX6, a, nthreads=8)
    bq, _ = orc.quant_dequant(orc.MX6, b, nthreads=8)
    rng = np.random.default_rng(5)
    ri, ci = rng.integers(0, M, 4096), rng.integers(0, N, 4096)
    ref = orc.gemm_nt_f64_sampled(aq, bq, ri, ci)
    got = c[ri, ci].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert np.isfinite(c).all()
    assert rel_frob(c[-256:], orc.gemm_nt_f64(aq[-256:], bq, nthreads=8)) <= 1e-5


def test_f8_tiles_walked_in_bands_with_split_tiles():
    # 8-bit operands above 64 MiB: 9 x 10 tiles in bands of eight tile rows; the 16 tiles of the last round are split
    # along K and accumulate into tiles that the first phase cleared, addressed in the same banded order
    M, N, K = 2304, 2560, 16384
    a = synth.normal_matrix(M, K, seed=22, stream=1)
    b = synth.normal_matrix(N, K, seed=22, stream=2, sigma=0.02)
    c, flag = gpu_gemm_f8(bdr.MX6, a, bdr.MX6, b)
    assert flag == 0
    assert np.isfinite(c).all()
    aq, _ = orc.quant_dequant(orc.MX6, a, nthreads=8)
    bq, _ = orc.quant_dequant(orc.MX6, b, nthreads=8)
    rng = np.random.default_rng(7)
    ri, ci = rng.integers(0, M, 8192), rng.integers(0, N, 8192)
    ref = orc.gemm_nt_f64_sampled(aq, bq, ri, ci)
    got = c[ri, ci].astype(np.float64)
    assert np.max(np.abs(got - ref)) <= 1e-4 * np.max(np.abs(ref))
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert rel_frob(c[-256:], orc.gemm_nt_f64(aq[-256:], bq, nthreads=8)) <= 1e-5   # the one-row band holds the split tiles


def test_f8_argument_errors():
    pa, pb = bdr.alloc_planes(bdr.MX6, 256, 256), bdr.alloc_planes(bdr.MX9, 256, 256)
    c = torch.empty((256, 256), device="cuda")
    ws = torch.empty(bdr.mx_gemm_f8_workspace_bytes(256, 256, 256), dtype=torch.uint8, device="cuda")
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_f8(bdr.MX6, pa, bdr.MX9, pb, 256, 256, 256, c, ws)                 # m = 7 needs eight significant bits
    assert e.value.status == -3
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_f8(bdr.MX6, pa, bdr.MX6, pa, 256, 256, 256, c, ws[:4096])          # workspace too small
    assert e.value.status == -6
    with pytest.raises(bdr.BdrError) as e:
        bdr.mx_gemm_f8(bdr.MX6, pa, bdr.MX6, pa, 256, 256, 128, c, ws)                 # K must be a multiple of 256
    assert e.value.status == -3
    torch.cuda.synchronize()


@pytest.mark.parametrize("seed", range(12))
def test_f8_random_exponent_structure(seed):
    # block exponents drawn at random per 16-element block (spread chosen per case from "always representable" to
    # "often not"), some blocks all zero, some rows scaled as a whole; whatever path the call takes on the device,
    # the product must match the oracle, and the re-encoding must be exact whenever it says so
    rng = np.random.default_rng(100 + seed)
    M, N, K = 256, 256 * int(rng.integers(1, 3)), 256 * int(rng.integers(1, 5))
    fa, fb = (bdr.MX6, bdr.MX4)[int(rng.integers(2))], (bdr.MX6, bdr.MX4)[int(rng.integers(2))]
    spread = int(rng.choice([0, 3, 8, 12, 16, 24]))

    def operand(rows):
        mant = rng.standard_normal((rows, K))
        e = rng.integers(-spread, 1, (rows, K // 16)) if spread else np.zeros((rows, K // 16), np.int64)
        x = mant * np.repeat(np.ldexp(1.0, e), 16, axis=1)
        x *= np.ldexp(1.0, rng.integers(-20, 20, (rows, 1)))
        x[np.repeat(rng.random((rows, K // 16)) < 0.05, 16, axis=1)] = 0.0
        return x.astype(np.float32)

    a, b = operand(M), operand(N)
    c, flag = gpu_gemm_f8(fa, a, fb, b)
    assert rel_frob(c, oracle_gemm(fa, a, fb, b)) <= 1e-5, (seed, flag)
    for cfg, x in ((fa, a), (fb, b)):
        got, inexact, _, _ = _reencode(cfg, x)
        want, _ = orc.quant_dequant(H.to_orc(cfg), x)
        if not inexact:
            assert np.array_equal(got, want.astype(np.float64)), seed
        else:
            assert flag == 1, seed
    if spread <= 8:
        assert flag == 0, seed
