"""The library's calls inside a CUDA graph: captured once (after a first call outside capture, which sets the
kernels' attributes), replayed on new data, results compared with the oracle.  bench.py times its step this way."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _bf16(x):
    return torch.from_numpy(synth.f32_to_bf16_bits(x).view(np.int16).reshape(x.shape)).view(torch.bfloat16).cuda()


def test_quantization_step_replayed_from_a_graph():
    rows, cols = 512, 4096
    host = [synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(H.make_input(k, rows, cols, "bf16", seed=s))).reshape(rows, cols)
            for k, s in (("normal", 1), ("laplace_outliers", 2))]
    x = _bf16(host[0])
    y_row, y_col, back = torch.empty_like(x), torch.empty_like(x), torch.empty_like(x)
    sums = torch.zeros((2, 2), dtype=torch.float64, device="cuda")
    planes = bdr.alloc_planes(bdr.MX6, rows, cols, 0)

    def step():
        sums.zero_()
        bdr.bdr_quant_dequant(bdr.MX9, x, y_row, axis=1, qsnr_sums=sums[0])
        bdr.bdr_quant_dequant(bdr.MX4, x, y_col, axis=0, qsnr_sums=sums[1])
        bdr.bdr_pack(bdr.MX6, x, planes, axis=0)
        bdr.bdr_unpack(bdr.MX6, planes, back, axis=0)

    step()                                   # first call outside capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for h in reversed(host):                 # replay on different data than the capture saw
        x.copy_(_bf16(h))
        g.replay()
        torch.cuda.synchronize()
        for cfg, axis, got, s in ((bdr.MX9, 1, y_row, sums[0]), (bdr.MX4, 0, y_col, sums[1])):
            want, so = orc.quant_dequant(H.to_orc(cfg), h, axis=axis)
            H.assert_bits_equal(H.device_to_host_f32(got), want, "%s axis=%d" % (cfg, axis))
            H.assert_qsnr_close(s.cpu().numpy(), so)
        H.assert_planes_equal(H.planes_to_host(planes), orc.pack(orc.MX6, h, axis=0), "planes")
        H.assert_bits_equal(H.device_to_host_f32(back), orc.quant_dequant(orc.MX6, h, axis=0)[0], "unpack")
    assert bdr.bdr_device_status() == 0


@pytest.mark.parametrize("entry", ["mx_gemm_f8", "mx_gemm_ws"])
def test_two_phase_gemms_replayed_from_a_graph(entry):
    M, N, K = 512, 512, 1024
    a = synth.normal_matrix(M, K, seed=3, stream=1)
    b = synth.normal_matrix(N, K, seed=3, stream=2, sigma=0.02)
    xa, xb = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    pa, pb = bdr.alloc_planes(bdr.MX6, M, K), bdr.alloc_planes(bdr.MX6, N, K)
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    size = bdr.mx_gemm_f8_workspace_bytes if entry == "mx_gemm_f8" else bdr.mx_gemm_workspace_bytes
    ws = torch.empty(size(M, N, K), dtype=torch.uint8, device="cuda")
    call = getattr(bdr, entry)

    def step():
        bdr.bdr_pack(bdr.MX6, xa, pa)
        bdr.bdr_pack(bdr.MX6, xb, pb)
        call(bdr.MX6, pa, bdr.MX6, pb, M, N, K, c, ws)

    step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    a2 = synth.outlier_channel_matrix(M, K, seed=4, stream=1, gain=20.0)
    xa.copy_(torch.from_numpy(a2))
    c.fill_(float("nan"))
    g.replay()
    torch.cuda.synchronize()
    assert bdr.mx_gemm_status() == 0 and bdr.bdr_device_status() == 0
    aq, bq = orc.quant_dequant(orc.MX6, a2)[0], orc.quant_dequant(orc.MX6, b)[0]
    ref = orc.gemm_nt_f64(aq, bq, nthreads=8)
    got = c.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5


def test_training_flow_calls_replayed_from_a_graph():
    # both packed copies from one read, Eq. 3 from the fused sums, the hardware-pipeline product and an embedding lookup
    rows, cols = 512, 512
    host = [H.make_input(k, rows, cols, "bf16", seed=s) for k, s in (("normal", 5), ("laplace_outliers", 6))]
    x = _bf16(host[0])
    pr, pc = bdr.alloc_planes(bdr.MX6, rows, cols, 1), bdr.alloc_planes(bdr.MX6, rows, cols, 0)
    sums = torch.zeros((2, 2), dtype=torch.float64, device="cuda")
    db = torch.zeros(2, dtype=torch.float64, device="cuda")
    c = torch.empty((rows, rows), dtype=torch.float32, device="cuda")
    idx = torch.tensor([5, 0, 511, 5], dtype=torch.int64, device="cuda")
    looked_up = torch.empty((4, cols), dtype=torch.bfloat16, device="cuda")

    def step():
        sums.zero_()
        bdr.bdr_pack2(bdr.MX6, x, pr, pc, sums[0], sums[1])
        bdr.bdr_qsnr_from_sums(sums, db)
        bdr.mx_gemm_hw(bdr.MX6, pr, bdr.MX6, pr, rows, rows, cols, c, r=64, f=12)
        bdr.bdr_gather_rows(bdr.MX6, pr, rows, idx, looked_up)

    step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for h in reversed(host):
        x.copy_(_bf16(h))
        g.replay()
        torch.cuda.synchronize()
        H.assert_planes_equal(H.planes_to_host(pr), orc.pack(orc.MX6, h, axis=1), "row planes")
        H.assert_planes_equal(H.planes_to_host(pc), orc.pack(orc.MX6, h, axis=0), "column planes")
        qd, so = orc.quant_dequant(orc.MX6, h, axis=1)
        want_db = [orc.qsnr_db(*so), orc.qsnr_db(*orc.quant_dequant(orc.MX6, h, axis=0)[1])]
        assert np.allclose(db.cpu().numpy(), want_db, rtol=H.QSNR_REL_TOL, atol=0)
        H.assert_bits_equal(c.cpu().numpy(), orc.gemm_hw(orc.MX6, h, orc.MX6, h, r=64, f=12), "hardware-pipeline product")
        H.assert_bits_equal(H.device_to_host_f32(looked_up), qd[[5, 0, 511, 5]], "lookup")
    assert bdr.bdr_device_status() == 0
