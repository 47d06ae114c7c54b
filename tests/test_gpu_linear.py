"""GPU parity of the MX linear-layer step (forward + backward, six quantizations, three GEMMs)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import linear, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _inputs(tokens, d_in, d_out, seed):
    x = synth.outlier_channel_matrix(tokens, d_in, seed=seed, stream=1, frac=0.01, gain=20.0)
    w = synth.normal_matrix(d_out, d_in, seed=seed, stream=2, sigma=0.02)
    dy = synth.normal_matrix(tokens, d_out, seed=seed, stream=3, sigma=1e-3)
    to_bf16 = lambda a: synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(a)).reshape(a.shape)
    return to_bf16(x), to_bf16(w), to_bf16(dy)


def _run(cfg, x, w, dy, two_phase=True):
    dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
    buf = linear.alloc(cfg, x.shape[0], x.shape[1], w.shape[0], two_phase=two_phase)
    assert (buf.workspace is not None) == two_phase
    y, dx, dw = linear.step(cfg, dev(x), dev(w), dev(dy), buf)
    torch.cuda.synchronize()
    assert bdr.mx_gemm_status() == 0
    return y.cpu().numpy(), dx.cpu().numpy(), dw.cpu().numpy(), linear.qsnr_db(buf), buf


@pytest.mark.parametrize("two_phase", [True, False], ids=["with_workspace", "no_workspace"])
@pytest.mark.parametrize("fmt", ["MX9", "MX6"])
def test_linear_step_small_shapes_full_oracle(fmt, two_phase):
    cfg = {"MX9": bdr.MX9, "MX6": bdr.MX6}[fmt]
    o = H.to_orc(cfg)
    x, w, dy = _inputs(512, 256, 768, seed=5)
    y, dx, dw, q, buf = _run(cfg, x, w, dy, two_phase)
    qd = lambda a, ax: orc.quant_dequant(o, a, axis=ax)
    (xr, sxr), (xc, sxc) = qd(x, 1), qd(x, 0)
    (wr, swr), (wc, swc) = qd(w, 1), qd(w, 0)
    (gr, sgr), (gc, sgc) = qd(dy, 1), qd(dy, 0)
    rel = lambda c, ref: np.linalg.norm(c - ref) / np.linalg.norm(ref)
    assert rel(y, orc.gemm_nt_f64(xr, wr, nthreads=8)) <= 1e-5
    assert rel(dx, orc.gemm_nt_f64(gr, np.ascontiguousarray(wc.T), nthreads=8)) <= 1e-5
    assert rel(dw, orc.gemm_nt_f64(np.ascontiguousarray(gc.T), np.ascontiguousarray(xc.T), nthreads=8)) <= 1e-5
    for key, s in (("x_row", sxr), ("x_col", sxc), ("w_row", swr), ("w_col", swc), ("dy_row", sgr), ("dy_col", sgc)):
        want = orc.qsnr_db(*s)
        assert abs(q[key] - want) <= H.QSNR_REL_TOL * abs(want), (key, q[key], want)
    # the column-direction planes are the row-direction planes of the transpose, byte for byte
    H.assert_planes_equal(H.planes_to_host(buf.planes[("w", 0)]), orc.pack(o, np.ascontiguousarray(w.T), axis=1))


def test_linear_step_config5_shapes_on_sampled_entries():
    cfg, o = bdr.MX9, orc.MX9
    tokens, d_in, d_out = 8192, 4096, 16384
    x, w, dy = _inputs(tokens, d_in, d_out, seed=0)
    y, dx, dw, q, _ = _run(cfg, x, w, dy)
    rng = np.random.default_rng(9)
    row = lambda a, i: orc.quant_dequant(o, a[i:i + 1, :], axis=1)[0][0]            # line i quantized along the row
    col = lambda a, j: orc.quant_dequant(o, a[:, j:j + 1], axis=0)[0][:, 0]          # line j quantized down the column
    err = []
    for _ in range(48):
        t, i, n = rng.integers(tokens), rng.integers(d_in), rng.integers(d_out)
        err.append((y[t, n], float(row(x, t).astype(np.float64) @ row(w, n).astype(np.float64))))
        err.append((dx[t, i], float(row(dy, t).astype(np.float64) @ col(w, i).astype(np.float64))))
        err.append((dw[n, i], float(col(dy, n).astype(np.float64) @ col(x, i).astype(np.float64))))
    got, ref = np.array([e[0] for e in err], dtype=np.float64), np.array([e[1] for e in err])
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert all(np.isfinite(v) and v > 30.0 for v in q.values()), q                   # MX9 keeps > 30 dB on all six
