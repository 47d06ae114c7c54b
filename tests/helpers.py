"""Shared helpers for the GPU parity tests: run the CUDA path through the C ABI binding and the
oracle on the same host arrays, and compare bit patterns."""
import math

import numpy as np
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth

# QSNR tolerance from the target statement: 1e-6 dB relative.
QSNR_REL_TOL = 1e-6
# Relative bound on the fused sums of Eq. 3 (derivation in assert_qsnr_close): 16 fp32 roundings per partial sum.
SUM_REL_TOL = 1.01 * 2.0 ** -20


def to_orc(cfg: bdr.Config) -> orc.Config:
    return orc.Config(cfg.k1, cfg.d1, cfg.k2, cfg.d2, cfg.m, cfg.scale_kind, cfg.rounding)


def host_to_device(x_f32: np.ndarray, dtype: str, ld: int | None = None) -> torch.Tensor:
    """x_f32: 2-D fp32 host array whose values are exactly representable in `dtype`."""
    rows, cols = x_f32.shape
    ld = cols if ld is None else ld
    t = torch.from_numpy(np.ascontiguousarray(x_f32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    buf = torch.zeros((rows, ld), dtype=t.dtype, device="cuda")
    buf[:, :cols] = t.cuda()
    return buf[:, :cols]


def device_to_host_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy()


def make_input(kind: str, rows: int, cols: int, dtype: str, seed: int) -> np.ndarray:
    n = rows * cols
    if kind == "normal":
        x = synth.normal(n, seed)
    elif kind == "edge":
        x = synth.edge_case_values(n, seed)
    elif kind == "laplace_outliers":
        x = synth.outlier_channel_matrix(rows, cols, seed, gain=50.0).ravel()
    elif kind == "tiny":
        x = synth.normal(n, seed) * np.float32(1e-38)
    elif kind == "huge":
        x = synth.normal(n, seed) * np.float32(1e37)
    else:
        raise ValueError(kind)
    x = x.reshape(rows, cols).astype(np.float32)
    if dtype == "bf16":
        x = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x)).reshape(rows, cols)
        x = np.where(np.isfinite(x), x, np.float32(1.0)).astype(np.float32)
    return x


def assert_bits_equal(got: np.ndarray, want: np.ndarray, what: str = ""):
    g = np.ascontiguousarray(got, dtype=np.float32).view(np.uint32)
    w = np.ascontiguousarray(want, dtype=np.float32).view(np.uint32)
    if not np.array_equal(g, w):
        bad = np.argwhere(g != w)
        i = tuple(bad[0])
        raise AssertionError("%s: %d of %d values differ; first at %s: got %r (0x%08x) want %r (0x%08x)" % (
            what, len(bad), g.size, i, got[i], g[i], want[i], w[i]))


def assert_qsnr_close(sums_gpu, sums_orc, what: str = ""):
    e_g, s_g = float(sums_gpu[0]), float(sums_gpu[1])
    e_o, s_o = sums_orc
    if math.isnan(e_o) or math.isnan(s_o):
        assert math.isnan(e_g) or math.isnan(s_g), what
        return
    # Both sums are sums of non-negative terms.  The kernels form each term in fp32 in the block-normalised
    # domain (one rounding, relative 2^-24, for the square of an fp32 input; exact for bf16 inputs and for the
    # error terms), add at most 16 of them in fp32 (at most 15 additions, each relative 2^-24 on a partial sum
    # of non-negative terms) and continue in fp64 after an exact power-of-two rescaling.  A sum of non-negative
    # terms inherits the worst relative error of its parts: (1 + 2^-24)^16 - 1 < 2^-20.  The fp64 part adds
    # at most a few 2^-53 per addition and is covered by the 1 % slack.
    assert s_g == np.float64(s_o) or abs(s_g - s_o) <= SUM_REL_TOL * abs(s_o), (what, s_g, s_o)
    q_g, q_o = orc.qsnr_db(e_g, s_g), orc.qsnr_db(e_o, s_o)
    if math.isinf(q_o) or math.isnan(q_o):
        assert (math.isinf(q_g) and math.isinf(q_o)) or (math.isnan(q_g) and math.isnan(q_o)), (what, q_g, q_o)
    else:
        assert abs(q_g - q_o) <= QSNR_REL_TOL * max(abs(q_o), 1e-3), (what, q_g, q_o)


def planes_to_host(p: bdr.Planes):
    return tuple(t.cpu().numpy() for t in (p.exps, p.micro, p.elems))


def assert_planes_equal(got, want, what: str = ""):
    for name, g, w in zip(("exps", "micro", "elems"), got, want):
        assert g.shape == w.shape, (what, name, g.shape, w.shape)
        if not np.array_equal(g, w):
            bad = np.argwhere(g != w)
            i = tuple(bad[0])
            raise AssertionError("%s plane %s: %d bytes differ; first at %s: got 0x%02x want 0x%02x" % (
                what, name, len(bad), i, g[i], w[i]))
