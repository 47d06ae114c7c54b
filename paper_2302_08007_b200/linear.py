"""One linear layer in MX training form (Section V, Fig. 8): every matmul of the forward and the
backward pass takes both operands MX-quantized along that matmul's reduction dimension, so each of
X, W and dY is quantized twice -- once along its rows and once along its columns (the "transpose,
then quantize" copy).  This module only sequences calls of the C ABI; all arithmetic is in the
kernels.

    Y  = X  W^T   reduce over in-features : X  row-wise, W  row-wise
    dX = dY W     reduce over out-features: dY row-wise, W  column-wise
    dW = dY^T X   reduce over tokens      : dY column-wise, X column-wise
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import binding as bdr


@dataclass
class LinearBuffers:
    """Everything the step writes, allocated once by the caller."""
    planes: dict           # (name, axis) -> Planes
    sums: torch.Tensor     # [6, 2] float64: Eq. 3 sums of the six quantizations
    y: torch.Tensor        # [tokens, out] float32
    dx: torch.Tensor       # [tokens, in] float32
    dw: torch.Tensor       # [out, in] float32
    workspace: torch.Tensor | None = None  # uint8 scratch for the two-phase GEMM (largest of the three products)


ORDER = (("x", 1), ("x", 0), ("w", 1), ("w", 0), ("dy", 1), ("dy", 0))


def alloc(cfg: bdr.Config, tokens: int, d_in: int, d_out: int, device="cuda", two_phase: bool = True) -> LinearBuffers:
    shapes = {"x": (tokens, d_in), "w": (d_out, d_in), "dy": (tokens, d_out)}
    planes = {(n, ax): bdr.alloc_planes(cfg, *shapes[n], ax, device=device) for n, ax in ORDER}
    ws = None
    if two_phase and tokens % 256 == 0 and d_in % 256 == 0 and d_out % 256 == 0:
        # formats with at most four significant bits take the 8-bit block-scaled GEMM, the others the bf16 one
        size = bdr.mx_gemm_f8_workspace_bytes if cfg.m <= 4 else bdr.mx_gemm_workspace_bytes
        nbytes = max(size(tokens, d_out, d_in), size(tokens, d_in, d_out), size(d_out, d_in, tokens))
        ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    return LinearBuffers(planes, torch.zeros((6, 2), dtype=torch.float64, device=device),
                         torch.empty((tokens, d_out), dtype=torch.float32, device=device),
                         torch.empty((tokens, d_in), dtype=torch.float32, device=device),
                         torch.empty((d_out, d_in), dtype=torch.float32, device=device), ws)


def step(cfg: bdr.Config, x: torch.Tensor, w: torch.Tensor, dy: torch.Tensor, buf: LinearBuffers, stream=None):
    """Six quantizations (three dual-direction calls, with fused QSNR sums) and three MX GEMMs.  Returns (Y, dX, dW)."""
    tokens, d_in = x.shape
    d_out = w.shape[0]
    src = {"x": x, "w": w, "dy": dy}
    buf.sums.zero_()
    for i, n in enumerate(("x", "w", "dy")):   # each tensor is read once and packed along both directions
        bdr.bdr_pack2(cfg, src[n], buf.planes[(n, 1)], buf.planes[(n, 0)], buf.sums[2 * i], buf.sums[2 * i + 1], stream=stream)
    p = buf.planes

    def gemm(a, b, M, N, K, c):
        if buf.workspace is not None and cfg.m <= 4:
            bdr.mx_gemm_f8(cfg, a, cfg, b, M, N, K, c, buf.workspace[:bdr.mx_gemm_f8_workspace_bytes(M, N, K)], stream=stream)
        elif buf.workspace is not None:
            bdr.mx_gemm_ws(cfg, a, cfg, b, M, N, K, c, buf.workspace, stream=stream)
        else:
            bdr.mx_gemm(cfg, a, cfg, b, M, N, K, c, stream=stream)

    gemm(p[("x", 1)], p[("w", 1)], tokens, d_out, d_in, buf.y)      # Y  = X W^T
    gemm(p[("dy", 1)], p[("w", 0)], tokens, d_in, d_out, buf.dx)    # dX = dY W
    gemm(p[("dy", 0)], p[("x", 0)], d_out, d_in, tokens, buf.dw)    # dW = dY^T X
    return buf.y, buf.dx, buf.dw


def qsnr_db(buf: LinearBuffers) -> dict:
    """Eq. 3 of the six quantized operands, from the sums the last step accumulated."""
    db = bdr.bdr_qsnr_from_sums(buf.sums, torch.empty(6, dtype=torch.float64, device=buf.sums.device)).cpu()
    return {"%s_%s" % (n, "row" if ax == 1 else "col"): float(db[i]) for i, (n, ax) in enumerate(ORDER)}
