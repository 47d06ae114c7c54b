"""Thin ctypes binding over the C ABI declared in ``include/bdr.h``.

Argument marshalling only: torch tensors provide device memory and streams, every step of the
method runs inside the CUDA library.  There is no CPU fallback: if the library is missing, loading
raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libbdr_b200.so")

SCALE_POW2, SCALE_FP32_INT, SCALE_FP32_FP, SCALE_FP32_VSQ = 0, 1, 2, 3
ROUND_NEAREST_EVEN, ROUND_NEAREST_AWAY = 0, 1
F32, BF16 = 0, 1

EXPORTS = ("bdr_strerror", "bdr_device_status", "bdr_packed_sizes", "bdr_quant_dequant", "bdr_pack", "bdr_unpack",
           "bdr_qsnr_workspace_bytes", "bdr_qsnr", "bdr_qsnr_static_max_cfgs", "bdr_qsnr_static", "mx_gemm",
           "mx_gemm_workspace_bytes", "mx_gemm_ws", "mx_gemm_f8_workspace_bytes", "mx_gemm_f8", "bdr_reencode_e4m3", "mx_gemm_e4m3", "bdr_set_workspace",
           "mx_gemm_status", "bdr_selftest_bounded_wait", "bdr_selftest_host", "bdr_qsnr_from_sums", "bdr_pack2", "bdr_qsnr_delayed", "bdr_amax", "bdr_tile_packing_efficiency", "mx_gemm_hw", "bdr_gather_rows", "bdr_device_status_reset", "bdr_quant_dequant_parent")


class BdrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, strerror(status), status))


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("k1", "d1", "k2", "d2", "m", "scale_kind", "rounding")]


class _Planes(C.Structure):
    _fields_ = [("exps", C.c_void_p), ("micro", C.c_void_p), ("elems", C.c_void_p),
                ("ld_exps", C.c_int64), ("ld_micro", C.c_int64), ("ld_elems", C.c_int64)]


@dataclass(frozen=True)
class Config:
    """bdr_config_t: the (k1, d1, k2, d2, m) tuple of Section III plus scale kind and tie rule."""
    k1: int
    d1: int
    k2: int
    d2: int
    m: int
    scale_kind: int = SCALE_POW2
    rounding: int = ROUND_NEAREST_EVEN

    def c(self) -> _Config:
        return _Config(self.k1, self.d1, self.k2, self.d2, self.m, self.scale_kind, self.rounding)


MX9 = Config(16, 8, 2, 1, 7)
MX6 = Config(16, 8, 2, 1, 4)
MX4 = Config(16, 8, 2, 1, 2)


@dataclass
class Planes:
    """Device tensors (uint8, [nlines, ld]) holding the three packed planes."""
    exps: torch.Tensor
    micro: torch.Tensor
    elems: torch.Tensor

    def c(self) -> _Planes:
        return _Planes(self.exps.data_ptr(), self.micro.data_ptr() if self.micro.numel() else None,
                       self.elems.data_ptr(), self.exps.stride(0), self.micro.stride(0) if self.micro.numel() else 0,
                       self.elems.stride(0))


_lib = None


def lib():
    """Load the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("CUDA library %s is missing: run paper_2302_08007_b200/build.py "
                              "(or __graft_entry__.build())" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        L.bdr_strerror.restype = C.c_char_p
        L.bdr_strerror.argtypes = [C.c_int]
        L.bdr_packed_sizes.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int, C.c_void_p, C.c_void_p]
        L.bdr_quant_dequant.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64,
                                        C.c_int, C.c_void_p, C.c_void_p]
        L.bdr_pack.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_void_p,
                               C.c_void_p, C.c_void_p, C.c_void_p]
        L.bdr_unpack.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int,
                                 C.c_void_p]
        L.bdr_qsnr_delayed.restype = C.c_int
        L.bdr_qsnr_delayed.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int,
                                       C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.bdr_amax.restype = C.c_int
        L.bdr_amax.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
        L.bdr_tile_packing_efficiency.restype = C.c_double
        L.bdr_tile_packing_efficiency.argtypes = [C.c_void_p, C.c_int64, C.c_int64]
        L.mx_gemm_hw.restype = C.c_int
        L.mx_gemm_hw.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int,
                                 C.c_void_p, C.c_int64, C.c_void_p]
        L.bdr_quant_dequant_parent.restype = C.c_int
        L.bdr_quant_dequant_parent.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64,
                                               C.c_int, C.c_void_p, C.c_void_p]
        L.bdr_gather_rows.restype = C.c_int
        L.bdr_gather_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int,
                                      C.c_int64, C.c_void_p]
        L.bdr_pack2.restype = C.c_int
        L.bdr_pack2.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.c_void_p, C.c_void_p]
        L.bdr_qsnr_workspace_bytes.restype = C.c_int64
        L.bdr_qsnr_workspace_bytes.argtypes = [C.c_int]
        L.bdr_qsnr.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int,
                               C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.mx_gemm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                              C.c_void_p, C.c_int64, C.c_void_p]
        L.bdr_qsnr_static_max_cfgs.restype = C.c_int
        L.bdr_qsnr_static_max_cfgs.argtypes = []
        L.bdr_qsnr_static.restype = C.c_int
        L.bdr_qsnr_static.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int,
                                      C.c_void_p, C.c_void_p]
        L.mx_gemm_workspace_bytes.restype = C.c_int64
        L.mx_gemm_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int64]
        L.mx_gemm_ws.restype = C.c_int
        L.mx_gemm_ws.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                 C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p]
        L.mx_gemm_f8_workspace_bytes.restype = C.c_int64
        L.mx_gemm_f8_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int64]
        L.mx_gemm_f8.restype = C.c_int
        L.mx_gemm_f8.argtypes = L.mx_gemm_ws.argtypes
        L.bdr_reencode_e4m3.restype = C.c_int
        L.bdr_reencode_e4m3.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.bdr_set_workspace.restype = C.c_int
        L.bdr_set_workspace.argtypes = [C.c_void_p, C.c_int64]
        L.mx_gemm_e4m3.restype = C.c_int
        L.mx_gemm_e4m3.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p,
                                   C.c_int64, C.c_void_p]
        L.mx_gemm_status.restype = C.c_int
        L.mx_gemm_status.argtypes = []
        L.bdr_device_status.restype = C.c_int
        L.bdr_device_status.argtypes = []
        L.bdr_device_status_reset.restype = C.c_int
        L.bdr_device_status_reset.argtypes = []
        L.bdr_selftest_bounded_wait.restype = C.c_int
        L.bdr_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_void_p]
        L.bdr_selftest_host.restype = C.c_int
        L.bdr_selftest_host.argtypes = []
        L.bdr_qsnr_from_sums.restype = C.c_int
        L.bdr_qsnr_from_sums.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        for fn in (L.bdr_packed_sizes, L.bdr_quant_dequant, L.bdr_pack, L.bdr_unpack, L.bdr_qsnr, L.mx_gemm):
            fn.restype = C.c_int
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().bdr_strerror(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise BdrError(status, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("tensor dtype must be float32 or bfloat16")


def _stream(stream) -> C.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _as2d(t: torch.Tensor):
    if t.dim() == 1:
        t = t.unsqueeze(0)
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 1-D or row-major 2-D tensor")
    return t


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def bdr_packed_sizes(cfg: Config, rows: int, cols: int, axis: int = 1):
    """Default line pitches and plane sizes in bytes: ([ld_exps, ld_micro, ld_elems], [bytes...])."""
    ld = (C.c_int64 * 3)()
    nb = (C.c_int64 * 3)()
    c = cfg.c()
    _check(lib().bdr_packed_sizes(C.addressof(c), rows, cols, axis, C.addressof(ld), C.addressof(nb)),
           "bdr_packed_sizes")
    return list(ld), list(nb)


def alloc_planes(cfg: Config, rows: int, cols: int, axis: int = 1, device="cuda") -> Planes:
    ld, _ = bdr_packed_sizes(cfg, rows, cols, axis)
    nlines = rows if axis == 1 else cols
    mk = lambda l: torch.empty((nlines, l), dtype=torch.uint8, device=device)
    return Planes(mk(ld[0]), mk(ld[1]), mk(ld[2]))


def bdr_quant_dequant(cfg: Config, x: torch.Tensor, y: torch.Tensor | None = None, axis: int = 1,
                      qsnr_sums: torch.Tensor | None = None, stream=None) -> torch.Tensor | None:
    """Q(x) into ``y`` (same dtype/shape/pitch as x; may be x itself).  ``qsnr_sums`` (2 float64 on
    the device) is accumulated into."""
    x2 = _as2d(x)
    y2 = _as2d(y) if y is not None else None
    if y2 is not None and (y2.shape != x2.shape or y2.stride(0) != x2.stride(0) or y2.dtype != x2.dtype):
        raise ValueError("y must match x in shape, pitch and dtype")
    c = cfg.c()
    _check(lib().bdr_quant_dequant(C.addressof(c), _ptr(x2), _ptr(y2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0),
                                   axis, _ptr(qsnr_sums), _stream(stream)), "bdr_quant_dequant")
    return y


def bdr_pack(cfg: Config, x: torch.Tensor, planes: Planes, axis: int = 1, y_dq: torch.Tensor | None = None,
             qsnr_sums: torch.Tensor | None = None, stream=None) -> Planes:
    x2 = _as2d(x)
    y2 = _as2d(y_dq) if y_dq is not None else None
    if y2 is not None and (y2.shape != x2.shape or y2.stride(0) != x2.stride(0) or y2.dtype != x2.dtype):
        raise ValueError("y_dq must match x in shape, pitch and dtype")
    c, p = cfg.c(), planes.c()
    _check(lib().bdr_pack(C.addressof(c), _ptr(x2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0), axis,
                          C.addressof(p), _ptr(y2), _ptr(qsnr_sums), _stream(stream)), "bdr_pack")
    return planes


def bdr_pack2(cfg: Config, x: torch.Tensor, planes_rows: Planes, planes_cols: Planes, qsnr_sums_rows: torch.Tensor | None = None,
              qsnr_sums_cols: torch.Tensor | None = None, stream=None):
    """Both packed copies of x -- quantized along its rows (axis 1) and along its columns (axis 0) -- from one read."""
    x2 = _as2d(x)
    c, pr, pc = cfg.c(), planes_rows.c(), planes_cols.c()
    _check(lib().bdr_pack2(C.addressof(c), _ptr(x2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0), C.addressof(pr),
                           C.addressof(pc), _ptr(qsnr_sums_rows), _ptr(qsnr_sums_cols), _stream(stream)), "bdr_pack2")
    return planes_rows, planes_cols


def bdr_quant_dequant_parent(cfg: Config, k_parent: int, x: torch.Tensor, y: torch.Tensor | None, axis: int = 1,
                             qsnr_sums: torch.Tensor | None = None, stream=None):
    """Three-level scaling: FP32 parent scale per k_parent elements of a line above the two-level quantizer (fp32 tensors)."""
    x2 = _as2d(x)
    y2 = _as2d(y) if y is not None else None
    if y2 is not None and (y2.shape != x2.shape or y2.stride(0) != x2.stride(0) or y2.dtype != x2.dtype):
        raise ValueError("y must match x in shape, pitch and dtype")
    c = cfg.c()
    _check(lib().bdr_quant_dequant_parent(C.addressof(c), k_parent, _ptr(x2), _ptr(y2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0),
                                          axis, _ptr(qsnr_sums), _stream(stream)), "bdr_quant_dequant_parent")
    return y


def bdr_gather_rows(cfg: Config, table: Planes, n_rows: int, idx: torch.Tensor, y: torch.Tensor, stream=None) -> torch.Tensor:
    """y[i, :] = decoded row idx[i] of a packed [n_rows, dim] table (axis-1 planes); idx int64 on the device."""
    assert idx.dtype == torch.int64 and idx.is_contiguous() and idx.is_cuda and y.dim() == 2 and y.shape[0] == idx.numel()
    c, p = cfg.c(), table.c()
    _check(lib().bdr_gather_rows(C.addressof(c), C.addressof(p), n_rows, y.shape[1], _ptr(idx), idx.numel(), _ptr(y), _dt(y),
                                 y.stride(0), _stream(stream)), "bdr_gather_rows")
    return y


def bdr_unpack(cfg: Config, planes: Planes, y: torch.Tensor, axis: int = 1, stream=None) -> torch.Tensor:
    y2 = _as2d(y)
    c, p = cfg.c(), planes.c()
    _check(lib().bdr_unpack(C.addressof(c), C.addressof(p), _ptr(y2), _dt(y2), y2.shape[0], y2.shape[1], y2.stride(0),
                            axis, _stream(stream)), "bdr_unpack")
    return y


def bdr_qsnr_workspace_bytes(n_cfgs: int) -> int:
    return int(lib().bdr_qsnr_workspace_bytes(int(n_cfgs)))


def bdr_qsnr(cfgs, x: torch.Tensor, out_db: torch.Tensor, workspace: torch.Tensor, axis: int = 1, stream=None):
    """QSNR in dB of x under every configuration of ``cfgs`` into out_db (float64, len(cfgs))."""
    x2 = _as2d(x)
    arr = (_Config * len(cfgs))(*[c.c() for c in cfgs])
    _check(lib().bdr_qsnr(C.addressof(arr), len(cfgs), _ptr(x2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0), axis,
                          _ptr(out_db), _ptr(workspace), workspace.numel() * workspace.element_size(),
                          _stream(stream)), "bdr_qsnr")
    return out_db


def bdr_qsnr_delayed(cfgs, x: torch.Tensor, amax_window: torch.Tensor, out_db: torch.Tensor, workspace: torch.Tensor,
                     axis: int = 1, stream=None):
    """bdr_qsnr with the FP32 kinds' first-level maximum taken from `amax_window` (float32 device tensor of earlier
    maxima) instead of from x."""
    assert amax_window.dtype == torch.float32 and amax_window.is_contiguous() and amax_window.is_cuda
    x2 = _as2d(x)
    arr = (_Config * len(cfgs))(*[c.c() for c in cfgs])
    _check(lib().bdr_qsnr_delayed(C.addressof(arr), len(cfgs), _ptr(x2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0), axis,
                                  _ptr(amax_window), amax_window.numel(), _ptr(out_db), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)), "bdr_qsnr_delayed")
    return out_db


def bdr_amax(x: torch.Tensor, amax: torch.Tensor, stream=None) -> torch.Tensor:
    """amax[0] = max(amax[0], max |x|); amax: one float32 on the device, zeroed by the caller."""
    assert amax.dtype == torch.float32 and amax.numel() == 1 and amax.is_cuda
    x2 = _as2d(x)
    _check(lib().bdr_amax(_ptr(x2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0), _ptr(amax), _stream(stream)), "bdr_amax")
    return amax


def bdr_tile_packing_efficiency(cfg: Config, tile_elems: int = 256, line_bytes: int = 64) -> float:
    c = cfg.c()
    return float(lib().bdr_tile_packing_efficiency(C.addressof(c), tile_elems, line_bytes))


def bdr_qsnr_static_max_cfgs() -> int:
    return int(lib().bdr_qsnr_static_max_cfgs())


def bdr_qsnr_static(cfgs, x: torch.Tensor, out_db: torch.Tensor, axis: int = 1, stream=None):
    """bdr_qsnr without a workspace argument: the scratch is built into the library, for callers that
    must not allocate device memory (see include/bdr.h).  At most bdr_qsnr_static_max_cfgs()
    configurations; calls that overlap on the GPU race on the shared scratch."""
    x2 = _as2d(x)
    arr = (_Config * len(cfgs))(*[c.c() for c in cfgs])
    _check(lib().bdr_qsnr_static(C.addressof(arr), len(cfgs), _ptr(x2), _dt(x2), x2.shape[0], x2.shape[1], x2.stride(0),
                                 axis, _ptr(out_db), _stream(stream)), "bdr_qsnr_static")
    return out_db


def mx_gemm(cfg_a: Config, a: Planes, cfg_b: Config, b: Planes, M: int, N: int, K: int, c: torch.Tensor, stream=None):
    """c[M,N] (float32) = deq(a)[M,K] @ deq(b)[N,K]^T from packed operands quantized along K."""
    ca, cb, pa, pb = cfg_a.c(), cfg_b.c(), a.c(), b.c()
    _check(lib().mx_gemm(C.addressof(ca), C.addressof(pa), C.addressof(cb), C.addressof(pb), M, N, K, _ptr(c),
                         c.stride(0), _stream(stream)), "mx_gemm")
    return c


def mx_gemm_hw(cfg_a: Config, a: Planes, cfg_b: Config, b: Planes, M: int, N: int, K: int, c: torch.Tensor, r: int = 64, f: int = 25,
               stream=None):
    """c[M,N] (float32) = the product as the dot-product pipeline of Section IV-B computes it (pass length r, f-bit frame)."""
    ca, cb, pa, pb = cfg_a.c(), cfg_b.c(), a.c(), b.c()
    _check(lib().mx_gemm_hw(C.addressof(ca), C.addressof(pa), C.addressof(cb), C.addressof(pb), M, N, K, r, f, _ptr(c),
                            c.stride(0), _stream(stream)), "mx_gemm_hw")
    return c


def mx_gemm_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().mx_gemm_workspace_bytes(M, N, K))


def mx_gemm_ws(cfg_a: Config, a: Planes, cfg_b: Config, b: Planes, M: int, N: int, K: int, c: torch.Tensor,
               workspace: torch.Tensor, stream=None):
    """mx_gemm in two phases: decode both operands once into `workspace` (uint8 device tensor of at least
    mx_gemm_workspace_bytes(M, N, K) bytes), then a TMA-fed tensor-core GEMM."""
    ca, cb, pa, pb = cfg_a.c(), cfg_b.c(), a.c(), b.c()
    _check(lib().mx_gemm_ws(C.addressof(ca), C.addressof(pa), C.addressof(cb), C.addressof(pb), M, N, K, _ptr(c),
                            c.stride(0), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "mx_gemm_ws")
    return c


def mx_gemm_f8_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().mx_gemm_f8_workspace_bytes(M, N, K))


def mx_gemm_f8(cfg_a: Config, a: Planes, cfg_b: Config, b: Planes, M: int, N: int, K: int, c: torch.Tensor,
               workspace: torch.Tensor, stream=None):
    """mx_gemm for MX4 / MX6 operands on the block-scaled 8-bit tensor-core path: exact re-encoding to E4M3 with
    one scale per 32 elements into `workspace` (at least mx_gemm_f8_workspace_bytes(M, N, K) bytes), then the GEMM."""
    ca, cb, pa, pb = cfg_a.c(), cfg_b.c(), a.c(), b.c()
    _check(lib().mx_gemm_f8(C.addressof(ca), C.addressof(pa), C.addressof(cb), C.addressof(pb), M, N, K, _ptr(c),
                            c.stride(0), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "mx_gemm_f8")
    return c


def bdr_reencode_e4m3(cfg: Config, planes: Planes, rows: int, K: int, out: torch.Tensor, scales: torch.Tensor,
                      inexact: torch.Tensor, stream=None):
    """Packed MX4 / MX6 operand -> E4M3 bytes `out` [rows, K], scale atoms `scales` (rows * K / 32 bytes) and the
    int32 flag `inexact` (set to 1, never cleared, if an element is not representable)."""
    cc, pp = cfg.c(), planes.c()
    _check(lib().bdr_reencode_e4m3(C.addressof(cc), C.addressof(pp), rows, K, _ptr(out), _ptr(scales), _ptr(inexact),
                                   _stream(stream)), "bdr_reencode_e4m3")
    return out, scales


def bdr_set_workspace(workspace: torch.Tensor | None):
    """Lends mx_gemm scratch memory on the current device (None takes it back).  The tensor must stay alive while lent."""
    if workspace is None:
        _check(lib().bdr_set_workspace(None, 0), "bdr_set_workspace")
    else:
        _check(lib().bdr_set_workspace(_ptr(workspace), workspace.numel() * workspace.element_size()), "bdr_set_workspace")


def mx_gemm_e4m3(a: torch.Tensor, scales_a: torch.Tensor, b: torch.Tensor, scales_b: torch.Tensor, M: int, N: int, K: int,
                 c: torch.Tensor, stream=None):
    """C = A B^T from operands re-encoded earlier with bdr_reencode_e4m3 (E4M3 bytes [rows, K] and scale atoms)."""
    _check(lib().mx_gemm_e4m3(_ptr(a), _ptr(scales_a), _ptr(b), _ptr(scales_b), M, N, K, _ptr(c), c.stride(0), _stream(stream)),
           "mx_gemm_e4m3")
    return c


def bdr_device_status() -> int:
    """Sticky per-device status of the kernels' bounded waits (0 = ok); synchronises."""
    return int(lib().bdr_device_status())


def bdr_device_status_reset() -> int:
    """Returns the sticky per-device status word and clears it; synchronises."""
    return int(lib().bdr_device_status_reset())


def bdr_qsnr_from_sums(sums: torch.Tensor, out_db: torch.Tensor, stream=None) -> torch.Tensor:
    """Eq. 3 in dB for every {error, signal} pair of `sums` ([n, 2] or [2] float64, device) into out_db ([n] float64)."""
    assert sums.dtype == torch.float64 and out_db.dtype == torch.float64 and sums.is_contiguous() and out_db.is_contiguous()
    n = sums.numel() // 2
    assert sums.numel() == 2 * n and out_db.numel() >= n
    _check(lib().bdr_qsnr_from_sums(C.c_void_p(sums.data_ptr()), n, C.c_void_p(out_db.data_ptr()), _stream(stream)),
           "bdr_qsnr_from_sums")
    return out_db


def bdr_selftest_bounded_wait(status_word) -> None:
    """Queues the kernel whose bounded wait runs out by design; it leaves BDR_ERR_TIMEOUT (-8) in `status_word`,
    one zeroed int32 on the device."""
    assert status_word.dtype == torch.int32 and status_word.numel() == 1 and status_word.is_cuda
    _check(lib().bdr_selftest_bounded_wait(C.c_void_p(status_word.data_ptr()), _stream(None)), "bdr_selftest_bounded_wait")


def bdr_selftest_host() -> int:
    """Host-only check of the per-device launch bookkeeping (0 = ok); makes no CUDA call."""
    return int(lib().bdr_selftest_host())


def mx_gemm_status() -> int:
    """0, or the (sticky) status of a launch whose bounded device-side wait ran out."""
    return int(lib().mx_gemm_status())
