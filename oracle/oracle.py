"""ctypes loader for the CPU oracle (``bdr_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's
CPU-baseline leg.  The product package never imports this module, and this module imports nothing
from the product package.  All arithmetic lives in the C++ file; this file only marshals numpy
arrays.  Arrays are fp32 on this side: bf16 tensors are widened exactly by the caller.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bdr_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle_bdr.so")

POW2, FP32_INT, FP32_FP, FP32_VSQ = 0, 1, 2, 3
RNE, RNA = 0, 1


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("k1", "d1", "k2", "d2", "m", "scale_kind", "rounding")]


@dataclass(frozen=True)
class Config:
    """The BDR parameter tuple of Section III plus scale kind and tie rule."""
    k1: int
    d1: int
    k2: int
    d2: int
    m: int
    scale_kind: int = POW2
    rounding: int = RNE

    def c(self) -> _Cfg:
        return _Cfg(self.k1, self.d1, self.k2, self.d2, self.m, self.scale_kind, self.rounding)


# Table II presets
MX9 = Config(16, 8, 2, 1, 7)
MX6 = Config(16, 8, 2, 1, 4)
MX4 = Config(16, 8, 2, 1, 2)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", _SRC,
                               "-o", _LIB, "-lpthread"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_bits_per_element.restype = C.c_double
        _lib.orc_theorem1_bound_db.restype = C.c_double
        _lib.orc_theorem1_bound_db.argtypes = [C.c_void_p, C.c_int64]
        _lib.orc_qsnr_db.restype = C.c_double
        _lib.orc_qsnr_db.argtypes = [C.c_double, C.c_double]
        _lib.orc_tile_packing_efficiency.restype = C.c_double
        _lib.orc_tile_packing_efficiency.argtypes = [C.c_void_p, C.c_int64, C.c_int64]
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def bits_per_element(cfg: Config) -> float:
    c = cfg.c()
    return lib().orc_bits_per_element(C.byref(c))


def theorem1_bound_db(cfg: Config, n: int) -> float:
    c = cfg.c()
    return lib().orc_theorem1_bound_db(C.cast(C.byref(c), C.c_void_p), n)


def qsnr_db(err2: float, sig2: float) -> float:
    return lib().orc_qsnr_db(float(err2), float(sig2))


def config_check(cfg: Config) -> int:
    c = cfg.c()
    return lib().orc_config_check(C.byref(c))


def tile_packing_efficiency(cfg: Config, tile_elems: int = 256, line_bytes: int = 64) -> float:
    c = cfg.c()
    return lib().orc_tile_packing_efficiency(C.cast(C.byref(c), C.c_void_p), tile_elems, line_bytes)


def quant_dequant(cfg: Config, x, axis: int = 1, alt: bool = False, nthreads: int = 1, amax: float | None = None):
    """Returns (y fp32 with x's 2-D shape, (sum_err2, sum_sig2)).  amax: the first-level maximum of the FP32-scaled
    kinds when it comes from elsewhere (a window of past tensors) instead of from x itself."""
    x = _f32(x)
    x2 = x.reshape(1, -1) if x.ndim == 1 else x
    rows, cols = x2.shape
    y = np.empty_like(x2)
    sums = np.zeros(2, dtype=np.float64)
    c = cfg.c()
    if amax is not None:
        rc = lib().orc_quant_dequant_scaled(C.byref(c), _p(x2), _p(y), _i64(rows), _i64(cols), _i64(cols), C.c_int(axis),
                                            _p(sums), C.c_float(float(amax)), C.c_int(nthreads))
    else:
        rc = lib().orc_quant_dequant_mt(C.byref(c), _p(x2), _p(y), _i64(rows), _i64(cols), _i64(cols), C.c_int(axis),
                                            _p(sums), C.c_int(int(alt)), C.c_int(nthreads))
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return y.reshape(x.shape), (float(sums[0]), float(sums[1]))


def qsnr(cfg: Config, x, axis: int = 1, nthreads: int = 1, amax: float | None = None) -> float:
    _, (e2, s2) = quant_dequant(cfg, x, axis, nthreads=nthreads, amax=amax)
    return qsnr_db(e2, s2)


def encode(cfg: Config, x, axis: int = 1):
    """Unpacked fields: F [nlines, nblocks] u8, tau [nlines, nblocks*k1/k2] u8, code [nlines, nblocks*k1] u16."""
    x = _f32(x)
    x2 = x.reshape(1, -1) if x.ndim == 1 else x
    rows, cols = x2.shape
    nlines, length = (rows, cols) if axis == 1 else (cols, rows)
    nb = (length + cfg.k1 - 1) // cfg.k1
    F = np.zeros((nlines, nb), dtype=np.uint8)
    tau = np.zeros((nlines, nb * (cfg.k1 // cfg.k2)), dtype=np.uint8)
    code = np.zeros((nlines, nb * cfg.k1), dtype=np.uint16)
    c = cfg.c()
    rc = lib().orc_encode(C.byref(c), _p(x2), _i64(rows), _i64(cols), _i64(cols), C.c_int(axis), _p(F), _p(tau),
                          _p(code))
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return F, tau, code


def packed_sizes(cfg: Config, rows: int, cols: int, axis: int = 1):
    ld = (C.c_int64 * 3)()
    nbytes = (C.c_int64 * 3)()
    c = cfg.c()
    rc = lib().orc_packed_sizes(C.byref(c), _i64(rows), _i64(cols), C.c_int(axis), ld, nbytes)
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return list(ld), list(nbytes)


def pack(cfg: Config, x, axis: int = 1):
    """Returns (exps, micro, elems) as uint8 arrays of shape [nlines, ld_*] with default pitches."""
    x = _f32(x)
    x2 = x.reshape(1, -1) if x.ndim == 1 else x
    rows, cols = x2.shape
    ld, _ = packed_sizes(cfg, rows, cols, axis)
    nlines = rows if axis == 1 else cols
    planes = [np.zeros((nlines, max(l, 0)), dtype=np.uint8) for l in ld]
    c = cfg.c()
    rc = lib().orc_pack(C.byref(c), _p(x2), _i64(rows), _i64(cols), _i64(cols), C.c_int(axis), _p(planes[0]),
                        _p(planes[1]), _p(planes[2]), _i64(ld[0]), _i64(ld[1]), _i64(ld[2]))
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return tuple(planes)


def unpack(cfg: Config, planes, rows: int, cols: int, axis: int = 1):
    exps, micro, elems = [np.ascontiguousarray(p, dtype=np.uint8) for p in planes]
    y = np.zeros((rows, cols), dtype=np.float32)
    c = cfg.c()
    rc = lib().orc_unpack(C.byref(c), _p(exps), _p(micro), _p(elems), _i64(exps.shape[1]), _i64(micro.shape[1]),
                          _i64(elems.shape[1]), _p(y), _i64(rows), _i64(cols), _i64(cols), C.c_int(axis))
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return y


def minifloat_round(x, ebits: int, mbits: int, rounding: int = RNE):
    x = _f32(x)
    out = np.empty_like(x)
    lib().orc_minifloat_round(_p(x), _p(out), _i64(x.size), C.c_int(ebits), C.c_int(mbits), C.c_int(rounding))
    return out


def gemm_nt_f64(a, b, nthreads: int = 1):
    """C = A @ B.T in fp64 from fp32 operands A [M,K], B [N,K]."""
    a, b = _f32(a), _f32(b)
    M, K = a.shape
    N = b.shape[0]
    c = np.empty((M, N), dtype=np.float64)
    lib().orc_gemm_nt_f64(_p(a), _p(b), _i64(M), _i64(N), _i64(K), _p(c), C.c_int(nthreads))
    return c


def gemm_nt_f64_sampled(a, b, ri, ci):
    a, b = _f32(a), _f32(b)
    ri = np.ascontiguousarray(ri, dtype=np.int64)
    ci = np.ascontiguousarray(ci, dtype=np.int64)
    out = np.empty(ri.size, dtype=np.float64)
    lib().orc_gemm_nt_f64_sampled(_p(a), _p(b), _i64(a.shape[1]), _p(ri), _p(ci), _i64(ri.size), _p(out))
    return out


def gemm_hw(cfg_a: Config, a, cfg_b: Config, b, r: int = 64, f: int = 25):
    """C = A B^T [M, N] fp32 as the dot-product pipeline of Section IV-B computes it (pass length r, f-bit fixed-point
    reduction) from the raw fp32 operands A [M, K], B [N, K], which are quantized along K first."""
    a, b = _f32(a), _f32(b)
    M, K = a.shape
    N = b.shape[0]
    assert b.shape[1] == K
    c = np.empty((M, N), dtype=np.float32)
    ca, cb = cfg_a.c(), cfg_b.c()
    rc = lib().orc_gemm_hw(C.byref(ca), _p(a), _i64(M), C.byref(cb), _p(b), _i64(N), _i64(K), C.c_int(r), C.c_int(f), _p(c))
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return c


def quant_dequant_parent(cfg: Config, k_parent: int, x, axis: int = 1):
    """Three-level scaling: an FP32 parent scale per k_parent elements of a line above the two-level quantizer.
    Returns (y fp32, (sum_err2, sum_sig2))."""
    x = _f32(x)
    x2 = x.reshape(1, -1) if x.ndim == 1 else x
    rows, cols = x2.shape
    y = np.empty_like(x2)
    sums = np.zeros(2, dtype=np.float64)
    c = cfg.c()
    rc = lib().orc_quant_dequant_parent(C.byref(c), _i64(k_parent), _p(x2), _p(y), _i64(rows), _i64(cols), _i64(cols), C.c_int(axis),
                                        _p(sums))
    if rc != 0:
        raise ValueError("oracle rejected the configuration or arguments")
    return y.reshape(x.shape), (float(sums[0]), float(sums[1]))
