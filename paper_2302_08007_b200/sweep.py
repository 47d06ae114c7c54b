"""The design-space sweep workload (Section IV): the list of configurations, in a fixed order.

Pure enumeration, no arithmetic of the method.  BDR grid: k1 in {8,16,32,64,128,256,1024},
k2 in {1,2,4,8}, d2 in {0,1,2}, m in {2..8}; d2 = 0 makes k2 irrelevant, so only one k2 is kept
there (441 distinct points).  Comparators: INT4 / INT8 and FP8 E4M3 / E5M2 under a per-tensor FP32
scale, and VSQ (INT4/6/8 elements, 4/6/8/10-bit integer sub-scale per 16 under an FP32 tensor
scale).  The MSFP-style points (k1 = 16, d2 = 0) are part of the grid already.
"""
from __future__ import annotations

from .binding import (Config, SCALE_FP32_FP, SCALE_FP32_INT, SCALE_FP32_VSQ, SCALE_POW2)

K1S = (8, 16, 32, 64, 128, 256, 1024)
K2S = (1, 2, 4, 8)
D2S = (0, 1, 2)
MS = (2, 3, 4, 5, 6, 7, 8)


def bdr_grid() -> list[tuple[str, Config]]:
    out = []
    for k1 in K1S:
        for k2 in K2S:
            for d2 in D2S:
                if d2 == 0 and k2 != K2S[0]:
                    continue
                for m in MS:
                    out.append(("bdr_k1=%d_k2=%d_d2=%d_m=%d" % (k1, k2, d2, m), Config(k1, 8, k2, d2, m, SCALE_POW2)))
    return out


def comparators() -> list[tuple[str, Config]]:
    out = [("int4", Config(0, 32, 1, 0, 3, SCALE_FP32_INT)), ("int8", Config(0, 32, 1, 0, 7, SCALE_FP32_INT)),
           ("fp8_e4m3", Config(0, 32, 1, 4, 3, SCALE_FP32_FP)), ("fp8_e5m2", Config(0, 32, 1, 5, 2, SCALE_FP32_FP))]
    for bits, m in ((4, 3), (6, 5), (8, 7)):
        for d2 in (4, 6, 8, 10):
            out.append(("vsq_int%d_d2=%d" % (bits, d2), Config(0, 32, 16, d2, m, SCALE_FP32_VSQ)))
    return out


def sweep_configs() -> list[tuple[str, Config]]:
    """457 named configurations: the BDR grid first, then the comparators."""
    return bdr_grid() + comparators()


def bits_per_element(cfg: Config) -> float:
    """Section III: (m + 1) + d1/k1 + d2/k2 (a per-tensor scale, k1 = 0, costs nothing per element)."""
    return (cfg.m + 1) + (cfg.d1 / cfg.k1 if cfg.k1 > 0 else 0.0) + (cfg.d2 / cfg.k2 if cfg.k2 > 0 else 0.0)


def pareto_frontier(points):
    """The QSNR-versus-cost frontier of Section IV-C from (name, cost, qsnr_db) triples: the points that no other
    point beats or equals on both axes (lower cost, higher QSNR), in order of rising cost.  Here the cost axis is
    bits per element divided by the tile packing efficiency; the paper's circuit-area factor is not reproducible."""
    best = []
    for name, cost, q in sorted(points, key=lambda p: (p[1], -p[2])):
        if q != q:
            continue
        if not best or q > best[-1][2]:
            best.append((name, cost, q))
    return best
