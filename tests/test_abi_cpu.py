"""CPU-only checks of the boundary: the C-ABI library loads without a GPU, exports every symbol the
header declares, and its host-only entry points and argument validation behave as documented."""
import ctypes as C
import os
import re

import pytest

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "bdr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+char\s*\*|int64_t|int|double)\s+(\w+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_library_loads_and_exports_every_declared_symbol():
    names = _declared_functions()
    assert {"bdr_quant_dequant", "bdr_pack", "bdr_unpack", "bdr_qsnr", "mx_gemm", "bdr_packed_sizes",
            "bdr_strerror"} <= set(names)
    L = bdr.lib()
    for n in names:
        assert getattr(L, n) is not None, n
    assert set(bdr.EXPORTS) <= set(names)


def test_strerror_covers_every_status():
    seen = {bdr.strerror(s) for s in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert bdr.strerror(-99) == "unknown status"


@pytest.mark.parametrize("cfg", [bdr.MX4, bdr.MX6, bdr.MX9, bdr.Config(64, 8, 8, 2, 3), bdr.Config(16, 8, 1, 0, 7),
                                 bdr.Config(8, 8, 1, 3, 8)], ids=str)
def test_packed_sizes_agree_with_the_oracle_and_the_bits_formula(cfg):
    o = orc.Config(cfg.k1, cfg.d1, cfg.k2, cfg.d2, cfg.m)
    for rows, cols in ((1, 65536), (8192, 8192), (5, 200), (3, 17), (0, 64)):
        for axis in (0, 1):
            assert bdr.bdr_packed_sizes(cfg, rows, cols, axis) == orc.packed_sizes(o, rows, cols, axis)
    _, nbytes = bdr.bdr_packed_sizes(cfg, 4, 4096, 1)
    assert sum(nbytes) * 8 == orc.bits_per_element(o) * 4 * 4096


def test_validation_happens_on_the_host():
    L = bdr.lib()
    bad = bdr.Config(16, 8, 3, 1, 4).c()
    ok = bdr.MX6.c()
    dummy = C.c_void_p(256)       # never dereferenced: validation fails first
    assert L.bdr_quant_dequant(None, dummy, dummy, 0, 1, 16, 16, 1, None, None) == -1
    assert L.bdr_quant_dequant(C.addressof(bad), dummy, dummy, 0, 1, 16, 16, 1, None, None) == -2
    assert L.bdr_quant_dequant(C.addressof(ok), None, dummy, 0, 1, 16, 16, 1, None, None) == -1
    assert L.bdr_quant_dequant(C.addressof(ok), dummy, dummy, 0, 1, 16, 8, 1, None, None) == -5   # ld < cols
    assert L.bdr_quant_dequant(C.addressof(ok), dummy, dummy, 0, -1, 16, 16, 1, None, None) == -5
    assert L.bdr_quant_dequant(C.addressof(ok), dummy, dummy, 0, 1, 16, 16, 2, None, None) == -2   # axis
    assert L.bdr_quant_dequant(C.addressof(ok), C.c_void_p(258), dummy, 0, 1, 16, 16, 1, None, None) == -4
    fp8 = bdr.Config(0, 32, 1, 4, 3, bdr.SCALE_FP32_FP).c()
    assert L.bdr_quant_dequant(C.addressof(fp8), dummy, dummy, 0, 1, 16, 16, 1, None, None) == -3
    assert L.bdr_pack(C.addressof(ok), dummy, 0, 1, 16, 16, 1, None, None, None, None) == -1
    assert L.bdr_unpack(C.addressof(ok), None, dummy, 0, 1, 16, 16, 1, None) == -1
    with pytest.raises(bdr.BdrError):
        bdr.bdr_packed_sizes(bdr.Config(16, 8, 5, 1, 4), 4, 64)


def test_per_device_launch_bookkeeping():
    # kernel attributes are per device: the library keeps "set up" flags per device, not per process.  The
    # self-test drives that bookkeeping with fake set-up functions for devices 0, 1, 2 and 63 (no CUDA call).
    assert bdr.bdr_selftest_host() == 0


def test_tile_packing_efficiency_agrees_with_the_oracle():
    C_ = bdr.Config
    for cfg in (bdr.MX4, bdr.MX6, bdr.MX9, C_(16, 8, 1, 0, 3), C_(64, 8, 8, 2, 5), C_(0, 32, 1, 4, 3, bdr.SCALE_FP32_FP),
                C_(0, 32, 16, 6, 3, bdr.SCALE_FP32_VSQ)):
        o = orc.Config(cfg.k1, cfg.d1, cfg.k2, cfg.d2, cfg.m, cfg.scale_kind, cfg.rounding)
        for tile, line in ((256, 64), (100, 32), (16, 128), (1, 1)):
            assert bdr.bdr_tile_packing_efficiency(cfg, tile, line) == pytest.approx(orc.tile_packing_efficiency(o, tile, line), rel=1e-15)
    assert bdr.bdr_tile_packing_efficiency(bdr.MX9) == 0.9
    assert bdr.bdr_tile_packing_efficiency(bdr.MX9, 0, 64) < 0
