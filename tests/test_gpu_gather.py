"""GPU parity of bdr_gather_rows: rows of a packed embedding table selected by device-side indices and decoded
(Section V, inferencing: embedding tables kept in MX format).  Expected values: the oracle's quantize-dequantize of the
table, indexed on the host."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", [bdr.MX4, bdr.MX6, bdr.MX9, bdr.Config(32, 8, 4, 2, 5), bdr.Config(8, 8, 1, 0, 3)], ids=str)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gathered_rows_equal_the_oracles_dequantized_table_rows(cfg, dtype):
    rng = np.random.default_rng(51)
    for n_rows, dim, n_idx, ld in ((1000, 128, 4096, None), (37, 100, 64, 104), (5, 16, 1, None), (300, 96, 777, 104), (64, 1024, 50, None)):
        table = H.make_input("laplace_outliers", n_rows, dim, dtype, seed=n_rows)
        planes = bdr.alloc_planes(cfg, n_rows, dim, 1)
        bdr.bdr_pack(cfg, H.host_to_device(table, dtype), planes, axis=1)
        want = orc.quant_dequant(H.to_orc(cfg), table, axis=1)[0]
        idx = rng.integers(0, n_rows, n_idx)                    # with repeats
        idx[0], idx[-1] = n_rows - 1, 0
        out = H.host_to_device(np.zeros((n_idx, dim), dtype=np.float32), dtype, ld)
        bdr.bdr_gather_rows(cfg, planes, n_rows, torch.from_numpy(idx).cuda(), out)
        torch.cuda.synchronize()
        H.assert_bits_equal(H.device_to_host_f32(out), want[idx], "%s %s %dx%d" % (cfg, dtype, n_rows, dim))
    assert bdr.bdr_device_status() == 0


def test_an_index_outside_the_table_is_reported_and_poisons_only_its_row():
    cfg = bdr.MX6
    table = H.make_input("normal", 64, 64, "f32", seed=52)
    planes = bdr.alloc_planes(cfg, 64, 64, 1)
    bdr.bdr_pack(cfg, H.host_to_device(table, "f32"), planes, axis=1)
    want = orc.quant_dequant(orc.MX6, table, axis=1)[0]
    idx = torch.tensor([3, 64, 0, -1, 63], dtype=torch.int64, device="cuda")
    out = torch.zeros((5, 64), dtype=torch.float32, device="cuda")
    assert bdr.bdr_device_status() == 0
    bdr.bdr_gather_rows(cfg, planes, 64, idx, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.isnan(got[1]).all() and np.isnan(got[3]).all()
    H.assert_bits_equal(got[[0, 2, 4]], want[[3, 0, 63]])
    assert bdr.bdr_device_status() == -5 and bdr.bdr_device_status_reset() == -5     # sticky until it is reset
    assert bdr.bdr_device_status() == 0
    with pytest.raises(bdr.BdrError) as e:                   # host-side checks
        bdr.bdr_gather_rows(cfg, planes, 64, idx, torch.zeros((5, 128), dtype=torch.float32, device="cuda"))   # planes too short for dim
    assert e.value.status == -5
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_lookup_of_rows_with_tiny_huge_and_nonfinite_blocks(dtype):
    # blocks outside the exponent range of the packed arithmetic (and Inf/NaN blocks) take the out-of-line decoder
    for name, cfg in (("MX4", bdr.MX4), ("MX6", bdr.MX6), ("MX9", bdr.MX9)):
        table = np.concatenate([H.make_input(k, 32, 128, dtype, seed=53) for k in ("tiny", "huge", "edge", "normal")])
        table[100, 40] = np.inf
        planes = bdr.alloc_planes(cfg, 128, 128, 1)
        bdr.bdr_pack(cfg, H.host_to_device(table, dtype), planes, axis=1)
        want = orc.quant_dequant(H.to_orc(cfg), table, axis=1)[0]
        idx = np.random.default_rng(54).permutation(128)
        out = H.host_to_device(np.zeros((128, 128), dtype=np.float32), dtype)
        bdr.bdr_gather_rows(cfg, planes, 128, torch.from_numpy(idx).cuda(), out)
        torch.cuda.synchronize()
        got = H.device_to_host_f32(out)
        nan = np.isnan(want[idx])
        assert np.array_equal(np.isnan(got), nan) and nan.any()
        H.assert_bits_equal(got[~nan], want[idx][~nan], "%s %s" % (name, dtype))
    assert bdr.bdr_device_status() == 0
