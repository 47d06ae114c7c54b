"""Failure handling of the library on the GPU, exercised without faulting, trapping or hanging it."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2302_08007_b200 import binding as bdr
from paper_2302_08007_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # The streaming kernels wait for their bulk copies with a bounded number of polls and report a wait that
    # gives up through a status word.  Here a one-warp kernel waits, with that same wait cut down to a few hundred
    # polls, on a barrier that nothing completes: the wait must run out, BDR_ERR_TIMEOUT must appear in the word
    # handed in, the library's own sticky words must stay clean, and ordinary calls must keep working.
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    bdr.bdr_selftest_bounded_wait(word)
    torch.cuda.synchronize()
    assert int(word.item()) == -8 and bdr.strerror(-8) == "bounded device-side wait ran out"
    assert bdr.bdr_device_status() == 0 and bdr.mx_gemm_status() == 0
    # a second run does not overwrite a status that is already set (first failure wins), and a fresh word is set again
    bdr.bdr_selftest_bounded_wait(word)
    word2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    bdr.bdr_selftest_bounded_wait(word2)
    torch.cuda.synchronize()
    assert int(word.item()) == -8 and int(word2.item()) == -8
    # the next ordinary call: bf16 MX6 row quantize-dequantize (a bulk-copy kernel with bounded waits) against the oracle
    x = H.make_input("laplace_outliers", 64, 4096, "bf16", seed=21)
    xd = H.host_to_device(x, "bf16")
    y = torch.empty_like(xd)
    sums = torch.zeros(2, dtype=torch.float64, device="cuda")
    bdr.bdr_quant_dequant(bdr.MX6, xd, y, axis=1, qsnr_sums=sums)
    torch.cuda.synchronize()
    want, ref_sums = orc.quant_dequant(orc.MX6, x, axis=1)
    H.assert_bits_equal(H.device_to_host_f32(y), want, "after the timeout self-test")
    H.assert_qsnr_close(sums.cpu().numpy(), ref_sums)
    assert bdr.bdr_device_status() == 0


def test_null_and_misaligned_status_words_are_refused_on_the_host():
    L = bdr.lib()
    assert L.bdr_selftest_bounded_wait(None, None) == -1
    assert L.bdr_selftest_bounded_wait(258, None) == -4
    torch.cuda.synchronize()


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs a second GPU in the same process")
def test_kernel_attributes_are_set_on_every_device_the_process_uses():
    # Kernels that need more than 48 KB of dynamic shared memory have that limit raised per device.  After using
    # device 0, the same entry points must work on device 1 (they failed with BDR_ERR_CUDA when the "already
    # set" flag was kept per process).
    x = H.make_input("laplace_outliers", 256, 2048, "bf16", seed=22)
    want, _ = orc.quant_dequant(orc.MX6, x, axis=1)
    want0, _ = orc.quant_dequant(orc.MX6, x, axis=0)
    for dev in (0, 1, 0):
        with torch.cuda.device(dev):
            xd = torch.from_numpy(x).to(torch.bfloat16).cuda()
            for axis, ref in ((1, want), (0, want0)):
                planes = bdr.alloc_planes(bdr.MX6, 256, 2048, axis)
                y, back = torch.empty_like(xd), torch.empty_like(xd)
                bdr.bdr_quant_dequant(bdr.MX6, xd, y, axis=axis)
                bdr.bdr_pack(bdr.MX6, xd, planes, axis=axis)
                bdr.bdr_unpack(bdr.MX6, planes, back, axis=axis)
                torch.cuda.synchronize()
                H.assert_bits_equal(H.device_to_host_f32(y), ref, "device %d axis %d" % (dev, axis))
                H.assert_bits_equal(H.device_to_host_f32(back), ref, "device %d axis %d unpack" % (dev, axis))
            assert bdr.bdr_device_status() == 0
