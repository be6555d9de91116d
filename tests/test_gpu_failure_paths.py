"""The failure-detection path of the kernels, exercised in the one form that harms nothing: a wait
with a short limit that runs out and returns.  Every device-side wait in the library is bounded;
a wait that gives up raises the CTA's abort flag, records a code in the device health word, and the
kernel drains and returns.  Here a tiny self-test kernel waits on a barrier nothing arrives on, with
a limit of a few milliseconds; the real GEMM, attention and reduction kernels are never stalled."""
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import _cabi, synth
from paper_2609_11356_b200.api import rg_selftest_bounded_wait
from tests._gpu_util import DEV, HW, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_reports_once_and_leaves_the_context_usable():
    assert rg.rg_device_status() == 0                            # healthy before
    counter = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    rg_selftest_bounded_wait(3_000_000, counter)                 # 3 ms
    t1.record()
    torch.cuda.synchronize()                                     # the launch returns
    ms = t0.elapsed_time(t1)
    assert 2.0 <= ms < 200.0, ms                                 # it waited out its limit, and not the 2 s default
    assert int(counter.item()) == 2                              # the waiter timed out, the second warp left through the flag
    code = _cabi.C.c_uint32(0)
    st = _cabi.load().rg_device_status(_cabi.C.byref(code))
    assert st == 8 and code.value == _cabi.RG_SELFTEST_WAIT_CODE  # RG_ERR_TIMEOUT with the recorded code
    assert rg.rg_device_status() == 0                            # read once, then clear
    # the context is intact: an ordinary GEMM afterwards is bit-correct
    A = synth.normal_bf16((70, 512), 1.0, 1); B = synth.normal_bf16((96, 512), 1.0, 2)
    assert_bits_equal(gpu_gemm(A, B, cuts=(256,), out_dtype=rgo.F32),
                      rgo.gemm(A, B, cuts=(256,), atom_model=HW, out_dtype=rgo.F32), "GEMM after the self-test")
    assert rg.rg_device_status() == 0


def test_limits_outside_the_allowed_range_launch_nothing():
    counter = torch.zeros(1, dtype=torch.int32, device=DEV)
    for bad in (0, 999, 10**9):
        with pytest.raises(rg.RgError) as ei:
            rg_selftest_bounded_wait(bad, counter)
        assert ei.value.status == 4
    torch.cuda.synchronize()
    assert int(counter.item()) == 0 and rg.rg_device_status() == 0
