"""The bounded waits of the kernels, run out on purpose in the one safe form: a barrier nobody
arrives at and a counter nobody raises, in test-only kernels with nothing else in flight.  Each
wait must end by itself after its limit, record DDD_ERR_TIMEOUT in the status word and let the
kernel finish normally; the context must be usable afterwards."""
import ctypes

import pytest
import torch

from tests.cuda import build_probe

pytestmark = pytest.mark.gpu
DDD_ERR_TIMEOUT = -5


def _lib():
    lib = ctypes.CDLL(build_probe.build())
    vp = ctypes.c_void_p
    lib.probe_mbarrier_timeout.argtypes = [vp, vp, ctypes.c_double, vp]
    lib.probe_grid_timeout.argtypes = [vp, vp, vp, vp, ctypes.c_int, ctypes.c_double, vp]
    return lib


def test_mbarrier_wait_gives_up_after_its_limit_and_reports_it():
    lib = _lib()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.full((3,), -1, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert lib.probe_mbarrier_timeout(status.data_ptr(), result.data_ptr(), 1.0, st) == 0
    torch.cuda.synchronize()                          # the kernel ended by itself: no fault, no hang
    ok, abort_flag, waited_us = result.cpu().tolist()
    assert ok == 0 and abort_flag == 1
    assert int(status.item()) == DDD_ERR_TIMEOUT
    assert 900 <= waited_us < 100000, waited_us       # about the 1 ms limit, not the 2 s default
    # the context is still usable
    assert int((torch.arange(10, device="cuda") * 2).sum().item()) == 90


def test_grid_hand_over_gives_up_and_releases_the_other_blocks():
    lib = _lib()
    blocks = 8
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.full((blocks,), -1, dtype=torch.int32, device="cuda")
    counter = torch.zeros(1, dtype=torch.int32, device="cuda")
    abort_word = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert lib.probe_grid_timeout(status.data_ptr(), result.data_ptr(), counter.data_ptr(), abort_word.data_ptr(),
                                  blocks, 1.0, st) == 0
    torch.cuda.synchronize()
    assert result.cpu().tolist() == [0] * blocks      # every wait returned "gave up"
    assert int(status.item()) == DDD_ERR_TIMEOUT and int(abort_word.item()) == 1
    assert int(counter.item()) == 1
