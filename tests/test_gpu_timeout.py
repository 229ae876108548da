"""The bounded device-side waits really are bounded, and SQ_ERR_TIMEOUT reaches the host.

A test-only kernel (tests/probe/wait_probe.cu, its own shared object) calls the library's wait
helpers on an mbarrier nobody completes, with poll limits of a few hundred; each must give up and
raise the abort flag, a second waiter must be released by that flag, and the kernel records
SQ_ERR_TIMEOUT in the library's status word.  sq_device_status must report it once and then be
clean again, and the library must work normally afterwards.  Nothing faults, traps or hangs."""
import ctypes

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2512_05409_b200 as sq

pytestmark = pytest.mark.gpu


def test_expired_waits_report_timeout_once():
    from probe import build
    lib = ctypes.CDLL(build())
    lib.sqt_expire_waits.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.sqt_expire_waits.restype = ctypes.c_int
    assert sq.sq_device_status() == sq.SQ_OK
    word = sq.sq_device_status_word()
    assert word != 0
    report = torch.full((10,), -1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.sqt_expire_waits(ctypes.c_void_p(word), ctypes.c_void_p(report.data_ptr()), ctypes.c_void_p(stream)) == 0
    torch.cuda.synchronize()                       # the kernel returned: no wait was endless
    r = report.cpu().numpy()
    assert r[8] == 1                               # a completed phase is seen as complete
    assert np.array_equal(r[0:4], [1, 1, 1, 1])    # every helper gave up on the barrier nobody completes
    assert np.array_equal(r[4:8], [1, 1, 1, 1])    # ... and raised the abort flag
    assert r[9] == 1                               # which released the other waiting role
    assert sq.sq_device_status() == sq.SQ_ERR_TIMEOUT
    assert sq.sq_device_status() == sq.SQ_OK       # read-and-clear
    # the context is intact: a normal call still runs and is still right
    fmt = sq.make_format(64, 8, False)
    X = gen.activations(8, 256, seed=2, device="cuda")
    enc = sq.sq_encode(fmt, X)
    ref = oracle.encode(64, 8, gen.bf16_bits(X))
    assert np.array_equal(enc.dq4.cpu().numpy(), ref.dq4)
    assert sq.sq_device_status() == sq.SQ_OK
