"""The failure path of the bounded device waits, exercised without faulting anything: a kernel whose only CTA waits
for a barrier phase that nothing completes gives up after the configured limit, returns by itself, and the device
status word reports it once.  Index and timeout conditions are separate bits of that word."""
import time

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_is_reported_once():
    import paper_2412_14363_b200 as resq
    assert resq.resq_device_status() == resq.OK
    resq.resq_set_option(resq.OPT_WAIT_LIMIT_US, 1000)            # 1 ms
    try:
        t0 = time.perf_counter()
        resq.resq_selftest_wait_runs_out()
        st = resq.resq_device_status()                            # synchronizes the stream
        dt = time.perf_counter() - t0
    finally:
        resq.resq_set_option(resq.OPT_WAIT_LIMIT_US, 2_000_000)
    assert st == resq.ERR_TIMEOUT
    assert dt < 1.0                                               # the 1 ms limit applied, not the 2 s default
    assert resq.resq_device_status() == resq.OK                   # reading cleared it
    # the context is intact: an ordinary call still works and reports nothing
    x = torch.ones((4, 64), dtype=torch.bfloat16, device="cuda")
    x8 = torch.empty((4, 32), dtype=torch.int8, device="cuda")
    x4 = torch.empty((4, 16), dtype=torch.uint8, device="cuda")
    s8 = torch.empty(4, dtype=torch.float32, device="cuda")
    s4 = torch.empty(4, dtype=torch.float32, device="cuda")
    resq.resq_project_quantize(x, None, 32, x8, x4, s8, s4)
    assert resq.resq_device_status() == resq.OK
    assert (x8.cpu().numpy() == 127).all() and (x4.cpu().numpy() == 0x77).all()


def test_timeout_and_index_conditions_are_separate_bits():
    """An out-of-range cache slot (index condition) and a wait that runs out (timeout condition) in the same
    interval: the timeout is reported (it wins), and nothing is left behind for the next read."""
    import paper_2412_14363_b200 as resq
    from paper_2412_14363_b200 import kv
    cache = kv.KvCache(1, 1, 32)
    cache.data.zero_()
    wq = torch.zeros((128, 128), dtype=torch.int8, device="cuda")
    s_u = torch.ones(128, dtype=torch.float32, device="cuda")
    k = torch.zeros((1, 1, 128), dtype=torch.bfloat16, device="cuda")
    bad_pos = torch.tensor([32], dtype=torch.int32, device="cuda")      # capacity is 32: out of range, skipped
    seq = torch.zeros(1, dtype=torch.int32, device="cuda")
    kv.resq_kv_append(cache, k, k, seq, bad_pos, wq, s_u)
    assert resq.resq_device_status() == resq.ERR_INDEX
    kv.resq_kv_append(cache, k, k, seq, bad_pos, wq, s_u)
    resq.resq_set_option(resq.OPT_WAIT_LIMIT_US, 500)
    try:
        resq.resq_selftest_wait_runs_out()
        assert resq.resq_device_status() == resq.ERR_TIMEOUT
    finally:
        resq.resq_set_option(resq.OPT_WAIT_LIMIT_US, 2_000_000)
    assert resq.resq_device_status() == resq.OK
    assert not np.any(cache.data.cpu().numpy())
