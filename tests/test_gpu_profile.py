"""const_profile_enable / const_profile_read: the per-kernel event timing the benchmark's kernel table comes from."""
import pytest
import torch

import paper_2401_04836_b200 as cb
from workloads import make_config
from tests.gpu_util import run_workload

pytestmark = pytest.mark.gpu


def test_profile_lists_every_kernel_of_a_step_once_per_launch():
    w = make_config(1)                                            # order-3 TTMc, 200^3: 24 key bits = three 8-bit passes
    run_workload(w)                                               # warm-up outside the record
    cb.const_profile_enable(True)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    run_workload(w)
    t1.record()
    torch.cuda.synchronize()
    prof = cb.const_profile_read()
    assert prof["pack_hist"][0] == 1 and prof["csf_count"][0] == 1 and prof["csf_scatter"][0] == 1
    assert prof["rs_onesweep"][0] == 3
    assert prof["chain3_kernel"][0] == 1
    assert all(n >= 1 and ms > 0.0 for n, ms in prof.values())
    assert sum(ms for _, ms in prof.values()) <= t0.elapsed_time(t1)
    # enabling again clears the record; disabling stops it
    cb.const_profile_enable(True)
    assert cb.const_profile_read() == {}
    cb.const_profile_enable(False)
    run_workload(w)
    assert cb.const_profile_read() == {}
