"""Bounded device-side waits: when the signal a wait is waiting for never comes, the kernel gives up
after its poll limit, records CONST_ERR_TIMEOUT, skips its stores and returns normally, and the
library keeps working afterwards.

The failure is made with the library's test hook, which withholds the signal (sort tiles do not publish
their digit counts; the tensor-core stage issues and commits nothing) and shortens the poll limit.
Nothing here faults or hangs: every wait involved has an iteration limit.
"""
import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from workloads import generators as gen
from workloads import ttmc3_workload, ttmc4_workload
from tests.gpu_util import assert_close, assert_csf_equal, build_csf, oracle, run_workload, to_dev

pytestmark = pytest.mark.gpu

TIMEOUT = 8


@pytest.fixture
def withheld():
    cb.const_debug_set(0, 200)          # polls before a wait gives up
    cb.const_debug_set(1, 1)            # withhold the signal
    try:
        yield
    finally:
        cb.const_debug_set(1, 0)
        cb.const_debug_set(0, 0)


def test_sort_lookback_times_out_and_recovers(withheld):
    rng = np.random.default_rng(3)
    op = gen._uniform_tensor((300, 1000, 777), 200_003, rng, "pm1", np.float32)      # 49 sort tiles
    with pytest.raises(cb.ConstError) as e:
        build_csf(op, (0, 1, 2))
    assert e.value.status == TIMEOUT
    cb.const_debug_set(1, 0)
    cb.const_debug_set(0, 0)
    h = build_csf(op, (0, 1, 2))                                # the context is intact
    assert_csf_equal(h, op, (0, 1, 2))


@pytest.mark.parametrize("family", ["ttmc4", "ttmc3"])
def test_tensor_stage_wait_times_out_and_recovers(family):
    if family == "ttmc4":
        w = ttmc4_workload((300, 40, 30, 50), 80_000, 8, slice_s=1.0, value="pm1", config_id=3)
    else:
        w = ttmc3_workload((500, 300, 700), 120_000, 16, slice_s=1.1, inner_s=0.9, value="unit", config_id=2)
    dtype = cb.F32
    handles = {n: build_csf(op, w.mode_orders[n]) for n, op in w.sparse.items()}
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, dtype)
    cb.const_plan_set_tensor_stage(plan, True)
    operands = dict(handles)
    operands.update({n: to_dev(a) for n, a in w.dense.items()})
    out = torch.full(w.out_shape, float("nan"), dtype=torch.float32, device="cuda")
    cb.const_debug_set(0, 50)
    cb.const_debug_set(1, 1)
    try:
        cb.const_execute(plan, operands, out)
        assert cb.const_last_device_status(plan) == TIMEOUT
    finally:
        cb.const_debug_set(1, 0)
        cb.const_debug_set(0, 0)
    got = out.cpu().numpy()
    assert np.all(np.isfinite(got))                             # zeroed before the nest; blocks that gave up stored nothing
    # a fresh plan on the same handles runs normally afterwards
    out2, _ = run_workload(w, handles=handles, tensor_stage=True)
    S, A = oracle(w)
    assert_close(out2, S, A, w.dtype)


def test_hook_argument_checks():
    with pytest.raises(cb.ConstError):
        cb.const_debug_set(7, 1)
    with pytest.raises(cb.ConstError):
        cb.const_debug_set(0, -1)
