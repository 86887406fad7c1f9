"""Several host threads inside the library at once, each on a stream of its own: const_csf_build and
const_execute are documented as safe for that (lazily created pools, per-device kernel attributes and the plan's
status word sit behind mutexes).  Every thread's CSF arrays and results are compared with the oracle."""
import threading

import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from workloads import mttkrp_workload, ttmc3_workload, ttmc4_workload
from tests.gpu_util import assert_close, assert_csf_equal, build_csf, oracle, to_dev

pytestmark = pytest.mark.gpu


def test_four_threads_build_and_execute_concurrently():
    workloads = [ttmc3_workload((600, 150, 160), 60_000, 16, slice_s=1.1, value="pm1", config_id=71),
                 ttmc3_workload((150, 200, 70), 45_000, 8, value="pm1", config_id=72),
                 mttkrp_workload((700, 160, 140), 70_000, 32, slice_s=1.2, value="unit", config_id=73),
                 ttmc4_workload((120, 30, 25, 20), 40_000, 8, slice_s=1.0, value="pm1", config_id=74)]
    expected = [oracle(w) for w in workloads]                     # on the CPU, before any thread starts
    errors = []
    start = threading.Barrier(len(workloads))

    def work(t):
        try:
            torch.cuda.set_device(0)
            w = workloads[t]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                dense = {n: to_dev(a) for n, a in w.dense.items()}
                plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
                start.wait()
                for _ in range(6):
                    X = build_csf(w.sparse["X"], w.mode_orders["X"])
                    out = torch.full(w.out_shape, float("nan"), dtype=torch.float32, device="cuda")
                    cb.const_execute(plan, dict(dense, X=X), out)
                    stream.synchronize()
                    assert cb.const_last_device_status(plan) == 0
                    assert_csf_equal(X, w.sparse["X"], w.mode_orders["X"])
                    assert_close(out.cpu().numpy(), expected[t][0], expected[t][1], np.float32)
        except BaseException as e:                                # reported by the main thread
            errors.append((t, repr(e)))
            start.abort()

    threads = [threading.Thread(target=work, args=(t,)) for t in range(len(workloads))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
