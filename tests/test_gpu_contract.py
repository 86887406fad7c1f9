"""Fused contraction kernels vs the fp64 oracle, element by element: |gpu - S| <= tol * sum|terms|."""
import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb
from workloads import (make_config, ttmc3_workload, ttmc4_workload, mttkrp_workload, network_workload)
from workloads import generators as gen
from tests.gpu_util import assert_close, build_csf, oracle, run_workload, to_dev

pytestmark = pytest.mark.gpu

# bin thresholds (light_max, heavy_max, chunk) that force every slice into one bin
ALL_LIGHT = (1 << 40, 1 << 41, 1 << 30)
ALL_HEAVY = (1, 1 << 40, 1 << 30)
ALL_GIANT = (1, 2, 700)
MIXED = (300, 3000, 1500)


def check(w, bins=None, tensor_stage=None):
    out, handles = run_workload(w, bins, tensor_stage=tensor_stage)
    S, A = oracle(w)
    return assert_close(out, S, A, w.dtype), handles


def test_config1_ttmc3_small():
    w = make_config(1)
    ratio, _ = check(w)
    assert ratio <= 1.0


@pytest.mark.parametrize("bins", [None, ALL_LIGHT, ALL_HEAVY, ALL_GIANT, MIXED])
@pytest.mark.parametrize("rank", [8, 16, 32])
def test_ttmc3_skewed_each_bin(rank, bins):
    w = ttmc3_workload((500, 300, 700), 120_000, rank, slice_s=1.1, inner_s=0.9, value="unit", config_id=2)
    _, handles = check(w, bins)
    c = cb.const_csf_bin_counts(handles["X"])
    if bins == ALL_LIGHT:
        assert c["heavy"] == c["giant"] == 0
    if bins == ALL_HEAVY:
        assert c["giant"] == 0 and c["heavy"] > 0
    if bins == ALL_GIANT:
        assert c["giant"] > 0 and c["items"] > c["giant"]


def test_ttmc3_mixed_ranks_and_long_fibres():
    w = ttmc3_workload((40, 30, 5000), 150_000, (8, 32), slice_s=1.0, inner_s=None, value="pm1", config_id=7)
    check(w)                                                   # ~125 nonzeros per fibre: the long-fibre path
    check(w, ALL_GIANT)
    w = ttmc3_workload((40, 30, 5000), 150_000, (32, 16), slice_s=1.0, inner_s=None, value="pm1", config_id=8)
    check(w, MIXED)


def test_ttmc3_other_mode_at_the_root():
    """Second TTMc of Sec. 5.3: the output is indexed by j, so the schedule stores X as (j,i,k)."""
    w = ttmc3_workload((60, 50, 40), 20_000, 16, config_id=9)
    X = w.sparse["X"]
    h = build_csf(X, (1, 0, 2))
    ext = {"i": 60, "j": 50, "k": 40, "x": 16, "z": 16}
    plan = cb.const_plan_create("B[j,x,z] = T[i,j,k] * A[i,x] * C[k,z]",
                                ["S[j,i,z] = T[i,j,k] * C[k,z]", "B[j,x,z] = S[j,i,z] * A[i,x]"],
                                {"T": (1, 0, 2)}, ["jikz", "jixz"], ext, cb.F32)
    A_fac = np.random.default_rng(0).standard_normal((60, 16)).astype(np.float32)
    out = torch.empty((50, 16, 16), device="cuda")
    cb.const_execute(plan, {"T": h, "A": to_dev(A_fac), "C": to_dev(w.dense["V"])}, out)
    from oracle import contract as oc
    S, A = oc.ttmc3([X.coords[1], X.coords[0], X.coords[2]], X.vals, A_fac, w.dense["V"], 50)
    assert_close(out.cpu().numpy(), S, A, np.float32)


@pytest.mark.parametrize("root", [0, 1, 2])
@pytest.mark.parametrize("family", ["mttkrp", "ttmc"])
def test_every_output_mode(family, root):
    """All three MTTKRPs (Sec. 5.2) and TTMcs (Sec. 5.3) of one tensor: the output is indexed by mode `root`,
    so the schedule stores the tensor with that mode at the CSF root and contracts the other two."""
    from oracle import contract as oc
    dims, rank = (70, 55, 45), 16
    w = ttmc3_workload(dims, 8_000, rank, slice_s=1.0, inner_s=None, value="pm1", config_id=11)
    X = w.sparse["X"]
    p, q = [m for m in range(3) if m != root]
    names = "ijk"
    r_, p_, q_ = names[root], names[p], names[q]
    rng = np.random.default_rng(5)
    Fp = rng.standard_normal((dims[p], rank)).astype(np.float32)
    Fq = rng.standard_normal((dims[q], rank)).astype(np.float32)
    ext = {"i": dims[0], "j": dims[1], "k": dims[2], "x": rank, "z": rank}
    h = build_csf(X, (root, p, q))
    coords = [X.coords[root], X.coords[p], X.coords[q]]
    if family == "mttkrp":
        plan = cb.const_plan_create(f"O[{r_},z] = X[i,j,k] * P[{p_},z] * Q[{q_},z]",
                                    [f"T[{r_},{p_},z] = X[i,j,k] * Q[{q_},z]", f"O[{r_},z] = T[{r_},{p_},z] * P[{p_},z]"],
                                    {"X": (root, p, q)}, [f"{r_}{p_}{q_}z", f"{r_}{p_}z"], ext, cb.F32)
        out = torch.full((dims[root], rank), float("nan"), device="cuda")
        S, A = oc.mttkrp3(coords, X.vals, Fp, Fq, dims[root])
    else:
        plan = cb.const_plan_create(f"O[{r_},x,z] = X[i,j,k] * P[{p_},x] * Q[{q_},z]",
                                    [f"T[{r_},{p_},z] = X[i,j,k] * Q[{q_},z]", f"O[{r_},x,z] = T[{r_},{p_},z] * P[{p_},x]"],
                                    {"X": (root, p, q)}, [f"{r_}{p_}{q_}z", f"{r_}{p_}xz"], ext, cb.F32)
        out = torch.full((dims[root], rank, rank), float("nan"), device="cuda")
        S, A = oc.ttmc3(coords, X.vals, Fp, Fq, dims[root])
    cb.const_execute(plan, {"X": h, "P": to_dev(Fp), "Q": to_dev(Fq)}, out)
    assert cb.const_last_device_status(plan) == 0
    assert_close(out.cpu().numpy(), S, A, np.float32)


@pytest.mark.parametrize("bins", [None, ALL_LIGHT, ALL_GIANT, MIXED])
@pytest.mark.parametrize("rank", [8, 16, 32])
def test_mttkrp_each_bin(rank, bins):
    w = mttkrp_workload((400, 350, 300), 100_000, rank, slice_s=1.2, value="unit", config_id=4)
    check(w, bins)


# order-4 TTMc: the per-slice stage Y_i = U_J^T Q_J runs on the tensor cores (split tf32 operands, the
# default at rank 8) or on the FMA pipes; both must meet the fp32 tolerance
@pytest.mark.parametrize("tensor_stage", [False, True])
@pytest.mark.parametrize("bins", [None, ALL_LIGHT, ALL_HEAVY, ALL_GIANT, MIXED])
def test_ttmc4_each_bin(bins, tensor_stage):
    w = ttmc4_workload((300, 40, 30, 50), 80_000, 8, slice_s=1.0, value="pm1", config_id=3)
    check(w, bins, tensor_stage=tensor_stage)


@pytest.mark.parametrize("tensor_stage", [False, True, None])
def test_ttmc4_sparse_like_the_benchmark(tensor_stage):
    w = make_config(3, scale=0.004)             # 200k nonzeros in 20000^4: every (i,j,k) fibre has one leaf
    check(w, tensor_stage=tensor_stage)
    w = ttmc4_workload((7, 5, 3, 4), 60, 8, slice_s=1.0, value="pm1", config_id=3)      # a handful of tiny slices
    check(w, tensor_stage=tensor_stage)


@pytest.mark.parametrize("tensor_stage", [False, True])
@pytest.mark.parametrize("bins", [None, ALL_LIGHT, ALL_HEAVY, ALL_GIANT, MIXED])
def test_ttmc3_rank16_tensor_stage_each_bin(bins, tensor_stage):
    # order-3 TTMc at rank 16 x 16: Y_i = T_J^T U_J on the tensor cores (split tf32 operands) or on the FMA pipes
    w = ttmc3_workload((500, 300, 700), 120_000, 16, slice_s=1.1, inner_s=0.9, value="unit", config_id=2)
    check(w, bins, tensor_stage=tensor_stage)
    w = ttmc3_workload((40, 30, 5000), 150_000, 16, slice_s=1.0, inner_s=None, value="pm1", config_id=7)   # long fibres
    check(w, bins, tensor_stage=tensor_stage)


def test_ttmc3_rank16_tensor_stage_tiny():
    w = ttmc3_workload((7, 5, 6), 40, 16, value="pm1", config_id=12)
    check(w, tensor_stage=True)
    check(make_config(2, scale=0.005), tensor_stage=True)


def test_tensor_stage_only_where_a_kernel_has_one():
    w = make_config(1)
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
    with pytest.raises(cb.ConstError):
        cb.const_plan_set_tensor_stage(plan, True)
    cb.const_plan_set_tensor_stage(plan, False)


def test_scaled_configs_2_and_4():
    check(make_config(2, scale=0.005))
    check(make_config(4, scale=0.003))


def test_network_small_and_scaled():
    check(network_workload(64, 16, 8, 0.25, config_id=5))
    check(network_workload(70, 13, 5, 0.4, config_id=6))        # extents that are not multiples of the tiles
    check(make_config(5, scale=0.25))


def test_atomics_run_to_run_within_tolerance():
    w = ttmc3_workload((50, 300, 700), 100_000, 16, slice_s=1.3, inner_s=0.9, value="unit", config_id=2)
    S, A = oracle(w)
    handles = None
    for _ in range(2):
        out, handles = run_workload(w, ALL_GIANT, handles)
        assert_close(out, S, A, w.dtype)


def test_empty_and_single_nonzero():
    S = gen.SparseOperand
    w = ttmc3_workload((6, 5, 4), 10, 8)
    w.sparse["X"] = S([np.zeros(0, np.int32)] * 3, np.zeros(0, np.float32), (6, 5, 4))
    out, _ = run_workload(w)
    assert np.all(out == 0)
    w.sparse["X"] = S([np.array([5], np.int32), np.array([4], np.int32), np.array([3], np.int32)],
                      np.array([2.0], np.float32), (6, 5, 4))
    out, _ = run_workload(w)
    expect = np.zeros((6, 8, 8)); expect[5] = 2.0 * np.outer(w.dense["U"][4], w.dense["V"][3])
    np.testing.assert_allclose(out, expect, rtol=1e-6)


def test_operand_validation():
    w = make_config(1)
    h = build_csf(w.sparse["X"], (0, 1, 2))
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, cb.F32)
    out = torch.empty(w.out_shape, device="cuda")
    U, V = to_dev(w.dense["U"]), to_dev(w.dense["V"])
    with pytest.raises(cb.ConstError):
        cb.const_execute(plan, {"X": h, "U": U}, out)                      # missing operand
    wrong = build_csf(w.sparse["X"], (1, 0, 2))
    with pytest.raises(cb.ConstError):
        cb.const_execute(plan, {"X": wrong, "U": U, "V": V}, out)          # CSF built with another mode order
    with pytest.raises(cb.ConstError):
        cb.const_execute(plan, {"X": U, "U": U, "V": V}, out)              # dense where CSF is expected
