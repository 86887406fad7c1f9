#!/usr/bin/env python
"""Benchmark of the whole hot path on seeded synthetic input.

One step = const_csf_build (COO -> CSF, including the load-balancing lists) followed by
const_execute (the fused contraction tree) on one batch.  Without --config all five benchmark
configurations are measured one after the other; the headline figures (`value`, `ms_per_step`,
`roofline`, `cpu_baseline`, `e2e`) are those of the large skewed order-3 TTMc (12 000 x 9 000 x 29 000,
77 M nonzeros, rank 16) and `per_config` holds the same set of figures for each configuration.
`value` is useful GFLOP/s of the fused schedule (2*R3*nnz + 2*R2*R3*fibres for TTMc) over the step
time with inputs resident in HBM; `e2e` is the same with host (pinned) buffers and the copies inside
the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--scale s] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the headline
configuration on its own GPU -- slices are independent, so there is no data-path collective -- and the
line reports the sum.  `--impl reference` times the CPU oracle on a bounded sample of the same workload
(rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

HEADLINE_CONFIG = 2
# nonzeros in the CPU-baseline sample of each configuration (about 2-5 s of oracle time on 16 cores)
ORACLE_SAMPLE_NNZ = {1: 20_000, 2: 20_000_000, 3: 3_000_000, 4: 40_000_000, 5: 250_000}

# DRAM bytes per nonzero and launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures
# summarised under profiles/; the kernels stream their inputs once, so the traffic of a full-size launch is this
# figure times its nonzero count.  Only valid for the kernel version the capture was taken from: an entry is
# dropped (traffic null) when its kernel changes.
NCU_TRAFFIC_BYTES_PER_NNZ = {("ttmc3", "rs_onesweep"): 527.0e6 / 23.1e6, ("ttmc3", "chain3_kernel"): 234.9e6 / 23.1e6}


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------------
# algorithmic work of one step (flops of the fused schedule, compulsory bytes)
# ------------------------------------------------------------------------------------------------
def algorithmic_work(w, level_sizes):
    """(useful flops, compulsory bytes) of const_execute; level_sizes: {sparse name: [n_0, ..., n_leaf]}."""
    fam = w.family
    out_bytes = int(np.prod(w.out_shape)) * w.dtype.itemsize
    fac_bytes = sum(a.nbytes for a in w.dense.values())
    if fam == "network":
        nu, nw = level_sizes["U"], level_sizes["W"]
        n_l, n_i = w.extents["l"], w.extents["i"]
        flops = 2 * n_l * nu[2] + 2 * n_i * nw[2]
        csf_bytes = sum(12 * n[2] + 8 * n[1] + 8 * n[0] for n in (nu, nw))
        return flops, csf_bytes + out_bytes + fac_bytes
    n = level_sizes["X"]
    nnz = n[-1]
    if fam == "ttmc3":
        r2, r3 = w.extents["a"], w.extents["b"]
        flops = 2 * r3 * nnz + 2 * r2 * r3 * n[1]
    elif fam == "mttkrp":
        r = w.extents["r"]
        flops = 2 * r * nnz + 2 * r * n[1]
    else:  # ttmc4
        r = w.extents["a"]
        flops = 2 * r * nnz + 2 * r * r * n[2] + 2 * r * r * r * n[1]
    csf_bytes = 8 * nnz + sum(8 * x for x in n[:-1])      # leaf: crd + value; inner nodes: crd + pos
    return flops, csf_bytes + out_bytes + fac_bytes


def build_bytes(w, level_sizes):
    """Compulsory bytes of const_csf_build: the COO arrays read once, the CSF arrays written once."""
    total = 0
    for name, op in w.sparse.items():
        n = level_sizes[name]
        v = op.vals.dtype.itemsize
        total += op.nnz * (4 * len(op.dims) + v) + n[-1] * (4 + v) + sum(8 * x for x in n[:-1])
    return total


def tensor_stage_flops(w, level_sizes):
    """Flops of the dense per-slice stage (the last contraction of a TTMc summed over a slice's fibres)."""
    n = level_sizes["X"]
    if w.family == "ttmc4":
        r = w.extents["a"]
        return 2 * r * r * r * n[1]
    if w.family == "ttmc3":
        return 2 * w.extents["a"] * w.extents["b"] * n[1]
    return 0


def sample_rows_for_oracle(w, target_nnz, seed=0):
    """A seeded subset of output rows whose slices hold about target_nnz nonzeros."""
    X = w.sparse["U" if w.family == "network" else "X"]
    rng = np.random.default_rng(seed)
    sizes = np.bincount(X.coords[0], minlength=X.dims[0])
    order = rng.permutation(X.dims[0])
    csum = np.cumsum(sizes[order])
    k = int(np.searchsorted(csum, target_nnz)) + 1
    return np.sort(order[:k])


def time_oracle(w, target_nnz):
    """The oracle, as it stands, on a seeded row sample; returns (cpu_baseline dict, seconds, rows, S, A)."""
    from oracle import contract as oc
    from oracle import workload as ow
    from workloads import row_sample
    rows = sample_rows_for_oracle(w, target_nnz)
    key = "U" if w.family == "network" else "X"
    sub = row_sample(w.sparse[key], rows)
    t0 = time.perf_counter()
    S, A = ow.evaluate(w, rows)
    dt = time.perf_counter() - t0
    # flops of the fused schedule restricted to the sampled slices
    if w.family == "network":
        W = w.sparse["W"]
        flops = 2 * w.extents["l"] * sub.nnz + 2 * len(rows) * W.nnz
    else:
        coords = sub.coords
        f1 = np.unique(coords[0].astype(np.int64) * sub.dims[1] + coords[1]).size
        if w.family == "ttmc4":
            f2 = np.unique((coords[0].astype(np.int64) * sub.dims[1] + coords[1]) * sub.dims[2] + coords[2]).size
            r = w.extents["a"]
            flops = 2 * r * sub.nnz + 2 * r * r * f2 + 2 * r * r * r * f1
        elif w.family == "ttmc3":
            flops = 2 * w.extents["b"] * sub.nnz + 2 * w.extents["a"] * w.extents["b"] * f1
        else:
            flops = 2 * w.extents["r"] * (sub.nnz + f1)
    return ({"value": flops / dt / 1e9, "unit": "GFLOP/s", "cores": oc.num_threads(), "kind": "oracle",
             "sample": f"{len(rows)} seeded output rows holding {sub.nnz} nonzeros, {dt:.2f} s"}, dt, rows, S, A)


def aggregate_over_ranks(ms_per_step, work, dist=None, device="cpu"):
    """Whole-job figures for independent replicas (one per rank, no data-path collective):
    the step time is the maximum over ranks, the work done is the sum over ranks."""
    if dist is None:
        return float(ms_per_step), float(work)
    import torch
    t = torch.tensor([float(ms_per_step)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    f = torch.tensor([float(work)], device=device, dtype=torch.float64)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t.item()), float(f.item())


def _generate(args):
    """Pool worker: draws one configuration (numpy only; never touches the GPU)."""
    config_id, scale, seed = args
    from workloads import make_config
    t0 = time.perf_counter()
    w = make_config(config_id, scale=scale, seed=seed)
    return config_id, w, time.perf_counter() - t0


# ------------------------------------------------------------------------------------------------
# clocks sampler
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    interval_ms = 20

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.interval_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([time.monotonic()] + [x.strip() for x in line.split(",")])

    def stop(self, t0=None, t1=None):
        """Ends the sampling; the summary covers the samples taken between the monotonic times t0 and t1
        (all of them when no window is given, or when the window holds none)."""
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        window = [r[1:] for r in self.rows if t0 is not None and t0 <= r[0] <= t1]
        self.rows = window if window else [r[1:] for r in self.rows]
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


FUSED_KERNELS = {"chain3_kernel", "chain3_tc_kernel", "ttmc4_kernel", "ttmc4_tc_kernel", "network_kernel",
                 "tree_kernel"}


def measure_machine_peaks(cb, local_rank):
    """Register-only FMA peaks (fp32, fp64) and the tf32 tensor-pipe peak, with the SM clock seen meanwhile."""
    sampler = ClockSampler(local_rank)
    sampler.start()
    out = {}
    for name, kind in (("fp32_fma_tflops", cb.BENCH_FP32_FMA), ("fp64_fma_tflops", cb.BENCH_FP64_FMA),
                       ("fp64_mma_tflops", cb.BENCH_FP64_MMA), ("tf32_mma_tflops", cb.BENCH_TF32_MMA)):
        best = 0.0
        for _ in range(3):
            ms, work = cb.const_microbench(kind, repeats=20 if kind != cb.BENCH_TF32_MMA else 5)
            best = max(best, work / (ms * 1e-3) / 1e12)
        out[name] = best
    clocks = sampler.stop()
    out["sm_mhz_during"] = clocks["sm_mhz"]
    out["how"] = ("const_microbench: 8 independent FMA chains per thread on 8 x 256 threads per SM; tcgen05.mma "
                  "kind::tf32 M128 N256 K8 from shared memory, one block per SM; mma.sync m8n8k4 f64 from registers; best of 3")
    return out


def measure_config(cb, torch, w, config_id, args, peaks, hbm_peak, peak_kind, rank, dist, want_oracle):
    """All figures of one configuration; the caller composes the JSON line from them."""
    dtype = cb.F32 if w.dtype == np.float32 else cb.F64
    tdtype = torch.float32 if dtype == cb.F32 else torch.float64
    steps = args.steps

    # host (pinned) and device copies of every input
    host = {}
    for name, op in w.sparse.items():
        host[name] = ([torch.from_numpy(np.ascontiguousarray(c)).pin_memory() for c in op.coords],
                      torch.from_numpy(np.ascontiguousarray(op.vals)).pin_memory())
    host_dense = {n: torch.from_numpy(a).pin_memory() for n, a in w.dense.items()}
    dev = {n: ([c.cuda() for c in cs], v.cuda()) for n, (cs, v) in host.items()}
    dev_dense = {n: a.cuda() for n, a in host_dense.items()}
    out = torch.empty(w.out_shape, dtype=tdtype, device="cuda")
    out_host = torch.empty(w.out_shape, dtype=tdtype).pin_memory()
    plan = cb.const_plan_create(w.expression, w.tree, w.mode_orders, w.loop_orders, w.extents, dtype)
    if args.tensor_stage >= 0 and w.family in ("ttmc4", "ttmc3"):
        cb.const_plan_set_tensor_stage(plan, bool(args.tensor_stage))
    if args.generic_executor:
        cb.const_plan_set_generic_executor(plan, True)
    stream = torch.cuda.current_stream()
    bins_override = tuple(int(x) for x in args.bins.split(",")) if args.bins else None

    def build_all(src):
        hs = {n: cb.const_csf_build(cs, v, w.sparse[n].dims, w.mode_orders[n]) for n, (cs, v) in src.items()}
        if bins_override:
            for h in hs.values():
                cb.const_csf_set_bins(h, *bins_override)
        return hs

    def step(src, dense):
        handles = build_all(src)
        ops = dict(handles)
        ops.update(dense)
        cb.const_execute(plan, ops, out)
        return handles

    def free(handles):
        for h in handles.values():
            cb.const_destroy(h)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # the clock record starts before the warm-up, so that the start-up of nvidia-smi (which takes driver locks) is
    # over when the timed region begins; only the samples taken inside the timed region are summarised
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    # warm-up (also sizes the stream-ordered memory pool)
    level_sizes, bins, gather = None, None, None
    for _ in range(args.warmup):
        handles = step(dev, dev_dense)
        if level_sizes is None:
            torch.cuda.synchronize()
            import ctypes
            level_sizes = {}
            for n, h in handles.items():
                ns = []
                for l in range(h.order):
                    cnt = ctypes.c_int64()
                    cb.load_library().const_csf_level(h.ptr, l, None, None, ctypes.byref(cnt))
                    ns.append(cnt.value)
                level_sizes[n] = ns
            bins = {n: cb.const_csf_bin_counts(h) for n, h in handles.items()}
            if w.family != "network" and rank == 0:
                # secondary ceiling: the factor-row gathers of this very tensor (leaf rows, then fibre rows) at the
                # rate the memory system sustains for that pattern
                X = handles["X"]
                ranks = [a.shape[1] for a in w.dense.values()]
                names = list(w.dense)
                g_ms = 0.0
                for lvl in range(1, X.order):
                    crd = cb.const_csf_level(X, lvl)[1]
                    fac = w.dense[names[lvl - 1]]
                    ms_g, _ = cb.const_microbench(cb.BENCH_ROW_GATHER, crd, fac.shape[0], fac.shape[1], repeats=3)
                    g_ms += ms_g
                    del crd
                gather = {"ms": g_ms, "what": "every factor row the schedule reads, gathered once with 128-bit loads "
                                                "(const_microbench row gather on this tensor's crd arrays)", "ranks": ranks}
        free(handles)
    if cb.const_last_device_status(plan) != 0:
        raise RuntimeError("device status word reports an error")
    flops, exec_bytes = algorithmic_work(w, level_sizes)
    step_bytes = exec_bytes + build_bytes(w, level_sizes)

    def timed_loop(flush=None):
        """K steps between two events (the contract's figure) plus one event pair per step and per execute."""
        marks = []
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pre = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
                torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        e0.record(stream)
        for s in range(steps):
            a, m, b = pre[s]
            if flush is not None:
                flush.zero_()                        # a write larger than L2 evicts what the last step left there
            a.record(stream)
            handles = build_all(dev)
            m.record(stream)
            ops = dict(handles); ops.update(dev_dense)
            cb.const_execute(plan, ops, out)
            b.record(stream)
            marks.append((a, m, b))
            free(handles)
        e1.record(stream)
        barrier()
        total = e0.elapsed_time(e1)
        per_step = [a.elapsed_time(b) for a, m, b in marks]
        per_exec = [m.elapsed_time(b) for a, m, b in marks]
        return total, per_step, per_exec

    # ---- timed region: device-resident inputs ----
    import gc
    cb.const_profile_enable(True)
    gc.disable()
    t_begin = time.monotonic()
    total_ms, per_step, per_exec = timed_loop()
    remeasured = None
    if max(per_step) > 3.0 * float(np.median(per_step)) and total_ms / steps > 1.2 * float(np.median(per_step)):
        # One step far outside the others (seen on shared hosts: a stall of the launching thread of a second or
        # so while the kernels themselves keep their times) spoils the mean.  Like a run with a throttled clock
        # it is measured again, once, and the first attempt is reported next to the second.
        remeasured = {"first_ms_per_step": total_ms / steps, "first_step_ms_max": float(max(per_step)),
                      "first_step_ms_median": float(np.median(per_step)),
                      "why": "one step above 3x the median step time; measured again once"}
        cb.const_profile_enable(True)                    # also clears the records of the first attempt
        t_begin = time.monotonic()
        total_ms, per_step, per_exec = timed_loop()
    t_end = time.monotonic()
    gc.enable()
    prof = cb.const_profile_read()
    cb.const_profile_enable(False)
    clocks = sampler.stop(t_begin, t_end)
    exec_ms = float(np.mean(per_exec))
    ms_per_step = total_ms / steps
    ms_per_step, total_flops = aggregate_over_ranks(ms_per_step, flops, dist, "cuda")

    nnz_total = sum(op.nnz for op in w.sparse.values())
    fits_l2 = exec_bytes < 126e6                 # what const_execute touches stays resident in the 126 MB L2
    flushed = None
    if fits_l2 and rank == 0:
        # the working set fits the 126 MB L2: also time the steps with L2 flushed before each of them
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        _, fs, fe = timed_loop(flush)
        del flush
        flushed = {"step_ms_median": float(np.median(fs)), "step_ms_min": float(np.min(fs)),
                   "execute_ms_median": float(np.median(fe)), "execute_ms_min": float(np.min(fe)),
                   "how": "256 MB written to device memory before every step, outside its event pair"}

    # ---- end to end: host buffers in, result out ----
    h2d = sum(sum(c.numel() * c.element_size() for c in cs) + v.numel() * v.element_size() for cs, v in host.values())
    h2d += sum(a.numel() * a.element_size() for a in host_dense.values())
    d2h = out.numel() * out.element_size()
    e2e_steps = 0 if args.kernels_only else max(2, min(steps, 5))

    def e2e_step():
        src = {n: ([c.cuda(non_blocking=True) for c in cs], v.cuda(non_blocking=True)) for n, (cs, v) in host.items()}
        dense = {n: a.cuda(non_blocking=True) for n, a in host_dense.items()}
        hs = step(src, dense)
        out_host.copy_(out, non_blocking=True)
        free(hs)

    if e2e_steps:
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps if e2e_steps else float("nan")
    e2e_ms, _ = aggregate_over_ranks(e2e_ms, flops, dist, "cuda")
    result_host = out_host.numpy().copy() if e2e_steps else out.cpu().numpy()
    if rank != 0:
        return None

    # ---- per-kernel summary and rooflines ----
    ksum = sum(ms for _, ms in prof.values()) or 1.0
    kernels = [{"name": k, "launches": n, "ms_total": round(ms, 4), "share": round(ms / ksum, 4)}
               for k, (n, ms) in sorted(prof.items(), key=lambda kv: -kv[1][1])]
    gpu_launches = int(sum(n for n, _ in prof.values()))
    vbytes = w.dtype.itemsize
    fp_peak = peaks["fp64_fma_tflops" if w.family == "network" else "fp32_fma_tflops"]
    tensor_on = any(k["name"] in ("ttmc4_tc_kernel", "chain3_tc_kernel") for k in kernels)

    def roofline_of(name):
        n, ms = prof[name]
        per_launch_ms = ms / n
        per_nnz = NCU_TRAFFIC_BYTES_PER_NNZ.get((w.family, name))
        traffic = None if per_nnz is None else per_nnz * nnz_total / len(w.sparse)
        if name in FUSED_KERNELS:
            stage = tensor_stage_flops(w, level_sizes) if tensor_on else 0
            t_hbm = exec_bytes / (hbm_peak * 1e9)
            t_alu = (flops - stage) / (fp_peak * 1e12)
            t_tensor = 3 * stage / (peaks["tf32_mma_tflops"] * 1e12)     # three tf32 products per fp32 product
            ceilings = {"hbm_ms": t_hbm * 1e3, "alu_ms": t_alu * 1e3, "tensor_ms": t_tensor * 1e3,
                        "gather_ms": gather["ms"] if gather else None}
            t_roof = max(t_hbm, t_alu, t_tensor)
            common = {"kernel": name, "ms_per_launch": per_launch_ms, "roofline_ms": t_roof * 1e3,
                      "frac": t_roof / (per_launch_ms * 1e-3), "ceilings": ceilings, "traffic": traffic,
                      "frac_of_gather_ceiling": (gather["ms"] / per_launch_ms) if gather else None}
            if t_roof == t_hbm:
                ach = exec_bytes / (per_launch_ms * 1e-3) / 1e9
                return dict(common, bound="hbm", achieved=ach, peak=hbm_peak, unit="GB/s", peak_source=peak_kind)
            if t_roof == t_alu:
                ach = (flops - stage) / (per_launch_ms * 1e-3) / 1e12
                return dict(common, bound="alu", achieved=ach, peak=fp_peak, unit="TFLOP/s",
                            peak_source="register-only FMA microbenchmark of this run")
            ach = 3 * stage / (per_launch_ms * 1e-3) / 1e12
            return dict(common, bound="tensor", achieved=ach, peak=peaks["tf32_mma_tflops"], unit="TFLOP/s",
                        peak_source="tcgen05 tf32 microbenchmark of this run")
        per_elem = {"rs_onesweep": 2 * (8 + vbytes), "pack_hist": 4 * len(next(iter(w.sparse.values())).dims) + 8,
                    "csf_count": 8, "csf_scatter": 8 + 4, "csf_compress": 8 + 4}.get(name)
        if per_elem is None:
            return None
        # launches alternate over the sparse operands; bytes per launch use the mean nonzero count
        bytes_per_launch = per_elem * nnz_total / len(w.sparse)
        ach = bytes_per_launch / (per_launch_ms * 1e-3) / 1e9
        return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s",
                "frac": ach / hbm_peak, "traffic": traffic, "peak_source": peak_kind, "ms_per_launch": per_launch_ms}

    rooflines = {k["name"]: roofline_of(k["name"]) for k in kernels}
    dominant = kernels[0]["name"] if kernels else None
    roofline = rooflines.get(dominant) or {"bound": "hbm", "achieved": None, "peak": hbm_peak, "unit": "GB/s",
                                           "frac": None, "traffic": None}
    fused = next((rooflines[k] for k in rooflines if k in FUSED_KERNELS and rooflines[k]), None)

    # ---- CPU baseline (the oracle on a bounded sample, on the host's cores) and the run's own parity check ----
    cpu_baseline, max_err_ratio = None, None
    if want_oracle:
        cpu_baseline, _, rows, S, A = time_oracle(w, args.oracle_nnz or ORACLE_SAMPLE_NNZ[config_id])
        tol = 1e-5 if dtype == cb.F32 else 1e-12
        err = np.abs(result_host[rows].astype(np.float64) - S[rows])
        bound = tol * A[rows]
        if not np.all(err <= bound):
            raise RuntimeError(f"config {config_id}: result differs from the oracle beyond {tol} * sum|terms|")
        max_err_ratio = float(np.max(err / np.maximum(bound, 1e-300)))

    return {
        "workload": w.name, "dtype": "f32" if dtype == cb.F32 else "f64",
        "ms_per_step": ms_per_step, "step_ms_median": float(np.median(per_step)), "step_ms_min": float(np.min(per_step)),
        "remeasured": remeasured,
        "value": total_flops / (ms_per_step * 1e-3) / 1e9, "unit": "GFLOP/s",
        "nnz": nnz_total, "level_sizes": level_sizes, "bins": bins,
        "l2": "inputs larger than L2 (no flush)" if not fits_l2 else
              "working set fits L2: l2_flushed holds the figures with L2 flushed before every step",
        "l2_flushed": flushed,
        "stages": {"csf_build_ms": ms_per_step - exec_ms, "execute_ms": exec_ms,
                   "execute_ms_median": float(np.median(per_exec)), "execute_ms_min": float(np.min(per_exec)),
                   "execute_gflops": flops / (exec_ms * 1e-3) / 1e9,
                   "execute_hbm_gbs": exec_bytes / (exec_ms * 1e-3) / 1e9,
                   "useful_flops": flops, "compulsory_bytes_execute": exec_bytes, "compulsory_bytes_step": step_bytes},
        "hbm_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
        "kernels": kernels, "roofline": roofline, "roofline_fused_kernel": fused,
        "rooflines": {k: v for k, v in rooflines.items() if v},
        "gather_ceiling": gather, "cpu_baseline": cpu_baseline, "max_err_ratio": max_err_ratio,
        "e2e": {"value": total_flops / (e2e_ms * 1e-3) / 1e9, "unit": "GFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "gpu_launches": gpu_launches, "clocks": clocks,
    }


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=0, help="1..5: only this configuration (default: all five)")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--impl", default="const")
    ap.add_argument("--oracle-nnz", type=int, default=0, help="nonzeros in the CPU-baseline sample (0 = auto)")
    ap.add_argument("--generic-executor", action="store_true",
                    help="run the schedules on the generic loop-tree executor instead of the hand-written kernels")
    ap.add_argument("--tensor-stage", type=int, default=-1,
                    help="TTMc: 1 = dense per-slice stage on the tensor cores, 0 = on the FMA pipes, -1 = library default")
    ap.add_argument("--bins", default="", help="light_max,heavy_max,chunk nonzero thresholds of the load balancer (default: the library's)")
    ap.add_argument("--smi-ms", type=int, default=20, help="sampling interval of the clock record (nvidia-smi -lms)")
    ap.add_argument("--kernels-only", action="store_true",
                    help="skip the end-to-end and CPU-baseline legs (for profiler captures of the timed kernels)")
    args = ap.parse_args()
    ClockSampler.interval_ms = max(5, args.smi_ms)
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from workloads import make_config, CONFIG_NAMES
    t_setup = time.perf_counter()

    if args.impl == "reference":
        if rank != 0:
            return 0
        cid = args.config or HEADLINE_CONFIG
        w = make_config(cid, scale=args.scale, seed=0)
        target = args.oracle_nnz or ORACLE_SAMPLE_NNZ[cid]
        for _ in range(args.warmup):
            time_oracle(w, target)
        vals, dts = [], []
        for _ in range(max(args.steps, 1)):
            cb_, dt = time_oracle(w, target)[:2]
            vals.append(cb_["value"]); dts.append(dt)
        cb_["value"] = float(np.mean(vals))
        line = {"impl": "reference", "metric": "useful GFLOP/s", "value": cb_["value"], "unit": "GFLOP/s",
                "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": float(np.mean(dts)) * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": CONFIG_NAMES[cid], "scale": args.scale},
                "cpu_baseline": cb_,
                "e2e": {"value": cb_["value"], "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return 0

    # which configurations this run measures; with several ranks every rank runs a replica of one
    if args.config:
        config_ids = [args.config]
    elif world > 1:
        config_ids = [HEADLINE_CONFIG]
    else:
        config_ids = [HEADLINE_CONFIG, 1, 3, 4, 5]
    headline = config_ids[0]

    # Inputs are drawn by worker processes, started with `spawn` before this process touches the GPU; the headline
    # configuration is taken first so that its measurement overlaps the generation of the others.
    import multiprocessing as mp
    from concurrent.futures import ProcessPoolExecutor
    pool = ProcessPoolExecutor(max_workers=min(len(config_ids), 4), mp_context=mp.get_context("spawn"))
    futures = {cid: pool.submit(_generate, (cid, args.scale, rank)) for cid in config_ids}

    import torch
    import paper_2401_04836_b200 as cb

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    hbm_peak, peak_kind = measured_peaks()
    peaks = measure_machine_peaks(cb, local_rank)
    results, gen_s = {}, {}
    for cid in config_ids:
        _, w, gs = futures[cid].result()
        gen_s[cid] = round(gs, 1)
        results[cid] = measure_config(cb, torch, w, cid, args, peaks, hbm_peak, peak_kind, rank, dist,
                                      want_oracle=not args.kernels_only)
        del w
    pool.shutdown()
    setup_s = time.perf_counter() - t_setup

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    h = results[headline]

    def brief(r):
        """The figures of one configuration that the line's `config` carries (the full set sits in `per_config`)."""
        keep = ("kernel", "bound", "achieved", "peak", "unit", "frac", "traffic", "frac_of_gather_ceiling")
        cut = lambda d: None if d is None else {k: d.get(k) for k in keep}
        return {"workload": r["workload"], "dtype": r["dtype"], "ms_per_step": r["ms_per_step"],
                "step_ms_median": r["step_ms_median"], "step_ms_min": r["step_ms_min"],
                "execute_ms": r["stages"]["execute_ms"], "value_gflops": r["value"],
                "roofline": cut(r["roofline"]), "roofline_fused_kernel": cut(r["roofline_fused_kernel"]),
                "cpu_baseline": r["cpu_baseline"], "e2e": r["e2e"], "max_err_ratio": r["max_err_ratio"],
                "l2_flushed": r["l2_flushed"]}

    line = {
        "metric": "useful GFLOP/s", "value": h["value"], "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": h["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": h["dtype"], "data": "synthetic",
        "config": {"workload": CONFIG_NAMES[headline], "scale": args.scale,
                   "step": "const_csf_build + const_execute", "nnz": h["nnz"], "level_sizes": h["level_sizes"],
                   "bins": h["bins"], "l2": h["l2"], "replicas": world, "generation_s": gen_s,
                   "wall_s": round(setup_s, 1),
                   "per_config": {str(cid): brief(results[cid]) for cid in sorted(results)}},
        "stages": h["stages"], "hbm_gbs": h["hbm_gbs"],
        "step_ms_median": h["step_ms_median"], "step_ms_min": h["step_ms_min"], "remeasured": h["remeasured"],
        "kernels": h["kernels"], "roofline": h["roofline"], "roofline_fused_kernel": h["roofline_fused_kernel"],
        "rooflines": h["rooflines"], "gather_ceiling": h["gather_ceiling"],
        "cpu_baseline": h["cpu_baseline"], "max_err_ratio": h["max_err_ratio"], "e2e": h["e2e"],
        "gpu_launches": int(sum(r["gpu_launches"] for r in results.values())),
        "clocks": h["clocks"], "machine_peaks": dict(peaks, hbm_gbs=hbm_peak, hbm_source=peak_kind),
        "per_config": {str(cid): {k: v for k, v in results[cid].items() if k not in ("kernels", "rooflines")}
                       for cid in sorted(results)},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
