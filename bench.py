#!/usr/bin/env python
"""Benchmark of the whole hot path on seeded synthetic input.

One step = const_csf_build (COO -> CSF, including the load-balancing lists) followed by
const_execute (the fused contraction tree) on one batch.  The default workload is the large skewed
order-3 TTMc (12 000 x 9 000 x 29 000, 77 M nonzeros, rank 16).  `value` is useful GFLOP/s of the
fused schedule (2*R3*nnz + 2*R2*R3*fibres for TTMc) over the step time with inputs resident in HBM;
`e2e` is the same with host (pinned) buffers and the copies inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--scale s] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its own
GPU -- slices are independent, so there is no data-path collective -- and the line reports the sum.
`--impl reference` times the CPU oracle on a bounded sample of the same workload (rank 0 only).
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

FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 148 SMs x 128 FMA lanes x 2 flop x max SM clock
FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12

# DRAM bytes per nonzero and launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture of
# configs 2 and 3 at scale 0.3 summarised under profiles/; the kernels stream their inputs once, so the traffic
# of a full-size launch is this figure times its nonzero count.  Only valid for that workload family.
NCU_TRAFFIC_BYTES_PER_NNZ = {("ttmc3", "rs_onesweep"): 530.7e6 / 23.1e6, ("ttmc3", "chain3_kernel"): 235.8e6 / 23.1e6,
                             ("ttmc4", "ttmc4_tc_kernel"): 352.9e6 / 15.0e6}


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
    """level_sizes: {sparse name: [n_0, ..., n_leaf]} measured from the built CSF."""
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
    from oracle import contract as oc
    from tests.gpu_util import oracle
    from workloads import row_sample
    rows = sample_rows_for_oracle(w, target_nnz)
    key = "U" if w.family == "network" else "X"
    sub = row_sample(w.sparse[key], rows)
    t0 = time.perf_counter()
    oracle(w, rows)
    dt = time.perf_counter() - t0
    # flops of the fused schedule restricted to the sampled slices
    if w.family == "network":
        W = w.sparse["W"]
        flops = 2 * w.extents["l"] * sub.nnz + 2 * len(rows) * W.nnz
    else:
        coords = sub.coords
        if w.family == "ttmc4":
            f1 = np.unique(coords[0].astype(np.int64) * sub.dims[1] + coords[1]).size
            f2 = np.unique((coords[0].astype(np.int64) * sub.dims[1] + coords[1]) * sub.dims[2] + coords[2]).size
            r = w.extents["a"]
            flops = 2 * r * sub.nnz + 2 * r * r * f2 + 2 * r * r * r * f1
        else:
            f1 = np.unique(coords[0].astype(np.int64) * sub.dims[1] + coords[1]).size
            if w.family == "ttmc3":
                flops = 2 * w.extents["b"] * sub.nnz + 2 * w.extents["a"] * w.extents["b"] * f1
            else:
                flops = 2 * w.extents["r"] * (sub.nnz + f1)
    return {"value": flops / dt / 1e9, "unit": "GFLOP/s", "cores": oc.num_threads(), "kind": "oracle",
            "sample": f"{len(rows)} seeded output rows holding {sub.nnz} nonzeros, {dt:.2f} s"}, dt


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


# ------------------------------------------------------------------------------------------------
# clocks sampler
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--impl", default="const")
    ap.add_argument("--oracle-nnz", type=int, default=0, help="nonzeros in the CPU-baseline sample (0 = auto)")
    ap.add_argument("--tensor-stage", type=int, default=-1,
                    help="TTMc: 1 = dense per-slice stage on the tensor cores, 0 = on the FMA pipes, -1 = library default")
    ap.add_argument("--bins", default="", help="light_max,heavy_max,chunk nonzero thresholds of the load balancer (default: the library's)")
    ap.add_argument("--kernels-only", action="store_true",
                    help="skip the end-to-end and CPU-baseline legs (for profiler captures of the timed kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from workloads import make_config, CONFIG_NAMES
    t_setup = time.perf_counter()

    if args.impl == "reference":
        if rank != 0:
            return 0
        w = make_config(args.config, scale=args.scale, seed=0)
        auto = {1: 20_000, 2: 40_000_000, 3: 8_000_000, 4: 100_000_000, 5: 400_000}[args.config]
        target = args.oracle_nnz or auto
        for _ in range(args.warmup):
            time_oracle(w, target)
        vals, dts = [], []
        for _ in range(max(args.steps, 1)):
            cb_, dt = time_oracle(w, target)
            vals.append(cb_["value"]); dts.append(dt)
        cb_["value"] = float(np.mean(vals))
        line = {"impl": "reference", "metric": "useful GFLOP/s", "value": cb_["value"], "unit": "GFLOP/s",
                "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": float(np.mean(dts)) * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": CONFIG_NAMES[args.config], "scale": args.scale},
                "cpu_baseline": cb_,
                "e2e": {"value": cb_["value"], "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return 0

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

    w = make_config(args.config, scale=args.scale, seed=rank)           # one independent replica per rank
    dtype = cb.F32 if w.dtype == np.float32 else cb.F64
    tdtype = torch.float32 if dtype == cb.F32 else torch.float64
    setup_s = time.perf_counter() - t_setup

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

    # warm-up (also sizes the stream-ordered memory pool)
    level_sizes = None
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
        free(handles)
    if cb.const_last_device_status(plan) != 0:
        raise RuntimeError("device status word reports an error")
    flops, exec_bytes = algorithmic_work(w, level_sizes)

    # ---- timed region: device-resident inputs ----
    sampler = ClockSampler(local_rank)
    sampler.start()
    cb.const_profile_enable(True)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps + 2)]
    barrier()
    ev[0].record(stream)
    mids = []
    for s in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        handles = build_all(dev)
        a.record(stream)
        ops = dict(handles); ops.update(dev_dense)
        cb.const_execute(plan, ops, out)
        b.record(stream)
        mids.append((a, b))
        free(handles)
    ev[1].record(stream)
    barrier()
    total_ms = ev[0].elapsed_time(ev[1])
    exec_ms = float(np.mean([a.elapsed_time(b) for a, b in mids]))
    prof = cb.const_profile_read()
    cb.const_profile_enable(False)
    clocks = sampler.stop()
    ms_per_step = total_ms / args.steps
    ms_per_step, total_flops = aggregate_over_ranks(ms_per_step, flops, dist, "cuda")

    # ---- end to end: host buffers in, result out ----
    h2d = sum(sum(c.numel() * c.element_size() for c in cs) + v.numel() * v.element_size() for cs, v in host.values())
    h2d += sum(a.numel() * a.element_size() for a in host_dense.values())
    d2h = out.numel() * out.element_size()
    e2e_steps = 0 if args.kernels_only else max(2, min(args.steps, 5))

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

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    # ---- per-kernel summary and roofline of the dominant kernel ----
    hbm_peak, peak_kind = measured_peaks()
    nnz_total = sum(op.nnz for op in w.sparse.values())
    ksum = sum(ms for _, ms in prof.values()) or 1.0
    kernels = [{"name": k, "launches": n, "ms_total": round(ms, 4), "share": round(ms / ksum, 4)}
               for k, (n, ms) in sorted(prof.items(), key=lambda kv: -kv[1][1])]
    gpu_launches = int(sum(n for n, _ in prof.values()))
    fused_names = {"chain3_kernel", "chain3_tc_kernel", "ttmc4_kernel", "ttmc4_tc_kernel", "network_kernel"}
    vbytes = w.dtype.itemsize

    def traffic_of(name):
        per = NCU_TRAFFIC_BYTES_PER_NNZ.get((w.family, name))
        return None if per is None else per * nnz_total / len(w.sparse)

    def roofline_of(name):
        r = _roofline_of(name)
        if r is not None:
            r["traffic"] = traffic_of(name)
        return r

    def _roofline_of(name):
        n, ms = prof[name]
        per_launch_ms = ms / n
        if name in fused_names:
            t_hbm = exec_bytes / (hbm_peak * 1e9)
            peak_alu = (FP64_PEAK_TFLOPS if w.family == "network" else FP32_PEAK_TFLOPS) * 1e12
            t_alu = flops / peak_alu
            if t_alu >= t_hbm:
                ach = flops / (per_launch_ms * 1e-3) / 1e12
                return {"kernel": name, "bound": "alu", "achieved": ach, "peak": peak_alu / 1e12, "unit": "TFLOP/s",
                        "frac": ach / (peak_alu / 1e12), "traffic": None,
                        "peak_source": "148 SMs x FMA lanes x 2 x 1.965 GHz (nominal max clock)",
                        "hbm_gbs_achieved": exec_bytes / (per_launch_ms * 1e-3) / 1e9}
            ach = exec_bytes / (per_launch_ms * 1e-3) / 1e9
            return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s",
                    "frac": ach / hbm_peak, "traffic": None, "peak_source": peak_kind}
        per_elem = {"rs_onesweep": 2 * (8 + vbytes), "rs_histogram": 8, "pack_keys": 4 * len(w.mode_orders) + 8,
                    "csf_count": 8, "csf_scatter": 8 + 4}.get(name)
        if per_elem is None:
            return None
        # launches alternate over the sparse operands; bytes per launch use the mean nonzero count
        bytes_per_launch = per_elem * nnz_total / len(w.sparse)
        ach = bytes_per_launch / (per_launch_ms * 1e-3) / 1e9
        return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s",
                "frac": ach / hbm_peak, "traffic": None, "peak_source": peak_kind}

    rooflines = {k["name"]: roofline_of(k["name"]) for k in kernels}
    dominant = kernels[0]["name"] if kernels else None
    roofline = rooflines.get(dominant) or {"bound": "hbm", "achieved": None, "peak": hbm_peak, "unit": "GB/s",
                                           "frac": None, "traffic": None}
    fused = next((rooflines[k] for k in rooflines if k in fused_names and rooflines[k]), None)

    # ---- CPU baseline: the oracle on a bounded sample, on this machine's host cores ----
    auto = {1: 20_000, 2: 40_000_000, 3: 8_000_000, 4: 100_000_000, 5: 400_000}[args.config]
    cpu_baseline = None if args.kernels_only else time_oracle(w, args.oracle_nnz or auto)[0]

    line = {
        "metric": "useful GFLOP/s", "value": total_flops / (ms_per_step * 1e-3) / 1e9,
        "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if dtype == cb.F32 else "f64", "data": "synthetic",
        "config": {"workload": CONFIG_NAMES[args.config], "scale": args.scale,
                   "step": "const_csf_build + const_execute", "nnz": nnz_total, "level_sizes": level_sizes,
                   "bins": bins, "l2": "inputs larger than L2 (no flush)" if nnz_total * 16 > 126e6
                   else "working set fits L2; no flush between iterations", "replicas": world,
                   "setup_s": round(setup_s, 1)},
        "stages": {"csf_build_ms": ms_per_step - exec_ms, "execute_ms": exec_ms,
                   "execute_gflops": flops / (exec_ms * 1e-3) / 1e9,
                   "execute_hbm_gbs": exec_bytes / (exec_ms * 1e-3) / 1e9,
                   "useful_flops": flops, "compulsory_bytes_execute": exec_bytes},
        "hbm_gbs": (exec_bytes + sum((rooflines[k["name"]] or {}).get("achieved", 0) * 0 for k in kernels))
                   / (ms_per_step * 1e-3) / 1e9,
        "kernels": kernels, "roofline": roofline, "roofline_fused_kernel": fused,
        "rooflines": {k: v for k, v in rooflines.items() if v},
        "cpu_baseline": cpu_baseline,
        "e2e": {"value": total_flops / (e2e_ms * 1e-3) / 1e9, "unit": "GFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "gpu_launches": gpu_launches, "clocks": clocks,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
