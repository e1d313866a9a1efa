#!/usr/bin/env python
"""Benchmark of the SpGEMM hot path (plan + execute = every step of Algorithm 3) on synthetic inputs.

    python bench.py --gpus 1 --steps 5 --warmup 3            # CUDA library, default workload
    python bench.py --impl reference --steps 2 --warmup 1    # CPU oracle on a bounded row sample

One "step" is one whole product C = A*B: row analysis, planning, light rows, and for the heavy rows
expansion, every multisplit level and the chunk accumulation, with A and B resident in HBM.  The
metric is SpGEMM GFLOP/s = 2 * intermediate products / time.  The line also carries the roofline
of the dominant kernel, the oracle timed on the host cores, and an end-to-end number measured
through the host-buffer entry point (copies inside the timed region).

Multi-GPU: the path does not shard in this build ("replicas only"): with --gpus N every rank runs
the same product on its own GPU, no collective touches the data path.
"""
from __future__ import annotations

import argparse
import ctypes
import gc
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

SMEM_BYTES = 232448
DEFAULT_CONFIG = 2  # R-MAT scale 20, edge factor 16, fp32: the largest fp32 power-law product


# DRAM bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum) over the algorithmic bytes of the same
# launch, from single-kernel, single-launch ncu captures of these kernels on the same product scaled down by 2**3
# (R-MAT scale 17: one batch holds the whole product, 1.09 G products, about 9 GB staged).  Traffic grows in
# proportion to the products processed, so a full-size launch is its algorithmic figure times this ratio.  A kernel
# that has changed since its capture must lose its entry (traffic is then reported as null).
TRAFFIC_RATIO = {"k4_expand": 1.03, "k5a_histogram": 1.00, "k5b_multisplit": 1.00, "k6_small_chunks": 0.63,
                 "k6_mid_chunks": 0.99, "k6_accumulate": 1.00, "k7_gather": 1.00}
TRAFFIC_SOURCE = ("single-kernel, single-launch ncu DRAM-counter captures on the same recipe 2**3 smaller (R-MAT scale 17, "
                  "one batch holds the whole product), scaled by products")


def ctypes_copy(dst, src):
    ctypes.memmove(ctypes.byref(dst), ctypes.byref(src), ctypes.sizeof(src))


def max_over_ranks(ms_local: float, world: int, device) -> float:
    """Step time of a multi-rank run: every rank times its own replica on its device, the job's time is the slowest
    rank's (MAX all-reduce; the backend is whatever the process group was made with)."""
    if world <= 1:
        return float(ms_local)
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicas_value(products_per_replica: int, world: int, ms_step: float) -> float:
    """Whole-job GFLOP/s of `world` independent replicas ("replicas only": no data-path collective): all ranks'
    products over the slowest rank's time."""
    return world * 2.0 * products_per_replica / (ms_step * 1e-3) / 1e9


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons during the timed region: NVML from a background thread (a few
    light queries every 200 ms; an nvidia-smi polling loop measurably slowed short steps), nvidia-smi as a
    fallback when the NVML binding is missing."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, interval: float = 0.2):
        self.gpu_index, self.proc, self.path, self.interval = gpu_index, None, None, interval
        self.thread, self.stop_flag, self.sm, self.mx, self.reasons = None, False, [], [], set()

    def _nvml_loop(self, nv, handle):
        masks = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                self.mx.append(float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM)))
                r = int(get_reasons(handle))
                for name, m in masks.items():
                    if r & m:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.interval)

    def start(self):
        try:
            import threading

            import pynvml as nv
            import torch

            nv.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(self.gpu_index).uuid)
            handle = None
            for i in range(nv.nvmlDeviceGetCount()):
                h = nv.nvmlDeviceGetHandleByIndex(i)
                u = nv.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u:
                    handle = h
            if handle is None:
                handle = nv.nvmlDeviceGetHandleByIndex(self.gpu_index)
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "500",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.thread is not None:
            time.sleep(0.25)
            self.stop_flag = True
            self.thread.join(timeout=2)
            if self.sm:
                out.update(sm_mhz=statistics.median(self.sm), sm_max_mhz=max(self.mx), reasons=sorted(self.reasons),
                           samples=len(self.sm), source="nvml")
            return out
        if self.proc is None:
            return out
        time.sleep(0.6)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                sm.append(float(f[1])), mx.append(float(f[2]))
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       source="nvidia-smi")
        return out


def _row_sample(n_rows: int, blocks: int, frac: float):
    """`blocks` evenly spaced contiguous row ranges that together cover `frac` of the rows."""
    blocks = max(1, min(blocks, n_rows))
    width = max(1, int(n_rows * frac / blocks))
    starts = np.linspace(0, max(n_rows - width, 0), blocks).astype(np.int64)
    return [(int(s), int(min(n_rows, s + width))) for s in starts]


def oracle_timed(A, B, budget_s: float = 15.0):
    """Times the CPU oracle (as it stands) on a bounded, evenly spread sample of row blocks.  Returns
    (gflops, cores, description, seconds, products)."""
    import oracle

    ip = oracle.row_products(A, B)
    total = int(ip.sum())
    # Every call of the oracle sets up one dense accumulator of C.m columns per thread; with millions of columns
    # that set-up must be spread over many rows, so a wide product is timed on a few large blocks.
    wide = B.n_cols > (1 << 21)
    n_blocks = 4 if wide else 64
    # calibrate on a small sample, then size the real one for roughly `budget_s`
    cal = _row_sample(A.n_rows, 2 if wide else 16, 0.02 if wide else 0.002)
    t = time.perf_counter()
    threads = 1
    for r0, r1 in cal:
        threads = oracle.spgemm(A, B, r0, r1).threads
    dt = max(time.perf_counter() - t, 1e-4)
    cal_products = sum(int(ip[r0:r1].sum()) for r0, r1 in cal)
    rate = max(cal_products, 1) / dt
    frac = min(1.0, max(0.004, budget_s * rate / max(total, 1)))
    blocks = _row_sample(A.n_rows, n_blocks, frac)
    products = sum(int(ip[r0:r1].sum()) for r0, r1 in blocks)
    t = time.perf_counter()
    for r0, r1 in blocks:
        oracle.spgemm(A, B, r0, r1)
    dt = time.perf_counter() - t
    desc = (f"{len(blocks)} evenly spaced row blocks = {100.0 * sum(b - a for a, b in blocks) / max(A.n_rows, 1):.2f}% of rows, "
            f"{products} of {total} products, {dt:.1f} s")
    return 2.0 * products / dt / 1e9, threads, desc, dt, products


def kernel_table(info, stats_avg, sv, nnz_b, n_light_entries_a):
    """Algorithmic (minimum) bytes per step for every kernel of the path, with its measured time."""
    se = 4 + sv
    e = info.products_heavy
    p = info.params
    rows_h = info.rows_heavy
    L = p.n_levels
    nnz_c, nnz_ch = stats_avg["c_nnz"], stats_avg["c_nnz_heavy"]
    chunks = stats_avg["final_chunks"]
    e_small, nnz_small = stats_avg["small_chunk_products"], stats_avg["small_chunk_entries"]
    e_mid, nnz_mid = stats_avg["mid_chunk_products"], stats_avg["mid_chunk_entries"]
    parents = [rows_h]
    for l in range(L):
        parents.append(parents[-1] * p.fanout[l])
    # the expansion writes the first level's children itself (level0_direct): no pass over the staging buffer for
    # that level, only per-segment run starts (read two child-boundary rows of B, write one row of prefixes)
    l0 = 1 if (L > 0 and info.level0_direct) else 0
    hist = sum(4 * e + 8 * (parents[l] + 1) + 4 * parents[l + 1] for l in range(l0, L))
    # a multisplit pass reads every column of the batch and moves (reads the value of, writes) only the products of
    # chunks that have not left the hierarchy early
    moved = stats_avg["split_products"]
    split = (2 * se * moved + 4 * ((L - l0) * e - moved)
             + sum(8 * (parents[l] + 1) + 8 * parents[l + 1] for l in range(l0, L)))
    seg_tables = (12 * p.fanout[0] * info.nnz_a_heavy + 4 * parents[1]) if l0 else 0
    tbl = {
        "k3_light_symbolic": (4 * n_light_entries_a + 8 * info.rows_light + 4 * nnz_b, stats_avg["ms_light_symbolic"]),
        "k3_light_numeric": (se * n_light_entries_a + se * nnz_b + se * (nnz_c - nnz_ch), stats_avg["ms_light_numeric"]),
        "k4_expand": (se * e + se * nnz_b + 24 * info.nnz_a_heavy + (4 * p.fanout[0] * info.nnz_a_heavy if l0 else 0),
                      stats_avg["ms_expand"]),
        "k5a_histogram": (hist + seg_tables, stats_avg["ms_histogram"]),
        "k5b_multisplit": (split, stats_avg["ms_multisplit"]),
        # chunks of few products are sorted by one warp each, mid-size ones take a small block each (its second pass
        # re-reads the chunk from L2: not counted), the dense-accumulator kernel owes the rest
        "k6_small_chunks": (se * e_small + se * nnz_small + 12 * chunks, stats_avg["ms_small_chunks"]),
        "k6_mid_chunks": (se * e_mid + se * nnz_mid, stats_avg["ms_mid_chunks"]),
        "k6_accumulate": (se * (e - e_small - e_mid) + se * (nnz_ch - nnz_small - nnz_mid) + 12 * chunks,
                          stats_avg["ms_accumulate"]),
        "k7_gather": (2 * se * nnz_ch + 24 * chunks, stats_avg["ms_gather"]),
    }
    return {k: {"bytes": int(b), "ms": float(ms), "gbs": (b / ms / 1e6 if ms > 0 else 0.0)} for k, (b, ms) in tbl.items()}


def run_reference(args, A, B, desc):
    vals, used = [], 1
    sample = ""
    for i in range(args.warmup + args.steps):
        gf, used, sample, dt, products = oracle_timed(A, B, budget_s=args.cpu_budget)
        if i >= args.warmup:
            vals.append((gf, dt))
    value = statistics.mean(v for v, _ in vals)
    ms = statistics.mean(d for _, d in vals) * 1e3
    line = {
        "impl": "reference", "metric": "spgemm_gflops", "value": value, "unit": "GFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32" if A.val.dtype == np.float32 else "f64", "data": "synthetic",
        "config": {"workload": gen.CONFIG_NAMES[args.config] + (f"_shrink{args.shrink}" if args.shrink else ""),
                   "description": desc,
                   "note": "CPU oracle (plain Gustavson) timed on a bounded row sample per step"},
        "cpu_baseline": {"value": value, "unit": "GFLOP/s", "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG, help="index into the five workloads (0..4)")
    ap.add_argument("--shrink", type=int, default=0, help="scale the workload down by 2**shrink (debugging)")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle time for the CPU baseline")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--clock-interval", type=float, default=0.2,
                    help="seconds between clock samples during the timed region (0: no sampling; diagnostic)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the forced-multisplit step and the per-config list (default workload only)")
    ap.add_argument("--opt", action="append", default=[], metavar="FIELD=INT",
                    help="set a field of gm_plan_opts (e.g. level0_multisplit=1, tau=4096); repeatable")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 1)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank != 0:
            return
        A, B, desc = gen.config_inputs(args.config, args.shrink)
        run_reference(args, A, B, desc)
        return

    import torch
    import torch.distributed as dist

    import paper_2607_22866_b200 as gm

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    A, B, desc = gen.config_inputs(args.config, args.shrink)
    sv = A.val.dtype.itemsize
    dA = gm.DeviceCSR.from_host(A)
    dB = dA if B is A else gm.DeviceCSR.from_host(B)
    opts = gm.PlanOpts()
    for kv in args.opt:
        field, _, value = kv.partition("=")
        if field not in dict(opts._fields_) or field == "reserved":
            raise SystemExit(f"--opt: gm_plan_opts has no field '{field}'")
        setattr(opts, field, int(value))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def measure(A, B, dA, dB, opts, steps, warmup, sample_clocks):
        """`warmup` untimed and `steps` timed products (plan + execute each).  Returns a dict with the step time,
        the plan's facts, the per-kernel table (algorithmic bytes, CUDA-event time) and the dominant kernel."""
        sv = A.val.dtype.itemsize
        step_parts = []

        def step(timing: bool):
            t_a = time.perf_counter()
            plan = gm.spgemm_plan(dA, dB, SMEM_BYTES, opts)
            t_b = time.perf_counter()
            if timing:
                plan.set_timing(True)
            C = gm.spgemm_execute(plan)
            t_c = time.perf_counter()
            info, st = plan.info(), plan.stats()
            nnz = C.nnz
            del C
            plan.destroy()
            if timing:  # host clock: plan, execute (both return after a stream synchronize); device: execute
                step_parts.append([round((t_b - t_a) * 1e3, 2), round((t_c - t_b) * 1e3, 2), round(float(st.ms_total), 2)])
            return info, st, nnz

        for _ in range(warmup):
            info, st, nnz = step(False)
        barrier()
        sampler = ClockSampler(local_rank, args.clock_interval) if sample_clocks and args.clock_interval > 0 else None
        if sampler:
            sampler.start()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record()
        launches = 0
        stats_sum: dict[str, float] = {}
        ms_steps = []  # host clock per step (execute returns after a stream synchronize): shows a hiccup if there is one
        for _ in range(steps):
            t_step = time.perf_counter()
            info, st, nnz = step(True)
            ms_steps.append(round((time.perf_counter() - t_step) * 1e3, 2))
            launches += int(info.launches + st.launches)
            for name, _t in st._fields_:
                if name != "reserved":
                    stats_sum[name] = stats_sum.get(name, 0.0) + float(getattr(st, name))
        ev1.record()
        barrier()
        clocks = sampler.stop() if sampler else None
        ms_step = max_over_ranks(ev0.elapsed_time(ev1), world, "cuda") / steps
        products = int(info.products_total)
        stats_avg = {k: v / steps for k, v in stats_sum.items()}
        # byte model: the row analysis (untimed plan) says which entries of A sit in light rows
        plan = gm.spgemm_plan(dA, dB, SMEM_BYTES, opts)
        ip_dev = plan.row_products().cpu().numpy()
        plan.destroy()
        n_light_entries_a = int(np.diff(A.row_ptr)[ip_dev <= info.params.tau].sum())
        kt = kernel_table(info, stats_avg, sv, B.nnz, n_light_entries_a)
        dom = max(kt, key=lambda k: kt[k]["ms"])
        return {"ms_step": ms_step, "value": replicas_value(products, world, ms_step), "products": products,
                "info": info, "kernels": kt, "dominant": dom, "launches": launches, "nnz": int(nnz), "clocks": clocks,
                "early_exit_products": int(stats_avg["early_exit_products"]), "ms_steps": ms_steps, "step_parts": step_parts,
                "ms_execute_device": stats_avg["ms_total"]}

    peak, peak_kind = _peaks()
    m = measure(A, B, dA, dB, opts, args.steps, args.warmup, True)
    info, kt, dom, nnz, products, launches = m["info"], m["kernels"], m["dominant"], m["nnz"], m["products"], m["launches"]
    value, ms_step, clocks, tau = m["value"], m["ms_step"], m["clocks"], info.params.tau

    # ---- roofline of the dominant kernel (times: CUDA events recorded by the library on the execute stream)
    n_b = max(int(info.n_batches), 1)
    n_split = max(info.params.n_levels - (1 if info.level0_direct else 0), 1)
    per_launch = {"k4_expand": n_b, "k5a_histogram": n_b * n_split,
                  "k5b_multisplit": n_b * n_split, "k6_accumulate": n_b,
                  "k6_small_chunks": n_b, "k6_mid_chunks": n_b, "k7_gather": n_b}.get(dom, 1)
    roofline = {"kernel": dom, "bound": "hbm", "achieved": kt[dom]["gbs"], "peak": peak, "unit": "GB/s",
                "frac": kt[dom]["gbs"] / peak, "peak_kind": f"of {peak_kind}",
                "traffic": (kt[dom]["bytes"] / per_launch * TRAFFIC_RATIO[dom]) if dom in TRAFFIC_RATIO else None,
                "traffic_source": TRAFFIC_SOURCE,
                "bytes_per_launch": kt[dom]["bytes"] / per_launch, "ms_per_launch": kt[dom]["ms"] / per_launch,
                "launches_per_step": per_launch}

    line = {
        "metric": "spgemm_gflops", "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if sv == 4 else "f64", "data": "synthetic",
        "config": {"workload": gen.CONFIG_NAMES[args.config] + (f"_shrink{args.shrink}" if args.shrink else ""),
                   "description": desc, "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "l2": "inputs, staging and C are far larger than L2 (126 MB); no flush needed",
                   "products": products, "products_heavy": int(info.products_heavy), "nnz_c": int(nnz),
                   "rows_heavy": int(info.rows_heavy), "tau": int(tau), "chunk_width": int(info.params.chunk_width),
                   "levels": info.params.levels(), "batches": int(info.n_batches), "smem_bytes": SMEM_BYTES,
                   "level0_direct": int(info.level0_direct),
                   "early_exit_products": m["early_exit_products"], "plan_opts": args.opt,
                   "step": "gm_spgemm_plan + gm_spgemm_execute (C freed after each step)"},
        "roofline": roofline, "kernels": kt, "clocks": clocks, "gpu_launches": launches,
        "ms_steps_host_clock": m["ms_steps"], "ms_execute_device": m["ms_execute_device"],
        "ms_plan_execute_host_execute_device": m["step_parts"],
    }

    def frac_of(k):
        return {"bytes": k["bytes"], "ms": k["ms"], "gbs": k["gbs"], "frac": k["gbs"] / peak, "peak_kind": f"of {peak_kind}"}

    if rank == 0 and not args.no_extra and info.params.n_levels > 0 and info.rows_heavy > 0:
        # The default plan of a one-level product lets the expansion place the products, so no multisplit pass runs
        # in the timed steps above.  Same workload once more with the first level as the separate histogram and
        # multisplit passes over the staging buffer (Algorithm 5 as printed): the multisplit kernel's own number.
        o2 = gm.PlanOpts()
        ctypes_copy(o2, opts)
        o2.level0_multisplit = 1
        o2.separate_histogram = 1
        mf = measure(A, B, dA, dB, o2, max(2, min(args.steps, 3)), 1, False)
        line["kernels_multisplit_forced"] = {
            "plan_opts": ["level0_multisplit=1", "separate_histogram=1"], "ms_per_step": mf["ms_step"], "value": mf["value"],
            "k4_expand": frac_of(mf["kernels"]["k4_expand"]), "k5a_histogram": frac_of(mf["kernels"]["k5a_histogram"]),
            "k5b_multisplit": frac_of(mf["kernels"]["k5b_multisplit"])}

    if rank == 0 and not args.no_extra and args.config == DEFAULT_CONFIG and args.shrink == 0:
        # the other four workloads, a few steps each: GFLOP/s and the dominant kernel's fraction of the HBM roof
        del dA, dB
        per_config = []
        for ci in [c for c in range(len(gen.CONFIG_NAMES)) if c != args.config]:
            gc.collect()
            torch.cuda.empty_cache()
            try:
                Ai, Bi, _d = gen.config_inputs(ci)
                dAi = gm.DeviceCSR.from_host(Ai)
                dBi = dAi if Bi is Ai else gm.DeviceCSR.from_host(Bi)
                mi = measure(Ai, Bi, dAi, dBi, gm.PlanOpts(), 3, 3, False)
                kd = mi["kernels"][mi["dominant"]]
                per_config.append({"workload": gen.CONFIG_NAMES[ci], "dtype": "f32" if Ai.val.dtype.itemsize == 4 else "f64",
                                   "value": mi["value"], "unit": "GFLOP/s", "ms_per_step": mi["ms_step"], "steps": 3,
                                   "products": mi["products"], "nnz_c": mi["nnz"], "levels": mi["info"].params.levels(),
                                   "batches": int(mi["info"].n_batches), "dominant_kernel": mi["dominant"],
                                   "achieved": kd["gbs"], "frac": kd["gbs"] / peak, "peak_kind": f"of {peak_kind}"})
                del dAi, dBi, Ai, Bi
            except (gm.GmError, MemoryError, RuntimeError) as exc:
                per_config.append({"workload": gen.CONFIG_NAMES[ci], "skipped": f"{type(exc).__name__}: {exc}"[:200]})
        line["per_config"] = per_config
        dA = dB = None

    if rank == 0 and not args.no_e2e:
        # the host entry point uploads A and B itself: give it the whole device (no resident copies, no cached blocks)
        dA = dB = None
        gc.collect()
        torch.cuda.empty_cache()
        try:
            line["e2e"] = e2e_leg(gm, torch, A, B, int(nnz), products, args.e2e_steps)
        except (gm.GmError, MemoryError, RuntimeError) as exc:  # the device-timed line above stands on its own
            line["e2e"] = {"value": None, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                           "skipped": f"{type(exc).__name__}: {exc}"[:300]}
    if rank == 0 and not args.no_cpu_baseline:
        gf, cores, sample, _dt, _p = oracle_timed(A, B, budget_s=args.cpu_budget)
        line["cpu_baseline"] = {"value": gf, "unit": "GFLOP/s", "cores": cores, "kind": "oracle", "sample": sample}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def e2e_leg(gm, torch, A, B, nnz, products, steps):
    """Same product through gm_spgemm_host: A and B start in pinned host memory, C ends in pinned host
    memory; the copies are inside the timed region."""
    sv = A.val.dtype.itemsize

    def pinned(arr):
        t = torch.from_numpy(arr)
        try:
            return t.pin_memory().numpy()
        except Exception:
            return arr

    class H:  # host CSR over pinned arrays
        pass

    def host_csr(M):
        h = H()
        h.n_rows, h.n_cols = M.n_rows, M.n_cols
        h.row_ptr, h.col, h.val = pinned(M.row_ptr), pinned(M.col), pinned(M.val)
        return h

    # C comes back into host buffers of nnz(C) entries: leave the leg out rather than have the host run out of memory
    need = nnz * (4 + sv) + 2 * (A.nnz + (0 if B is A else B.nnz)) * (4 + sv)
    try:
        import psutil
        avail = psutil.virtual_memory().available
    except Exception:
        avail = None
    if avail is not None and need > 0.7 * avail:
        return {"value": None, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "skipped": f"host buffers of {need / 1e9:.0f} GB for A, B and C do not fit beside the generator's "
                           f"copies in {avail / 1e9:.0f} GB of available host memory"}
    hA = host_csr(A)
    hB = hA if B is A else host_csr(B)
    # Destination of C: page-locked in place (torch's pinned allocator would round 39 GB up to 64 GB per array)
    out_rp = np.empty(A.n_rows + 1, np.int64)
    out_col = np.empty(nnz, np.int32)
    out_val = np.empty(nnz, A.val.dtype)
    rt = torch.cuda.cudart()
    registered = []
    pin = True
    for arr in (out_rp, out_col, out_val):
        try:
            if arr.nbytes and int(rt.cudaHostRegister(arr.ctypes.data, arr.nbytes, 0)) == 0:
                registered.append(arr)
            else:
                pin = False
        except Exception:
            pin = False
    h2d = 2 * ((A.n_rows + 1) * 8 + A.nnz * (4 + sv)) if B is A else \
        (A.n_rows + 1) * 8 + A.nnz * (4 + sv) + (B.n_rows + 1) * 8 + B.nnz * (4 + sv)
    d2h = (A.n_rows + 1) * 8 + nnz * (4 + sv)
    gm.spgemm_host(hA, hB, out_rp, out_col, out_val, SMEM_BYTES)  # warm-up
    torch.cuda.synchronize()
    t = time.perf_counter()
    for _ in range(steps):
        got = gm.spgemm_host(hA, hB, out_rp, out_col, out_val, SMEM_BYTES)
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t) / steps
    assert got == nnz and int(out_rp[-1]) == nnz
    for arr in registered:
        rt.cudaHostUnregister(arr.ctypes.data)
    return {"value": 2.0 * products / dt / 1e9, "unit": "GFLOP/s", "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "ms_per_step": dt * 1e3, "steps": steps, "pinned_host_buffers": pin,
            "api": "gm_spgemm_host"}


if __name__ == "__main__":
    main()
