#!/usr/bin/env python
"""Benchmark of the batched inverse-Helmholtz tensor-product operator on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload i] [--no-cpu-baseline] [--no-e2e]

One *step* is one pass of the whole operator over the workload's E elements (one
library call).  Default workload: the largest inverse-Helmholtz configuration
(n = 14, E = 131072, fp64, 8.63 GB of u/D/v per step -- far larger than L2, so every
step streams from HBM).  Prints ONE JSON line on rank 0.

For N > 1 launch with ``python -m torch.distributed.run --nproc-per-node N``: every
rank holds its own E elements (weak scaling; elements are independent, so there is
no data-path collective -- NCCL is used only for the barrier and the max-over-ranks
of the device time).

``--impl reference`` times the CPU oracle, as it stands, on the host cores over a
bounded sample of the same workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "elements/s (fp64 SEM inverse-Helmholtz); GFLOP/s and roofline fraction alongside"
UNIT = "elements/s"

# FP64 roof derived from unit counts and clocks: 148 SMs x 64 FP64 FMA lanes per SM per
# clock x 2 flops x 1.965 GHz (clocks.max.sm).
FP64_LANES_PER_SM = 64
SM_COUNT = 148
SM_MAX_GHZ = 1.965
FP64_PEAK_TFLOPS = SM_COUNT * FP64_LANES_PER_SM * 2 * SM_MAX_GHZ / 1e3
HBM_FALLBACK_GBS = 6650.0

# Nominal figures quoted for context beside the measured ones: HBM3e bandwidth and the FP64
# rate of the data sheet.
NOMINAL_HBM_GBS = 8000.0
NOMINAL_FP64_TFLOPS = 40.0
L2_BYTES = 126e6


def ncu_traffic_bytes_per_element(wl_index: int):
    """DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per element of the operator
    kernel from the ncu capture recorded in profiles/dram_traffic.json (taken on a smaller E of
    the same kernel; traffic is proportional to the number of elements).  None if there is no
    capture for this workload or the kernel sources have changed since it was taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            entry = json.load(f).get(f"cfg{wl_index}")
        from paper_2604_19906_b200 import profile_summary
        if entry and entry.get("source_digest") == profile_summary.source_digest():
            return float(entry["bytes_per_element"])
    except Exception:
        pass
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                return json.load(f), "measured"
        except Exception:
            pass
    return {"hbm_gbs": HBM_FALLBACK_GBS}, "fallback"


# ------------------------------------------------------------------------------ clocks

class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML (read-only)."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, uuid: str | None, index: int, period: float = 0.02):
        super().__init__(daemon=True)
        self.period = period
        self.samples, self.power, self.mask = [], [], 0
        self.sm_max = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-")
                                                          else "GPU-" + uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.mask |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self) -> dict:
        self._halt.set()
        if self.is_alive():
            self.join()
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["unavailable"]}
        reasons = [name for bit, name in self.REASONS.items() if self.mask & bit]
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.sm_max,
                "sm_min_mhz": min(self.samples), "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None,
                "reasons": reasons}


# ------------------------------------------------------------------------------ CPU oracle leg

def oracle_run(wl, e0, e1):
    """Oracle over elements [e0,e1) of the workload; returns (seconds, output, inputs)."""
    import oracle
    from paper_2604_19906_b200 import inputs
    host = inputs.host_case(wl, e0, e1)
    t0 = time.perf_counter()
    if wl.op == "inv_helmholtz":
        v = oracle.inv_helmholtz(host["S"], host["D"], host["u"])
    elif wl.op == "convection":
        v = oracle.convection(host["Dvq"], host["Ivq"], host["M"], host["P"])
        v = np.ascontiguousarray(np.moveaxis(v, 0, 1))        # [E,3,nv,nv,nv]: element first
    else:
        v = oracle.tpo_apply(host["A"], host["B"], host["C"], host["u"])
    return time.perf_counter() - t0, v, host


def oracle_call(wl, host, threads=0):
    import oracle
    if wl.op == "inv_helmholtz":
        return oracle.inv_helmholtz(host["S"], host["D"], host["u"], threads)
    if wl.op == "convection":
        return oracle.convection(host["Dvq"], host["Ivq"], host["M"], host["P"], threads)
    return oracle.tpo_apply(host["A"], host["B"], host["C"], host["u"], threads)


def cpu_baseline(wl, target_seconds=4.0, max_elements=None):
    """The oracle, as it stands, on all host cores over a bounded sample (the first Ns
    elements) of the workload: one untimed pass, then the best of three timed ones.  Also a
    1-thread figure on (at most) the first 8192 elements -- the batch size and the "seq."
    column of the paper's Table 2.  Returns the cpu_baseline object, the sample's output."""
    import oracle
    from paper_2604_19906_b200 import inputs
    probe = min(wl.E, 256)
    t_probe, _, _ = oracle_run(wl, 0, probe)
    rate = probe / max(t_probe, 1e-6)
    ns = int(min(wl.E, max(probe, rate * target_seconds)))
    if max_elements:
        ns = min(ns, max_elements)
    _, v, host = oracle_run(wl, 0, ns)                        # warm-up pass, keeps the output
    times = []
    for _ in range(3):
        t0 = time.perf_counter()
        oracle_call(wl, host)
        times.append(time.perf_counter() - t0)
    t = min(times)
    cores = oracle.threads_used(0)
    n1 = min(wl.E, 8192, ns)
    host1 = host if n1 == ns else inputs.host_case(wl, 0, n1)
    oracle_call(wl, host1, 1)
    t0 = time.perf_counter()
    oracle_call(wl, host1, 1)
    t1 = time.perf_counter() - t0
    return {"value": ns / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "gflops": ns * wl.flops_per_element / t / 1e9,
            "sample": f"first {ns} of {wl.E} elements of {wl.name}, best of 3 warm passes "
                      f"({t:.2f} s) on {cores} threads",
            "one_thread": {"value": n1 / t1, "unit": UNIT, "elements": n1,
                           "ms": t1 * 1e3,
                           "note": "1 thread; the paper's Table 2 times 8192-element batches"}
            }, v, ns


def small_sets(wl) -> int:
    """Buffer sets the cold variant of a workload that fits in L2 rotates over."""
    return int(min(4096, max(3, -(-int(3 * L2_BYTES) // (wl.E * wl.bytes_per_element)))))


def config_for(wl, world: int) -> dict:
    """The `config` object of the JSON line; the same for both arms."""
    nbytes = wl.E * wl.bytes_per_element
    if nbytes > 2 * L2_BYTES:
        l2 = f"inputs larger than L2 ({nbytes / 1e9:.2f} GB per step)"
    elif world == 1 and wl.op == "inv_helmholtz" and wl.dtype == "f64":
        l2 = f"rotating over {small_sets(wl)} buffer sets (3 x L2) between calls"
    else:
        l2 = "working set fits in L2 (warm)"
    return {"workload": wl.name, "elements_per_gpu": wl.E, "l2": l2,
            "parallelism": f"elements sharded over {world} GPU(s), no collective"}


def reference_arm(args, wl, rank):
    """``--impl reference``: the oracle timed on the host cores, bounded sample per step."""
    if rank != 0:
        return
    import oracle
    probe = min(wl.E, 128)
    t_probe, _, _ = oracle_run(wl, 0, probe)
    budget = 90.0 / max(1, args.steps + args.warmup)            # whole run ~1.5 minutes
    ns = int(min(wl.E, max(32, probe / max(t_probe, 1e-6) * min(budget, 10.0))))
    from paper_2604_19906_b200 import inputs
    host = inputs.host_case(wl, 0, ns)

    def step():
        if wl.op == "inv_helmholtz":
            oracle.inv_helmholtz(host["S"], host["D"], host["u"])
        elif wl.op == "convection":
            oracle.convection(host["Dvq"], host["Ivq"], host["M"], host["P"])
        else:
            oracle.tpo_apply(host["A"], host["B"], host["C"], host["u"])

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    cores = oracle.threads_used(0)
    value = ns * args.steps / dt
    sample = f"first {ns} of {wl.E} elements of {wl.name} per step on {cores} threads"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": config_for(wl, int(os.environ.get("WORLD_SIZE", "1"))),
            "sample_elements_per_step": ns,
            "gflops": value * wl.flops_per_element / 1e9,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ GPU arm

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3)
    ap.add_argument("--elements", type=int, default=0, help="override E (profiling on small cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-probes", action="store_true",
                    help="skip the FP64-rate probes that run after the timed region")
    ap.add_argument("--context", action="store_true",
                    help="add the E = 8192 rows (the batch size of the paper's Table 2) for "
                         "n = 4, 8, 12, 14 to the line; on by default for the default workload "
                         "on one GPU")
    ap.add_argument("--no-context", action="store_true", help="leave those rows out")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2604_19906_b200 import inputs
    wl = inputs.CONFIGS[args.workload]
    if args.elements:
        wl = inputs.Workload(wl.index, wl.op, wl.n, wl.m, args.elements, wl.dtype)

    if args.impl == "reference":
        reference_arm(args, wl, rank)
        return

    # The oracle leg runs first, before any CUDA call (its OpenMP pool and the CUDA
    # context do not interact, and the GPUs are not held while the host works).
    base = None
    if rank == 0 and not args.no_cpu_baseline:
        # under torchrun the other ranks wait at the first barrier: keep the sample small there
        base, v_oracle, ns_oracle = cpu_baseline(wl, max_elements=None if world == 1 else 8192)

    import torch
    from paper_2604_19906_b200 import build, ops, sharding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if local_rank >= torch.cuda.device_count():
        raise SystemExit(f"LOCAL_RANK {local_rank} but only {torch.cuda.device_count()} GPU(s) visible")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        # one process per node (re)builds the in-tree libraries, the others wait for it
        if local_rank == 0:
            build.build()
        dist.barrier()
    else:
        dist = None
        build.build()
    if world != args.gpus and rank == 0:
        print(f"# note: --gpus {args.gpus} but WORLD_SIZE={world}", file=sys.stderr)

    lib = ops.library()
    e0, e1 = sharding.weak_range(wl.E, rank, world)
    case = inputs.device_case(wl, dev, e0, e1)
    E = wl.E
    if wl.op == "inv_helmholtz":
        v = torch.empty_like(case["u"])
        a = (case["S"].data_ptr(), case["D"].data_ptr(), case["u"].data_ptr(), v.data_ptr(),
             wl.n[0], E)
        fn = lib.ekl_tpo_inv_helmholtz if wl.dtype == "f64" else lib.ekl_tpo_inv_helmholtz_f32
    elif wl.op == "convection":
        v = torch.empty((3, E) + tuple(wl.m), dtype=torch.float64, device=dev)
        a = (case["Dvq"].data_ptr(), case["Ivq"].data_ptr(), case["M"].data_ptr(),
             case["P"].data_ptr(), v.data_ptr(), wl.n[0], wl.m[0], E)
        fn = lib.ekl_tpo_convection
        import ctypes as _ct
        fn.argtypes = [_ct.c_void_p] * 5 + [_ct.c_int, _ct.c_int, _ct.c_longlong, _ct.c_void_p]
        fn.restype = _ct.c_int
    else:
        v = torch.empty((E,) + tuple(wl.m), dtype=torch.float64, device=dev)
        a = (case["A"].data_ptr(), case["B"].data_ptr(), case["C"].data_ptr(),
             case["u"].data_ptr(), v.data_ptr(), *wl.n, *wl.m, E)
        fn = lib.ekl_tpo_apply
    stream = torch.cuda.Stream(dev)
    sp = stream.cuda_stream

    def step():
        st = fn(*a, sp)
        if st:
            raise ops.EklTpoError(st, "bench step")

    def barrier():
        if dist is not None:
            dist.barrier()

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step()
        torch.cuda.synchronize(dev)
        props = torch.cuda.get_device_properties(dev)
        sampler = ClockSampler(str(getattr(props, "uuid", "")), local_rank)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        per = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
        barrier()
        torch.cuda.synchronize(dev)
        sampler.start()
        ev0.record(stream)
        for k in range(args.steps):
            per[k][0].record(stream)
            step()
            per[k][1].record(stream)
        ev1.record(stream)
        torch.cuda.synchronize(dev)
        barrier()
        clocks = sampler.stop()
    total_ms = ev0.elapsed_time(ev1)
    launch_ms = [p[0].elapsed_time(p[1]) for p in per]
    if dist is not None:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * E / (ms_per_step * 1e-3)

    # ---------------------------------------------------------------- parity on the oracle's sample
    max_rel_err = None
    if base is not None:
        import oracle
        got = (v[:, :ns_oracle].permute(1, 0, 2, 3, 4).contiguous() if wl.op == "convection"
               else v[:ns_oracle]).cpu().numpy().astype(np.float64)
        max_rel_err = float(oracle.rel_err_per_element(got, v_oracle).max())

    # ---------------------------------------------------------------- FP64 rates of this device, live
    probe_rates = {}
    if rank == 0 and not args.no_probes:
        from paper_2604_19906_b200 import probes
        try:
            probe_rates = probes.run_probes(dev, stream)
        except Exception as exc:                      # a missing probe library is not fatal here
            probe_rates = {"error": str(exc)}

    # ---------------------------------------------------------------- small workloads: cold and graph
    small = None
    if rank == 0 and E * wl.bytes_per_element < 2 * L2_BYTES:
        small = small_workload_variants(torch, inputs, wl, fn, dev, stream, ops)
        if small is not None and world == 1:
            # the timed region above re-used one buffer set (warm L2); the headline of a
            # workload that fits in L2 is the cold figure, each call on another buffer set
            ms_per_step = small["cold_us"] / 1e3
            value = E / (ms_per_step * 1e-3)
            launch_ms = [ms_per_step]

    # ---------------------------------------------------------------- E = 8192 context rows
    context = None
    # (the rows time the oracle too, so --no-cpu-baseline leaves them out as well)
    default_run = (world == 1 and args.workload == 3 and not args.elements
                   and not args.no_cpu_baseline)
    if rank == 0 and not args.no_context and (args.context or default_run):
        context = context_rows(torch, inputs, ops, dev, stream)

    # ---------------------------------------------------------------- end to end with host buffers
    e2e = None
    if not args.no_e2e and wl.op != "convection":
        e2e = run_e2e(torch, ops, wl, case, dev, stream, args.e2e_steps, world, dist)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_src = measured_peaks()
    traffic_pe = ncu_traffic_bytes_per_element(wl.index)
    avg_launch_ms = statistics.fmean(launch_ms)
    flops_launch = E * wl.flops_per_element
    bytes_launch = E * wl.bytes_per_element
    tf = flops_launch / (avg_launch_ms * 1e-3) / 1e12
    gbs = bytes_launch / (avg_launch_ms * 1e-3) / 1e9
    hbm_peak = float(peaks.get("hbm_gbs", HBM_FALLBACK_GBS))
    t_alu = flops_launch / (FP64_PEAK_TFLOPS * 1e12)
    t_hbm = bytes_launch / (hbm_peak * 1e9)
    if wl.dtype == "f32":
        # single precision runs on the TF32 tensor path, three tensor steps per product; its
        # peak is the measured bf16 figure times the nominal tf32/bf16 ratio (1.1/2.25)
        tf32_peak = float(peaks.get("bf16_tflops", 1590.0)) * (1.1 / 2.25)
        t_alu = 3.0 * flops_launch / (tf32_peak * 1e12)
    if wl.dtype == "f32" and t_alu >= t_hbm:
        roof = {"bound": "tensor", "achieved": 3.0 * tf, "peak": tf32_peak, "unit": "TFLOP/s",
                "frac": 3.0 * tf / tf32_peak}
    elif t_alu >= t_hbm:
        roof = {"bound": "alu", "achieved": tf, "peak": FP64_PEAK_TFLOPS, "unit": "TFLOP/s",
                "frac": tf / FP64_PEAK_TFLOPS}
    else:
        roof = {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s",
                "frac": gbs / hbm_peak}
    roof.update({
        "traffic": (traffic_pe * E if traffic_pe is not None else None),
        "traffic_note": "bytes per launch: ncu dram read+write per element "
                        "(profiles/dram_traffic.json) x E; null if there is no capture of the "
                        "current kernel sources",
        "algorithmic_bytes": bytes_launch, "algorithmic_flops": flops_launch,
        "kernel_ms": avg_launch_ms,
        "peak_source": ("alu: 148 SMs x 64 FP64 FMA/clk x 2 x 1.965 GHz; hbm: "
                        f"MEASURED_PEAKS.json ({peak_src})" if wl.dtype == "f64" else
                        f"hbm: MEASURED_PEAKS.json ({peak_src}); tensor: bf16 x 1.1/2.25, "
                        "three TF32 steps per product"),
        "fp64_tflops": tf, "fp64_peak_derived": FP64_PEAK_TFLOPS,
        "fp64_peak_probe_tflops": probe_rates.get("fma_chain"),
        "fp64_peak_probe_dfma_tflops": probe_rates.get("fma_contraction"),
        "fp64_peak_probe_dmma_tflops": probe_rates.get("dmma_2chains"),
        "fp64_peak_probe_dmma_plus_fma_tflops": probe_rates.get("dmma_plus_fma"),
        "stage_loop_n14_dmma_tflops": probe_rates.get("stage_loop_n14_dmma"),
        "stage_loop_n14_dmma_padded_tflops": probe_rates.get("stage_loop_n14_dmma_padded"),
        "stage_loop_n14_fma_tflops": probe_rates.get("stage_loop_n14_fma"),
        "nominal": {"hbm_gbs": NOMINAL_HBM_GBS, "fp64_tflops": NOMINAL_FP64_TFLOPS,
                    "min_roof_ms": max(flops_launch / (NOMINAL_FP64_TFLOPS * 1e12),
                                       bytes_launch / (NOMINAL_HBM_GBS * 1e9)) * 1e3,
                    "frac_of_min_roof": max(flops_launch / (NOMINAL_FP64_TFLOPS * 1e12),
                                            bytes_launch / (NOMINAL_HBM_GBS * 1e9)) * 1e3
                    / avg_launch_ms} if wl.dtype == "f64" else None,
        "hbm_gbs": gbs, "hbm_peak_gbs": hbm_peak, "hbm_frac": gbs / hbm_peak,
        "min_roof_ms": max(t_alu, t_hbm) * 1e3,
        "frac_of_min_roof": max(t_alu, t_hbm) * 1e3 / avg_launch_ms})
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": config_for(wl, world),
            "gflops": value * wl.flops_per_element / 1e9,
            "roofline": roof, "clocks": clocks, "gpu_launches": args.steps,
            "max_rel_err_vs_oracle": max_rel_err}
    if base is not None:
        line["cpu_baseline"] = base
    if e2e is not None:
        line["e2e"] = e2e
    if small is not None:
        line["small_workload"] = small
    if context is not None:
        line["paper_batch_8192"] = context
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def _event_ms(torch, stream, fn_once, reps):
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    for k in range(reps):
        fn_once(k)
    s1.record(stream)
    stream.synchronize()
    return s0.elapsed_time(s1) / reps


def small_workload_variants(torch, inputs, wl, fn, dev, stream, ops, reps=200):
    """For a workload whose working set fits in L2 (configurations 0 and 1): microseconds per
    call (a) warm, the same buffers every call, (b) cold, rotating over enough distinct buffer
    sets to exceed three times the L2, (c) warm, replayed from a CUDA graph of 20 calls.  At
    this size the call is at the scale of the launch path, not of either roof."""
    if wl.op != "inv_helmholtz" or wl.dtype != "f64":
        return None
    n, E = wl.n[0], wl.E
    base = inputs.device_case(wl, dev)
    set_bytes = E * wl.bytes_per_element
    sets = small_sets(wl)
    us = [base["u"]] + [base["u"].clone() for _ in range(sets - 1)]
    Ds = [base["D"]] + [base["D"].clone() for _ in range(sets - 1)]
    vs = [torch.empty_like(base["u"]) for _ in range(sets)]
    sp = stream.cuda_stream

    def call(k):
        st = fn(base["S"].data_ptr(), Ds[k].data_ptr(), us[k].data_ptr(), vs[k].data_ptr(), n, E, sp)
        if st:
            raise ops.EklTpoError(st, "small workload step")

    out = {"sets": sets, "bytes_per_set": set_bytes, "calls": reps}
    with torch.cuda.stream(stream):
        for k in range(sets):
            call(k)
        stream.synchronize()
        out["warm_us"] = 1e3 * _event_ms(torch, stream, lambda k: call(0), reps)
        out["cold_us"] = 1e3 * _event_ms(torch, stream, lambda k: call(k % sets), reps)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(20):
                call(0)
        graph.replay()
        stream.synchronize()
        out["graph_us"] = 1e3 * _event_ms(torch, stream, lambda k: graph.replay(), 10) / 20
    flops, nbytes = E * wl.flops_per_element, set_bytes
    peaks, _ = measured_peaks()
    roof_us = 1e6 * max(flops / (FP64_PEAK_TFLOPS * 1e12),
                        nbytes / (float(peaks.get("hbm_gbs", HBM_FALLBACK_GBS)) * 1e9))
    out["roofline_us"] = roof_us
    out["cold_frac_of_roof"] = roof_us / out["cold_us"]
    out["note"] = "latency-limited: the roofline time is below the cost of one kernel launch"
    return out


def context_rows(torch, inputs, ops, dev, stream, reps=50):
    """E = 8192 (the batch the paper's Table 2 measures on) at n = 4, 8, 12, 14, fp64 inverse
    Helmholtz: milliseconds per call (rotating over buffer sets larger than L2) and the
    oracle on one host thread beside it."""
    import oracle
    rows = []
    lib = ops.library()
    for n in (4, 8, 12, 14):
        wl = inputs.Workload(1, "inv_helmholtz", (n, n, n), (n, n, n), 8192, "f64")
        base = inputs.device_case(wl, dev)
        set_bytes = wl.E * wl.bytes_per_element
        sets = int(max(2, -(-int(3 * L2_BYTES) // set_bytes)))
        us = [base["u"]] + [base["u"].clone() for _ in range(sets - 1)]
        Ds = [base["D"]] + [base["D"].clone() for _ in range(sets - 1)]
        v = torch.empty_like(base["u"])
        sp = stream.cuda_stream

        def call(k):
            st = lib.ekl_tpo_inv_helmholtz(base["S"].data_ptr(), Ds[k % sets].data_ptr(),
                                           us[k % sets].data_ptr(), v.data_ptr(), n, wl.E, sp)
            if st:
                raise ops.EklTpoError(st, "context row")

        with torch.cuda.stream(stream):
            for k in range(sets):
                call(k)
            stream.synchronize()
            ms = _event_ms(torch, stream, call, reps)
        host = inputs.host_case(wl, 0, wl.E)
        oracle.inv_helmholtz(host["S"], host["D"], host["u"], 1)
        t0 = time.perf_counter()
        oracle.inv_helmholtz(host["S"], host["D"], host["u"], 1)
        t1 = time.perf_counter() - t0
        rows.append({"n": n, "E": wl.E, "ms": ms, "elements_per_s": wl.E / (ms * 1e-3),
                     "gflops": wl.E * wl.flops_per_element / (ms * 1e-3) / 1e9,
                     "oracle_1thread_ms": t1 * 1e3,
                     "oracle_1thread_elements_per_s": wl.E / t1})
    return rows


def run_e2e(torch, ops, wl, case, dev, stream, steps, world, dist):
    """Same metric through the public API with HOST buffers: every step copies u and D
    from pinned host memory, runs the operator, and copies v back."""
    E = wl.E
    names = ("D", "u") if wl.op == "inv_helmholtz" else ("u",)
    host_in = {k: torch.empty(case[k].shape, dtype=case[k].dtype, pin_memory=True).copy_(case[k])
               for k in names}
    out_shape = (E,) + tuple(wl.m)
    host_out = torch.empty(out_shape, dtype=case["u"].dtype, pin_memory=True)
    mats = {k: case[k].cpu() for k in (("S",) if wl.op == "inv_helmholtz" else ("A", "B", "C"))}
    torch.cuda.synchronize(dev)

    def step():
        if wl.op == "inv_helmholtz":
            ops.ekl_tpo_inv_helmholtz_host(mats["S"], host_in["D"], host_in["u"], host_out,
                                           device=dev)
        else:
            ops.ekl_tpo_apply_host(mats["A"], mats["B"], mats["C"], host_in["u"], host_out,
                                   device=dev)

    with torch.cuda.stream(stream):
        step()
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(steps):
            step()
        torch.cuda.synchronize(dev)
        dt = time.perf_counter() - t0
    if dist is not None:
        t = torch.tensor([dt], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dt = float(t.item())
    h2d = sum(t.numel() * t.element_size() for t in host_in.values()) + \
        sum(t.numel() * t.element_size() for t in mats.values())
    d2h = host_out.numel() * host_out.element_size()
    return {"value": world * E * steps / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": dt / steps * 1e3, "steps": steps,
            "api": "ekl_tpo_*_host (pinned host buffers in, pinned host buffer out)"}


if __name__ == "__main__":
    main()
