#!/usr/bin/env python
"""Benchmark of the condensed constant-fan-in linear forward.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one cfi_forward over one batch of the headline workload: the 768 -> 3072, k = 77 (90 % sparse)
fp32 layer at batch 256.  Prints ONE JSON line: effective GFLOP/s (2 * B * n_active * k / t), ms per step,
the roofline object for the forward kernel, an end-to-end number with host buffers, the CPU oracle timed
on this host as a reported baseline, and the batch-1 (online inference) numbers next to it.

Timing: steps run as replays of a CUDA graph that holds the launches back to back, between CUDA events on
the launching stream; consecutive steps use different replicas of the layer and of x / y whose total size
exceeds twice the L2, so every step streams its operands from HBM.  With N > 1 (torchrun) every rank runs
the same workload on its own GPU and its own batches (no exchange step exists in this path), the time is
the maximum over ranks and the value the sum of all ranks' work.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2305_02299_b200 import inputs  # noqa: E402

METRIC = "cfi_forward effective GFLOP/s (2*B*n_active*k/t), 768->3072 k=77 fp32, batch 256"
FMA_LANES_PER_SM = 128      # fp32 FMA lanes per SM
L2_BYTES_FALLBACK = 126 * 1024 * 1024


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


def algorithmic_bytes(w: inputs.Workload, n_active: int, elem: int = 4) -> int:
    """values + int32 indices once, x once, y once, bias and the active-row list."""
    return n_active * w.k * (elem + 4) + w.batch * w.in_features * elem + w.batch * w.out_features * elem \
        + w.out_features * 4 + n_active * 4


def algorithmic_flops(w: inputs.Workload, n_active: int) -> int:
    return 2 * w.batch * n_active * w.k


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while a region runs."""
    _REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], set()
        self.max_mhz, self._stop, self._thr, self._h = None, threading.Event(), None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and vis.split(",")[index].isdigit() else index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _once(self):
        nv = self._nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
        try:
            mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
        except Exception:
            mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
        for bit, name in self._REASONS.items():
            if mask & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------------
# device-side timing
# --------------------------------------------------------------------------------------------------
class Replicas:
    """R independent copies of (layer, x, y) so that consecutive steps touch different memory."""

    def __init__(self, w: inputs.Workload, cfi, torch, min_total_bytes: int, dtype: str = "f32", seed: int = 0,
                 rank: int = 0, max_replicas: int = 64, layer=None, packed=None, layouts: int = 7, streamed_bytes=None):
        self.w, self.cfi, self.torch = w, cfi, torch
        tdt = torch.float32 if dtype == "f32" else torch.bfloat16
        base = layer if layer is not None else w.layer(seed=seed, replica=0)
        v, ix, rows = packed if packed is not None else cfi.cfi_pack(base.w_dense, base.mask)
        self.n_active = int(rows.shape[0])
        elem = 4 if dtype == "f32" else 2
        self.bytes_per_step = algorithmic_bytes(w, self.n_active, elem)
        # What one call streams from memory decides how many replicas make the rotation cold: the condensed arrays
        # and activations, or more when the kernel in use reads the dense copy.
        per = max(self.bytes_per_step, streamed_bytes or 0)
        self.R = int(max(2, min(max_replicas, -(-min_total_bytes // per))))
        self.layers, self.x, self.y = [], [], []
        rng = np.random.default_rng(1234 + rank)
        for r in range(self.R):
            # Same structure statistics, different numbers: permute rows of the base layer's condensed arrays
            # (cheap) instead of drawing a fresh dense matrix per replica.
            p = rng.permutation(self.n_active)
            self.layers.append(cfi.cfi_create(v[p], ix[p], rows, base.bias, w.in_features, w.out_features,
                                              dtype=dtype, act=w.act, layouts=layouts))
            xr = w.x(seed=seed, replica=r + 100 * rank)
            self.x.append(torch.from_numpy(xr).to("cuda", tdt).contiguous())
            self.y.append(torch.empty((w.batch, w.out_features), device="cuda", dtype=tdt))
        self.total_bytes = self.R * per
        self.layouts = layouts

    def step(self, i: int, variant: str = "auto"):
        r = i % self.R
        self.cfi.cfi_forward_variant(self.layers[r], self.x[r], self.y[r], self.w.batch, variant=variant)

    def close(self):
        for l in self.layers:
            l.close()


def time_steps(rep: Replicas, torch, steps: int, warmup: int, variant: str = "auto", graph_len: int = 1000,
               barrier=None, sampler=None, target_s: float = 0.25, max_passes: int = 5000):
    """Times passes of exactly `steps` steps each (CUDA-graph replays between CUDA events on the launching stream)
    and returns a dict: median and standard deviation of the per-step time over the passes, the number of passes,
    the launches of one pass.  A short pass (few steps) is repeated until about `target_s` seconds have been timed,
    at least five times, so that the figure is a steady-state one and the clock sampler sees the region.
    Warm-up covers every replica at least once."""
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            rep.step(i, variant)
        for i in range(rep.R):
            rep.step(i, variant)
        stream.synchronize()
        g_len = max(1, min(graph_len, steps))
        n_replay, rem = divmod(steps, g_len)
        graphs = []
        for length in ([g_len] if n_replay else []) + ([rem] if rem else []):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(length):
                    rep.step(i, variant)
            graphs.append(g)
        main = graphs[0] if n_replay else None
        tail = graphs[-1] if rem else None

        def one_pass():
            for _ in range(n_replay):
                main.replay()
            if tail is not None:
                tail.replay()

        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        one_pass()                  # graph upload
        stream.synchronize()
        a.record(stream)
        one_pass()                  # untimed estimate of a pass
        b.record(stream)
        b.synchronize()
        est = max(a.elapsed_time(b) * 1e-3, 1e-6)
        passes = int(min(max_passes, max(5, -(-target_s // est))))
        if barrier:
            barrier()
        torch.cuda.synchronize()
        events = [torch.cuda.Event(enable_timing=True) for _ in range(passes + 1)]
        ctx = sampler if sampler is not None else _Null()
        with ctx:
            events[0].record(stream)
            for p in range(passes):
                one_pass()
                events[p + 1].record(stream)
            events[-1].synchronize()
        torch.cuda.synchronize()
        if barrier:
            barrier()
    per_pass = [events[p].elapsed_time(events[p + 1]) * 1e-3 for p in range(passes)]
    return {"sec_per_step": statistics.median(per_pass) / steps, "std_sec_per_step": statistics.pstdev(per_pass) / steps,
            "passes": passes, "steps_per_pass": steps, "launches_per_pass": steps,
            "timed_s": events[0].elapsed_time(events[-1]) * 1e-3}


def us(t):
    """Per-step microseconds of a time_steps result."""
    return t["sec_per_step"] * 1e6


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def time_e2e(rep: Replicas, torch, steps: int, warmup: int):
    """Through cfi_forward_host: pinned host x -> device, forward, y -> pinned host, every step.  The warm-up calls
    every replica once, so each layer's staging buffers exist before the timed region starts (the entry point
    allocates them on a layer's first call)."""
    w = rep.w
    tdt = rep.x[0].dtype
    xh = [rep.x[r].cpu().pin_memory() for r in range(min(rep.R, 8))]
    yh = torch.empty((w.batch, w.out_features), dtype=tdt).pin_memory()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(max(3, warmup, rep.R)):
            rep.cfi.cfi_forward_host(rep.layers[i % rep.R], xh[i % len(xh)], yh, w.batch)
        torch.cuda.synchronize()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(stream)
        for i in range(steps):
            rep.cfi.cfi_forward_host(rep.layers[i % rep.R], xh[i % len(xh)], yh, w.batch)
        end.record(stream)
        end.synchronize()
    sec = start.elapsed_time(end) * 1e-3
    return sec, xh[0].numel() * xh[0].element_size(), yh.numel() * yh.element_size()


# --------------------------------------------------------------------------------------------------
# CPU oracle timing (reported baseline, and the --impl reference arm)
# --------------------------------------------------------------------------------------------------
def time_oracle(w: inputs.Workload, budget_s: float, sample_rows=None, threads=None, packed=None, layer=None):
    """The oracle as it stands on this host, on the first `sample_rows` batch rows of the workload (all of them by
    default, fewer if one call would take longer than the budget): median seconds per call and the flops of a call."""
    import oracle
    L = layer if layer is not None else w.layer(seed=0)
    v, ix, rows = packed if packed is not None else oracle.pack(L.w_dense, L.mask)
    x = w.x(seed=0)
    all_threads = oracle.max_threads()
    if threads:
        oracle.set_threads(threads)
    try:
        n = w.batch if sample_rows is None else min(sample_rows, w.batch)
        t0 = time.perf_counter()
        oracle.forward(v, ix, rows, L.bias, w.in_features, w.out_features, x[:1], act=w.act)
        per_row = max(time.perf_counter() - t0, 1e-7)
        n = int(max(1, min(n, budget_s / 5.0 / per_row)))          # at least five calls fit the budget
        xs = np.ascontiguousarray(x[:n])
        call = lambda: oracle.forward(v, ix, rows, L.bias, w.in_features, w.out_features, xs, act=w.act)
        call()
        t0 = time.perf_counter()
        call()
        one = time.perf_counter() - t0
        repeats = int(max(5, min(2000, budget_s / max(one, 1e-6))))
        times = []
        for _ in range(repeats):
            t0 = time.perf_counter()
            call()
            times.append(time.perf_counter() - t0)
    finally:
        oracle.set_threads(all_threads)
    return {"median_s": statistics.median(times), "std_s": statistics.pstdev(times), "flops": 2 * n * rows.shape[0] * w.k,
            "calls": repeats, "rows": n, "cores": threads or all_threads}


def config_keys(w, n_active):
    """The keys both arms print under `config`: they name the workload and nothing else."""
    return {"workload": w.name, "in": w.in_features, "out": w.out_features, "k": w.k, "n_active": int(n_active), "batch": w.batch}


def run_reference(args, w):
    """The oracle as it stands on the host cores; each step is one forward over a bounded sample of the batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    total = args.steps + args.warmup
    L = w.layer(seed=0)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    x = w.x(seed=0)
    t0 = time.perf_counter()
    oracle.forward(v, ix, rows, L.bias, w.in_features, w.out_features, x[:8])
    per_row = max((time.perf_counter() - t0) / 8, 1e-7)
    sample = int(max(1, min(w.batch, (120.0 / max(total, 1)) / per_row)))
    xs = np.ascontiguousarray(x[:sample])
    for _ in range(args.warmup):
        oracle.forward(v, ix, rows, L.bias, w.in_features, w.out_features, xs)
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        oracle.forward(v, ix, rows, L.bias, w.in_features, w.out_features, xs)
        times.append(time.perf_counter() - t0)
    sec = sum(times)
    gflops = 2 * sample * rows.shape[0] * w.k * args.steps / sec / 1e9
    cores = oracle.max_threads()
    desc = f"{sample} of {w.batch} batch rows per step, all {w.out_features} output rows"
    line = {"impl": "reference", "metric": METRIC, "value": gflops, "unit": "GFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_keys(w, rows.shape[0]),
            "cpu_baseline": {"value": gflops, "unit": "GFLOP/s", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": gflops, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--variant", default="auto")
    ap.add_argument("--no-extras", action="store_true", help="skip the batch-1 and CPU-baseline legs")
    ap.add_argument("--target-s", type=float, default=0.25,
                    help="seconds of timed passes to aim for (at least five passes are always timed); small values for profiler runs")
    ap.add_argument("--stack-only", type=int, default=0, metavar="ROWS",
                    help="run only the bf16 MLP stack leg on ROWS batch rows (for profiling) and print its JSON")
    ap.add_argument("--sweep-only", default=None, metavar="NAMES",
                    help="run only the floor probe and the sweep over these named workloads (comma separated; 'all') and print its JSON")
    ap.add_argument("--srigl-only", action="store_true",
                    help="run only the SRigL mask-update leg (for profiling) and print its JSON")
    args = ap.parse_args()
    W = inputs.workloads()
    w = W[args.workload]

    if args.impl == "reference":
        args.steps = 20 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        run_reference(args, w)
        return
    args.steps = 20000 if args.steps is None else args.steps
    args.warmup = 20 if args.warmup is None else args.warmup

    import torch
    from paper_2305_02299_b200 import binding as cfi   # raises if the CUDA library is missing

    if args.srigl_only:
        torch.cuda.set_device(0)
        peaks, _ = measured_peaks()
        print(json.dumps(srigl_update_leg(cfi, torch, peaks)))
        return
    if args.sweep_only:
        torch.cuda.set_device(0)
        peaks, kind = measured_peaks()
        props = torch.cuda.get_device_properties(0)
        l2 = getattr(props, "L2_cache_size", None) or L2_BYTES_FALLBACK
        only = None if args.sweep_only == "all" else set(args.sweep_only.split(","))
        floor = floor_leg(cfi, torch, l2)
        print(json.dumps({"floor": floor, "sweep": sweep_leg(W, cfi, torch, l2, Ceilings(peaks, kind, props.multi_processor_count),
                                                               floor, only=only, cpu=False)}))
        return
    if args.stack_only:
        torch.cuda.set_device(0)
        peaks, _ = measured_peaks()
        print(json.dumps(stack_leg(cfi, torch, peaks, torch.cuda.get_device_properties(0).multi_processor_count,
                                   rows=args.stack_only, blocks=1)))
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    barrier = (lambda: dist.barrier()) if dist else None

    peaks, peak_kind = measured_peaks()
    props = torch.cuda.get_device_properties(local)
    l2 = getattr(props, "L2_cache_size", None) or L2_BYTES_FALLBACK
    sm_count = props.multi_processor_count
    ceil_ = Ceilings(peaks, peak_kind, sm_count)

    rep = Replicas(w, cfi, torch, 2 * l2 + (32 << 20), rank=rank)
    sampler = ClockSampler(local)
    timed = time_steps(rep, torch, args.steps, args.warmup, args.variant, barrier=barrier, sampler=sampler, target_s=args.target_s)
    per_call = max_over_ranks(timed["sec_per_step"], dist, "cuda")
    flops = algorithmic_flops(w, rep.n_active)
    value = whole_job_value(flops, world, per_call)

    # End to end through the host-buffer entry point (each rank on its own GPU).
    e2e_steps = int(min(max(args.steps, 200), 2000)) if args.target_s >= 0.25 else 8
    e2e_sec, h2d, d2h = time_e2e(rep, torch, e2e_steps, 5)
    e2e_sec = max_over_ranks(e2e_sec, dist, "cuda")
    e2e_value = whole_job_value(flops, world, e2e_sec / e2e_steps)

    line = None
    if rank == 0:
        achieved_tflops = flops / per_call / 1e12
        hbm_gbs = rep.bytes_per_step / per_call / 1e9
        info = cfi.cfi_layer_info(rep.layers[0])
        chosen = VARIANT_NAMES[cfi.cfi_choose_variant(rep.layers[0], w.batch)] if args.variant == "auto" else args.variant
        shape = dense_shape(cfi, rep.layers[0], w.batch) if chosen == "dense_tc" else None
        line = {
            "metric": METRIC, "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": per_call * 1e3, "us_per_call": per_call * 1e6,
            "us_per_call_std": timed["std_sec_per_step"] * 1e6, "timed_passes": timed["passes"], "timed_s": timed["timed_s"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(config_keys(w, rep.n_active), variant=chosen, dense_shape=shape,
                           l2=f"inputs larger than L2: {rep.R} rotating replicas of layer+x+y, "
                              f"{rep.total_bytes / 1e6:.0f} MB vs L2 {l2 / 1e6:.0f} MB",
                           timing=f"{timed['passes']} passes of {args.steps} steps each (CUDA-graph replays between CUDA events "
                                  "on the launching stream); ms_per_step is the median pass / steps"),
            "roofline": {"bound": "alu", "achieved": achieved_tflops, "peak": ceil_.fma_tflops, "unit": "TFLOP/s",
                         "frac": achieved_tflops / ceil_.fma_tflops,
                         # dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu capture summarised
                         # under profiles/ for exactly this kernel and launch shape; null otherwise
                         "traffic": CAPTURED_TRAFFIC.get((w.name, kernel_name(chosen, shape), json.dumps(shape))),
                         "peak_source": ceil_.fma_source,
                         "kernel": kernel_name(chosen, shape),
                         "note": "bound/peak are the sparse problem's own roofline (2*B*n_active*k FMAs on the fp32 FMA "
                                 "pipes, the bound of the gather formulation; its shared-memory ceiling is given beside "
                                 "it); when the chosen kernel is the tensor-core variant the dense flops it executes are "
                                 "given under tensor_*",
                         "smem_ceiling_tflops": ceil_.smem_tflops, "smem_ceiling_frac": achieved_tflops / ceil_.smem_tflops,
                         "hbm_achieved_gbs": hbm_gbs, "hbm_peak_gbs": peaks["hbm_gbs"],
                         "hbm_frac": hbm_gbs / peaks["hbm_gbs"], "hbm_peak_source": f"{peak_kind} copy bandwidth",
                         "algorithmic_bytes": rep.bytes_per_step, "algorithmic_flops": flops,
                         "weight_bytes_streamed_per_batch_tile": int(info.weight_bytes_batch)},
            "variants_us": {},
            "e2e": {"value": e2e_value, "unit": "GFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "us_per_call": e2e_sec / e2e_steps * 1e6, "calls_timed": e2e_steps, "api": "cfi_forward_host",
                    "note": "every replica's staging buffers exist before the timed region"},
            "gpu_launches": timed["launches_per_pass"],
            "clocks": sampler.summary(),
        }
        if chosen == "dense_tc":
            dense = 3 * 2.0 * w.batch * w.out_features * w.in_features   # three TF32 products per fp32 product
            tf32_peak = peaks["bf16_tflops"] * 0.5                      # nominal TF32 : bf16 ratio on the measured bf16 peak
            line["roofline"].update({"tensor_executed_tflops": dense / per_call / 1e12, "tensor_peak_tflops": tf32_peak,
                                     "tensor_frac": dense / per_call / 1e12 / tf32_peak,
                                     "tensor_peak_source": f"{peak_kind} bf16 matmul peak x 0.5 (nominal TF32:bf16)"})
        if world == 1 and not args.no_extras:
            for v in ("batch", "dense_tc"):
                try:
                    line["variants_us"][v] = us(time_steps(rep, torch, 2000, 10, v, target_s=0.05))
                except Exception as exc:  # a variant that cannot run this shape
                    line["variants_us"][v] = str(exc)
    rep.close()

    if rank == 0 and world == 1 and not args.no_extras:
        line["floor"] = floor_leg(cfi, torch, l2)
        line["sweep"] = sweep_leg(W, cfi, torch, l2, ceil_, line["floor"])
        line["batch1"] = {k: v for k, v in line["sweep"].items() if k in W and W[k].batch == 1}
        cb = time_oracle(w, budget_s=10.0)
        c1 = time_oracle(w, budget_s=10.0, threads=1)
        line["cpu_baseline"] = {"value": cb["flops"] / cb["median_s"] / 1e9, "unit": "GFLOP/s", "cores": cb["cores"],
                                "kind": "oracle", "us_per_call": cb["median_s"] * 1e6, "us_per_call_std": cb["std_s"] * 1e6,
                                "sample": f"{cb['rows']} of {w.batch} batch rows per call, median of {cb['calls']} calls",
                                "one_thread": {"value": c1["flops"] / c1["median_s"] / 1e9, "unit": "GFLOP/s", "cores": 1,
                                               "us_per_call": c1["median_s"] * 1e6,
                                               "sample": f"{c1['rows']} of {w.batch} batch rows per call, median of {c1['calls']} calls"}}
        line["context"] = context_leg(W, torch)
        line["stack_c5"] = stack_leg(cfi, torch, peaks, sm_count)
        line["batch2048"] = batch2048_leg(W, cfi, torch, l2, peaks, sm_count)
        # Ceilings measured in this run by the library's own micro-probes (fp32 FMA, L2 read, empty launch).
        try:
            line["device_probe"] = cfi.cfi_probe_device().as_dict()
        except Exception as exc:
            line["device_probe"] = str(exc)
        line["stack_batch1"] = stack_batch1_leg(cfi, torch, l2, peaks)
        line["srigl_update"] = srigl_update_leg(cfi, torch, peaks)
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


VARIANT_NAMES = {1: "simple", 2: "splitk", 3: "batch", 4: "dense_tc", 5: "slab"}
# DRAM bytes (read + written) of one launch from an ncu capture, keyed by (workload, kernel, launch shape); see profiles/.
CAPTURED_TRAFFIC = {
    # profiles/cfi_dense_split_kernel_c2_768x3072_k77_b256.md: 10.307 MB read (dense copy + x), 0 written (y still in L2)
    ("c2", "cfi_dense_split_kernel<96>", json.dumps({"batch_tile": 96, "cluster_k_split": 2})): 10.307e6,
}


def dense_shape(cfi, layer, batch):
    tile, cluster = cfi.cfi_dense_tile_shape(layer, batch)
    return {"batch_tile": tile, "cluster_k_split": cluster}


def kernel_name(variant, shape=None, dtype="f32"):
    if variant == "dense_tc":
        return f"cfi_dense_split_kernel<{shape['batch_tile']}>" if shape else "cfi_dense_split_kernel"
    return {"batch": "cfi_batch_kernel<float>", "splitk": "cfi_splitk_kernel<float>", "simple": "cfi_simple_kernel<float>",
            "slab": "cfi_slab_kernel<float>"}[variant]


class Ceilings:
    """The denominators: fp32 FMA peak derived from the unit counts and the maximum clock, the measured shared-memory
    gather ceiling of the gather formulation (25.5 FMA per clock and SM: one 4-byte gather per FMA at 128 bytes per
    clock, measured with a stand-alone copy of the inner loop), and the measured copy bandwidth."""

    def __init__(self, peaks, peak_kind, sm_count):
        self.sm_mhz = float(peaks.get("sm_max_mhz", 1965.0))
        self.fma_tflops = sm_count * FMA_LANES_PER_SM * 2 * self.sm_mhz * 1e6 / 1e12
        self.fma_source = f"{sm_count} SMs x {FMA_LANES_PER_SM} fp32 FMA lanes x 2 x {self.sm_mhz:.0f} MHz"
        self.smem_tflops = sm_count * 25.5 * 2 * self.sm_mhz * 1e6 / 1e12
        self.hbm_gbs = float(peaks["hbm_gbs"])
        self.peak_kind = peak_kind


def max_over_ranks(seconds: float, dist, device) -> float:
    """Device time of a multi-rank run: the slowest rank's (all-reduce MAX over the process group)."""
    if dist is None:
        return seconds
    import torch
    t = torch.tensor([seconds], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flops_per_rank_step: float, world: int, seconds_per_step: float) -> float:
    """GFLOP/s of all ranks together: every rank runs the same workload on its own batches (weak scaling)."""
    return flops_per_rank_step * world / seconds_per_step / 1e9


def _time_torch(fn, torch, iters=200):
    for _ in range(10):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    b.synchronize()
    return a.elapsed_time(b) * 1e-3 / iters


def context_leg(W, torch):
    """Library routines on the same masked weights, as context (not a target): cuBLAS dense through torch.matmul on
    the full masked weight, cuBLAS dense on the active rows only (the "structured" representation of Sec. 4.4: neuron
    ablation alone), cuSPARSE CSR through torch's sparse matmul.  Warm (one layer), eager launches."""
    out = {}
    for name in ("c2", "c3_b256"):
        w = W[name]
        L = w.layer(seed=0)
        wd = torch.from_numpy(L.w_dense * L.mask).cuda()
        active = np.setdiff1d(np.arange(w.out_features), L.ablated)
        wa = wd[torch.from_numpy(active).cuda()].contiguous()
        csr = wd.to_sparse_csr()
        for batch in (w.batch, 1):
            x = torch.from_numpy(w.x(seed=0, batch=batch)).cuda()
            xt = x.t().contiguous()
            out[f"{name.split('_')[0]}_b{batch}"] = {
                "cublas_dense_us": _time_torch(lambda: torch.matmul(x, wd.t()), torch) * 1e6,
                "cublas_dense_active_rows_us": _time_torch(lambda: torch.matmul(x, wa.t()), torch) * 1e6,
                "cusparse_csr_us": _time_torch(lambda: torch.matmul(csr, xt), torch) * 1e6,
                "active_rows": int(active.size), "rows": w.out_features}
    out["note"] = "torch.matmul (cuBLAS fp32, TF32 off) on all rows and on the active rows only, torch CSR matmul (cuSPARSE); " \
                  "warm, eager; paper: 1.7x / 13.0x faster than dense / CSR at batch 256 on a Titan V, 3.4x / 2.5x on a " \
                  "Xeon W-2145 at batch 1"
    return out


def stack_leg(cfi, torch, peaks, sm_count, rows=None, blocks=12):
    """The bf16 MLP stack (12 blocks of 768 -> 3072 GELU -> 768, 5 % of rows ablated, 50,432 rows)."""
    s = inputs.StackWorkload(blocks=blocks) if rows is None else inputs.StackWorkload(blocks=blocks, batch=rows)
    layers, flops, bytes_ = [], 0, 0
    for L, sp in zip(s.layers(seed=0), s.layer_specs()):
        v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
        layers.append(cfi.cfi_create(v, ix, rows, L.bias, sp[0], sp[1], dtype="bf16", act=sp[4]))
        flops += 2 * s.batch * rows.shape[0] * sp[2]
        bytes_ += rows.shape[0] * sp[2] * 6 + s.batch * (sp[0] + sp[1]) * 2 + sp[1] * 4
    stack = cfi.cfi_stack_create(layers, s.batch)
    x = torch.from_numpy(s.x(seed=0)).to("cuda", torch.bfloat16)
    y = torch.empty((s.batch, s.d_model), device="cuda", dtype=torch.bfloat16)
    sec = _time_torch(lambda: cfi.cfi_stack_forward(stack, x, y, s.batch), torch, iters=5)
    stack.close()
    for l in layers:
        l.close()
    fma_peak = sm_count * FMA_LANES_PER_SM * 2 * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
    return {"ms_per_pass": sec * 1e3, "layers": len(layers), "rows": s.batch, "dtype": "bf16",
            "effective_tflops": flops / sec / 1e12, "fma_frac": flops / sec / 1e12 / fma_peak,
            "algorithmic_bytes": bytes_, "hbm_frac": bytes_ / sec / 1e9 / peaks["hbm_gbs"],
            "l2": "activations of one layer (388 MB) exceed L2"}


def batch2048_leg(W, cfi, torch, l2, peaks, sm_count):
    """The headline layer at batch 2048, the largest batch of the paper's GPU figures (appendix, condensed
    GPU benchmarks).  Cold: rotating replicas larger than L2."""
    import dataclasses
    w = dataclasses.replace(W["c2"], name="c2_b2048", batch=2048)
    rep = Replicas(w, cfi, torch, 2 * l2 + (32 << 20), max_replicas=16)
    out = {"batch": w.batch}
    for v in ("auto", "batch"):
        out[f"us_per_call_{v}"] = us(time_steps(rep, torch, 500, 10, v, target_s=0.05))
    flops = algorithmic_flops(w, rep.n_active)
    fma_peak = sm_count * FMA_LANES_PER_SM * 2 * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
    out["effective_tflops"] = flops / (out["us_per_call_auto"] * 1e-6) / 1e12
    out["fma_frac"] = out["effective_tflops"] / fma_peak
    out["variant"] = VARIANT_NAMES[cfi.cfi_choose_variant(rep.layers[0], w.batch)]
    rep.close()
    return out


def stack_batch1_leg(cfi, torch, l2, peaks, blocks=12, replicas=4):
    """Online inference through a whole fp32 MLP stack at batch 1: 2 * blocks dependent launches per pass, each
    released early by the one before it (programmatic dependent launch), replayed from a CUDA graph.  Rotating
    replicas of the stack (together larger than L2) make every pass stream its weights from HBM."""
    s = inputs.StackWorkload(blocks=blocks, batch=1, dtype="f32")
    stacks, keep, flops, bytes_ = [], [], 0, 0
    for r in range(replicas):
        layers = []
        for L, sp in zip(s.layers(seed=r), s.layer_specs()):
            v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
            layers.append(cfi.cfi_create(v, ix, rows, L.bias, sp[0], sp[1], dtype="f32", act=sp[4]))
            if r == 0:
                flops += 2 * rows.shape[0] * sp[2]
                bytes_ += rows.shape[0] * sp[2] * 8 + (sp[0] + 2 * sp[1]) * 4 + rows.shape[0] * 4
        stacks.append(cfi.cfi_stack_create(layers, 1))
        keep.append(layers)
    x = torch.from_numpy(s.x(seed=0)).to("cuda", torch.float32)
    y = torch.empty((1, s.d_model), device="cuda", dtype=torch.float32)
    stream = torch.cuda.Stream()
    passes = 50 * replicas
    with torch.cuda.stream(stream):
        for st in stacks:
            cfi.cfi_stack_forward(st, x, y, 1)
        stream.synchronize()
        eager = _time_torch(lambda: cfi.cfi_stack_forward(stacks[0], x, y, 1), torch, iters=200)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(passes):
                cfi.cfi_stack_forward(stacks[i % replicas], x, y, 1)
        g.replay()
        stream.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(20):
            g.replay()
        b.record(stream)
        b.synchronize()
    sec = a.elapsed_time(b) * 1e-3 / (20 * passes)
    for st in stacks:
        st.close()
    for layers in keep:
        for l in layers:
            l.close()
    return {"layers": 2 * blocks, "dtype": "f32", "us_per_pass_graph_cold": sec * 1e6, "us_per_layer": sec * 1e6 / (2 * blocks),
            "us_per_pass_eager_warm": eager * 1e6, "algorithmic_bytes": bytes_,
            "hbm_frac": bytes_ / sec / 1e9 / peaks["hbm_gbs"], "gflops": flops / sec / 1e9,
            "l2": f"{replicas} rotating stacks, {replicas * bytes_ / 1e6:.0f} MB vs L2 {l2 / 1e6:.0f} MB"}


def srigl_update_leg(cfi, torch, peaks):
    """One SRigL mask update (Sec. 3.1, steps 1-7) on the device for the two ViT MLP layer shapes and the 4096 x 4096
    layer at 80 % sparsity; K = 30 % of the active weights, gamma_sal = 0.3.  Algorithmic bytes: w, mask and grad
    read once (9 B per entry), w and mask written once (5 B)."""
    import time
    out = {}
    for name, (out_f, in_f, k) in {"768x3072_k77": (3072, 768, 77), "3072x768_k307": (768, 3072, 307),
                                   "4096x4096_k819": (4096, 4096, 819)}.items():
        L = inputs.make_layer(in_f, out_f, k, seed=11, bias=False)
        g = torch.from_numpy(inputs.make_x(out_f, in_f, seed=12)).cuda()
        w0, m0 = torch.from_numpy(L.w_dense).cuda(), torch.from_numpy(L.mask).cuda()
        K = int(0.3 * out_f * k)
        times = []
        for it in range(6):
            w, m = w0.clone(), m0.clone()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            k_new, n_act = cfi.cfi_srigl_update(w, m, g, K, 0.3)     # returns after its stream has drained
            times.append(time.perf_counter() - t0)
        sec = float(np.median(times[1:]))
        nbytes = 14 * out_f * in_f
        out[name] = {"us_per_update": sec * 1e6, "K": K, "k_new": k_new, "n_active_new": n_act,
                     "algorithmic_bytes": nbytes, "hbm_frac": nbytes / sec / 1e9 / peaks["hbm_gbs"]}
    return out


def floor_leg(cfi, torch, l2):
    """What a forward call costs with all of the layer's work taken out, measured the way the forward is timed (a CUDA
    graph of back-to-back launches with the forward kernels' launch attributes): an empty kernel, and a kernel in
    which every CTA makes one dependent trip to DRAM and one store.  A batch-1 call can be no faster than the second."""
    buf = torch.empty(max(4 * l2, 256 << 20) // 4, dtype=torch.float32, device="cuda")
    buf.zero_()
    scratch = torch.zeros(1024, dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    out = {}
    with torch.cuda.stream(stream):
        for kind, name in ((0, "empty_node_us"), (1, "dram_roundtrip_node_us")):
            for _ in range(10):
                cfi.cfi_probe_floor_launch(kind, buf, scratch)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(1000):
                    cfi.cfi_probe_floor_launch(kind, buf, scratch)
            g.replay()
            stream.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(21)]
            ev[0].record(stream)
            for i in range(20):
                g.replay()
                ev[i + 1].record(stream)
            ev[-1].synchronize()
            t = [ev[i].elapsed_time(ev[i + 1]) for i in range(20)]
            out[name] = statistics.median(t)           # ms per 1000 launches = us per launch
            out[name.replace("_us", "_std_us")] = statistics.pstdev(t)
    out["note"] = "us per node of a 1000-node CUDA graph, median of 20 replays; nodes are launched with programmatic " \
                  "dependent launch like the forward kernels, one CTA per SM"
    return out


# Layer shapes of the named workloads: every batch size of a shape is timed on the same replicas of the layer.
SWEEP = [("c1", ["c1", "c2"]), ("c3_b1", ["c3_b1", "c3_b64", "c3_b256"])] + \
        [(f"c4_s{sp}_b1", [f"c4_s{sp}_b{b}" for b in (1, 16, 256)]) for sp in (80, 90, 95, 99)]


def sweep_leg(W, cfi, torch, l2, ceil_, floor, only=None, cpu=True):
    """Every named workload, cold (rotating replicas of layer, x and y larger than twice the L2): us per call (median
    and standard deviation over the passes), the kernel the library picks, algorithmic bytes and flops, the time the
    HBM and the fp32 FMA rooflines allow, the fraction of the binding one, the fraction of the gather formulation's
    shared-memory ceiling for batch > 1, the launch floor for batch 1, and the oracle on this host's cores."""
    import oracle
    out = {}
    for base_name, names in SWEEP:
        names = [n for n in names if only is None or n in only]
        if not names:
            continue
        base = W[base_name]
        L = base.layer(seed=0)
        packed = cfi.cfi_pack(L.w_dense, L.mask)
        opk = oracle.pack(L.w_dense, L.mask) if cpu else None   # the oracle's own pack for its own timing
        probe = cfi.cfi_create(packed[0], packed[1], packed[2], L.bias, base.in_features, base.out_features)
        for name in names:
            w = W[name]
            # The replicas hold the layouts the chosen kernel needs (all three for the tensor-core variant, whose dense
            # copy is then what a call streams; the two condensed ones otherwise; the small-batch one alone at batch 1).
            variant = VARIANT_NAMES[cfi.cfi_choose_variant(probe, w.batch)]
            shape = dense_shape(cfi, probe, w.batch) if variant == "dense_tc" else None
            dense_bytes = int(cfi.cfi_layer_info(probe).bytes_dense) if variant == "dense_tc" else None
            layouts = 7 if variant == "dense_tc" else 1 if w.batch == 1 else 3
            rep = Replicas(w, cfi, torch, 2 * l2 + (32 << 20), max_replicas=200, layer=L, packed=packed, layouts=layouts,
                           streamed_bytes=dense_bytes)
            assert VARIANT_NAMES[cfi.cfi_choose_variant(rep.layers[0], w.batch)] == variant
            t = time_steps(rep, torch, 1000, 10, target_s=0.05)
            sec = t["sec_per_step"]
            flops, nbytes = algorithmic_flops(w, rep.n_active), rep.bytes_per_step
            t_hbm, t_fma = nbytes / (ceil_.hbm_gbs * 1e9), flops / (ceil_.fma_tflops * 1e12)
            info = cfi.cfi_layer_info(rep.layers[0])
            e = {"us_per_call": sec * 1e6, "us_per_call_std": t["std_sec_per_step"] * 1e6, "passes": t["passes"],
                 "variant": variant, "dense_shape": shape, "algorithmic_bytes": nbytes, "algorithmic_flops": flops,
                 "gflops": flops / sec / 1e9, "hbm_gbs": nbytes / sec / 1e9,
                 "t_hbm_us": t_hbm * 1e6, "t_fma_us": t_fma * 1e6, "bound": "hbm" if t_hbm >= t_fma else "alu",
                 "frac_of_bound": max(t_hbm, t_fma) / sec, "hbm_frac": t_hbm / sec, "fma_frac": t_fma / sec,
                 "replicas": rep.R, "layouts": layouts, "device_bytes_per_layer": int(info.device_bytes)}
            if w.batch > 1:
                e["smem_ceiling_frac"] = flops / sec / 1e12 / ceil_.smem_tflops
            else:
                e["floor_us"] = floor["dram_roundtrip_node_us"]
                e["times_floor"] = sec * 1e6 / floor["dram_roundtrip_node_us"]
                e["streamed_bytes"] = int(info.weight_bytes_splitk) + (w.in_features + 2 * w.out_features) * 4
                one = Replicas(w, cfi, torch, 0, max_replicas=2, layer=L, packed=packed, layouts=layouts)
                one.R = 1
                e["us_per_call_warm"] = us(time_steps(one, torch, 1000, 10, target_s=0.02))
                one.close()
            rep.close()
            out[name] = e
            if not cpu:
                continue
            cb = time_oracle(w, budget_s=1.0, layer=L, packed=opk)
            e["cpu_oracle"] = {"us_per_call_scaled": cb["median_s"] * 1e6 * w.batch / cb["rows"], "rows_timed": cb["rows"],
                               "cores": cb["cores"], "gflops": cb["flops"] / cb["median_s"] / 1e9}
            out[name] = e
        probe.close()
    if not cpu:
        return out
    # The bf16 stack's CPU time: one block's two layers on a 788-row slice (1/64 of the batch), scaled.
    s = inputs.StackWorkload(blocks=1)
    x = s.x(seed=0, batch=788)
    tot = 0.0
    for Ls, sp in zip(s.layers(seed=0), s.layer_specs()):
        pk = oracle.pack(Ls.w_dense, Ls.mask)
        xin = oracle.round_bf16(x) if sp[0] == s.d_model else np.zeros((788, sp[0]), np.float32)
        t0 = time.perf_counter()
        oracle.forward(oracle.round_bf16(pk[0]), pk[1], pk[2], Ls.bias, sp[0], sp[1], xin, act=sp[4])
        tot += time.perf_counter() - t0
    out["c5_cpu_oracle"] = {"ms_per_pass_scaled": tot * 12 * 64 * 1e3, "rows_timed": 788, "blocks_timed": 1,
                            "cores": oracle.max_threads(), "note": "one block on 788 of 50,432 rows, x 64 x 12"}
    return out


if __name__ == "__main__":
    main()
