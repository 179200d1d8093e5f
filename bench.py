#!/usr/bin/env python
"""Benchmark of the b200 GEMM hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config c1..c5]

A step is one pass of the whole hot path (plan already made; tensor-map encode, tile scheduling,
TMA/tcgen05 main loop, epilogue) over one batch of synthetic input.  The headline workload is
config c2 (8192^3 bf16, A row-major, B column-major, bf16 output), the configuration the
metric is quoted on; ``--all`` (default on) adds one entry per benchmark configuration under
``configs_measured``.  Prints ONE JSON line on rank 0.

Timing: CUDA events on the launching stream around K back-to-back steps, after W >= 3 warm-up
steps; every configuration rotates through at least two (HBM-bound ones: three) seeded sets of
inputs AND outputs, and through as many as it takes to exceed twice the L2 capacity, so no step
finds its operands, or a dirty copy of its output, in cache (the paper's Section 5.1 protocol:
different random inputs per run).  ``e2e`` repeats the measurement with host-resident pinned
inputs and output: every step copies A and B to the device, runs the GEMM and copies D back.
``library_reference`` times the vendor GEMM (torch) on the same buffers in the same loop and
``sustained`` repeats the headline for at least four seconds: both are context, outside the product.

``--impl reference`` times the CPU oracle (the fp64 triple loop) on a bounded sample of the same
workload; it is a deliberately slow program and only a reported baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as wl  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
NOMINAL = {"tensor_tflops": 2250.0, "hbm_gbs": 8000.0}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# The ncu summary of each configuration's kernel (profiles/): its line "dram traffic per launch (read + write): N bytes"
# is dram__bytes_read.sum + dram__bytes_write.sum of one captured launch and becomes roofline.traffic.
PROFILE_OF = {"c1": "dense_1cta_c1_512_nn.txt", "c2": "wide_2cta_c2_square_8192.txt", "c3": "dense_2cta_c3_proj_bias_gelu.txt",
              "c4": "wide_2cta_c4_batched_fp16.txt", "c5": "skinny_streamk_c5_8x28672x8192.txt"}


def ncu_traffic_bytes(key: str):
    """DRAM bytes per launch from the committed ncu summary of this configuration's kernel, or None."""
    name = PROFILE_OF.get(key)
    if not name:
        return None
    try:
        with open(os.path.join(ROOT, "profiles", name)) as f:
            for line in f:
                if line.startswith("dram traffic per launch (read + write):"):
                    return int(line.split(":")[1].split()[0])
    except (OSError, ValueError):
        pass
    return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"]))}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
                 nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown"}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def roofline_for(w: wl.Workload, key: str, seconds: float, peaks: dict, peak_kind: str) -> dict:
    """Roofline entry of the step's single kernel: the bound is whichever of (flops / tensor peak)
    and (compulsory bytes / HBM bandwidth) is slower."""
    fp8 = w.ab_dtype in (wl.FP8_E4M3, wl.FP8_E5M2)
    # a contraction takes the peak of its own operand type: the measured bf16 figure times the nominal fp8 : bf16 ratio
    tensor_peak = peaks["bf16_tflops"] * (2.0 if fp8 else 1.0)
    t_tensor = w.flops / (tensor_peak * 1e12)
    t_hbm = w.min_bytes / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        achieved, peak, unit, bound = w.flops / seconds / 1e12, tensor_peak, "TFLOP/s", "tensor"
    else:
        achieved, peak, unit, bound = w.min_bytes / seconds / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    return {"bound": bound, "achieved": round(achieved, 2), "peak": peak, "unit": unit, "frac": round(achieved / peak, 4),
            "traffic": ncu_traffic_bytes(key), "peak_source": f"of {peak_kind}" + (" bf16 x 2 (nominal fp8 ratio)" if fp8 and bound == "tensor" else ""),
            "frac_of_nominal": round(achieved / (NOMINAL["tensor_tflops"] * (2.0 if fp8 else 1.0) if bound == "tensor" else NOMINAL["hbm_gbs"]), 4),
            "algorithmic_flops": w.flops, "algorithmic_bytes": w.min_bytes}


# --------------------------------------------------------------------------- our arm

def _torch_dt(torch, code):
    return {wl.BF16: torch.bfloat16, wl.F16: torch.float16, wl.F32: torch.float32}[code]


def _to_torch(torch, arr, code, device=None, pin=False):
    if code == wl.F32 or arr.dtype == np.uint8:   # fp32 values, or the bytes of 8-bit floats
        t = torch.from_numpy(arr)
    else:
        t = torch.from_numpy(arr.view(np.int16)).view(_torch_dt(torch, code))
    if pin:
        t = t.pin_memory()
    return t.to(device) if device is not None else t


class DeviceCase:
    """One benchmark configuration resident in HBM: R rotating input sets and a plan."""

    def __init__(self, torch, bg, key: str, w: wl.Workload, flags: int, device, nsets_cap: int = 160):
        self.torch, self.bg, self.key, self.w, self.device = torch, bg, key, w, device
        footprint = w.min_bytes
        # Rotating sets (inputs and output buffers, different seeds): as many as make the combined footprint exceed twice
        # the L2, and never fewer than two -- three for an HBM-bound problem, whose time is all memory traffic -- so that
        # a step finds neither its operands nor a dirty copy of its output in cache.  Capped at 12 GB of device memory.
        hbm_bound = w.min_bytes / 6.5e12 > w.flops / 1.6e15
        want = max(3 if hbm_bound else 2, -(-2 * L2_BYTES // int(footprint)))
        self.nsets = int(max(1 if nsets_cap == 1 else 2, min(want, 160, nsets_cap, int(12e9 // footprint))))
        self.sets = []
        for r in range(self.nsets):
            inp = wl.make_inputs(w, seed_offset=1000 * r)
            A = _to_torch(torch, inp["A"], w.ab_dtype, device)
            B = _to_torch(torch, inp["B"], w.ab_dtype, device)
            if inp["C"] is not None:
                C = _to_torch(torch, inp["C"], w.c_dtype, device)
            else:
                C = torch.empty(w.elems_c(), dtype=_torch_dt(torch, w.c_dtype), device=device)
            bias = None if inp["bias"] is None else _to_torch(torch, inp["bias"], wl.F32, device)
            self.sets.append((A, B, C, bias))
            if r == 0:
                self.host_inputs = inp
        d = bg.make_desc(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, w.c_dtype, w.lda, w.ldb, w.ldc, w.batch,
                         w.stride_a, w.stride_b, w.stride_c, w.epilogue,
                         flags | bg.make_flags(bias_per_row=w.bias_per_row, a_lower=w.a_tri == 1, a_upper=w.a_tri == 2,
                                               d_lower=w.d_tri == 1, d_upper=w.d_tri == 2),
                        structure=w.b_tri | (4 if w.d_mirror else 0))
        self.desc = d
        self.plan = bg.Plan(d)
        self.plan.workspace(device)
        self.i = 0
        self._calls = None
        self.warm_launches = 0

    def _bind(self, plan):
        """One pre-marshalled gemm_run call per input set (C ABI, raw device addresses, current stream)."""
        ws = plan.workspace(self.device)
        wsp, wsb = (0, 0) if ws is None else (ws.data_ptr(), ws.numel())
        stream = self.torch.cuda.current_stream(self.device).cuda_stream
        return [self.bg.bind_run(plan.handle, A.data_ptr(), B.data_ptr(), C.data_ptr(), 0 if bias is None else bias.data_ptr(),
                                 float(self.w.alpha), float(self.w.beta), wsp, wsb, stream) for A, B, C, bias in self.sets]

    def step(self):
        """One pass of the hot path through the C ABI: gemm_run on the next input set."""
        if self._calls is None:
            self._calls = self._bind(self.plan)
        self._calls[self.i % self.nsets]()
        self.i += 1

    def use_plan(self, flags: int):
        """Replace the plan by one made with extra descriptor flags (same problem, same buffers)."""
        d = self.bg.Desc.from_buffer_copy(self.desc)
        d.flags |= flags
        self.plan.close()
        self.plan = self.bg.Plan(d)
        self.plan.workspace(self.device)
        self._calls = None

    def time_steps(self, steps: int, warmup: int, step=None) -> float:
        """Seconds per step over `steps` back-to-back steps (CUDA events on the launching stream).  `step` replaces the
        library call by another function of no arguments (the vendor-library reference point runs in this same loop).
        self.warm_launches counts the untimed launches that preceded the timed region."""
        torch = self.torch
        step = step or self.step
        self.warm_launches = warmup + 8
        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        # A configuration whose whole timed region lasts well under a millisecond would otherwise be measured while the
        # clocks are still ramping up from idle (the pause between configurations lets them drop): such a one keeps
        # warming up, untimed, until 30 ms have passed.  (The first launches carry one-off costs, so the step time is
        # estimated from a second small batch.)
        t_warm = time.perf_counter()
        for _ in range(8):
            step()
        torch.cuda.synchronize()
        step_sec = (time.perf_counter() - t_warm) / 8
        # (short steps only: a step of several hundred microseconds has ramped the clocks up within the requested warm-up,
        # and tens of further launches would only move it from the rested towards the power-capped state)
        short_region = step_sec * steps < 0.03 and step_sec < 2.0e-4
        while short_region and time.perf_counter() - t_warm < 0.03:
            for _ in range(16):
                step()
            self.warm_launches += 16
            torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        st = self.plan.status()
        if st != self.bg.OK:
            raise RuntimeError(f"device status {self.bg.status_string(st)} after timing {self.key}")
        return e0.elapsed_time(e1) * 1e-3 / steps

    def library_step(self):
        """The vendor library (torch -> cuBLAS) on this configuration's own buffers, as a function of no arguments for
        time_steps, and a description of what it runs.  Reference point only: nothing in the product calls it."""
        torch, w = self.torch, self.w
        if w.ab_dtype not in (wl.BF16, wl.F16) or w.a_tri or w.b_tri or w.d_tri:
            return None, "no plain library counterpart"
        F = torch.nn.functional
        views = []
        for A, B, C, bias in self.sets:
            a3 = torch.as_strided(A, (w.batch, w.K if w.transa else w.M, w.M if w.transa else w.K), (w.stride_a, w.lda, 1))
            b3 = torch.as_strided(B, (w.batch, w.N if w.transb else w.K, w.K if w.transb else w.N), (w.stride_b, w.ldb, 1))
            opa = a3.transpose(1, 2) if w.transa else a3
            opb = b3.transpose(1, 2) if w.transb else b3
            c3 = torch.as_strided(C, (w.batch, w.M, w.N), (w.stride_c, w.ldc, 1))
            views.append((opa, opb, c3, bias))
        same_out = w.c_dtype == w.ab_dtype
        out_note = "" if same_out else " (output in the operand type: the library call has no fp32 output for 16-bit operands" + \
            ("; beta * C is not applied)" if w.beta != 0.0 else ")")
        fused_bias = w.batch == 1 and w.has_bias and not w.bias_per_row and (w.beta == 0.0 or not same_out)
        bias16 = [None if b is None else b.to(_torch_dt(torch, w.ab_dtype)) for _, _, _, b in self.sets]
        scratch = [torch.empty((w.batch, w.M, w.N), dtype=_torch_dt(torch, w.ab_dtype), device=self.device) for _ in self.sets] \
            if not same_out else None
        act = w.epilogue >> 1
        i = [0]

        def step():
            opa, opb, c3, bias = views[i[0] % self.nsets]
            out = c3 if same_out else scratch[i[0] % self.nsets]
            k = i[0] % self.nsets
            i[0] += 1
            if fused_bias:   # one library call with the bias in its epilogue
                torch.addmm(bias16[k], opa[0], opb[0], alpha=w.alpha, out=out[0])
            elif w.alpha != 1.0 or (w.beta != 0.0 and same_out):
                torch.baddbmm(c3 if same_out else out, opa, opb, beta=w.beta if same_out else 0.0, alpha=w.alpha, out=out)
            else:
                torch.bmm(opa, opb, out=out)
            if w.has_bias and not fused_bias:
                out.add_(bias16[k] if not w.bias_per_row else bias16[k][:, None])
            if act == 1:
                out.relu_()
            elif act == 2:
                out.copy_(F.gelu(out))
            elif act == 3:
                out.copy_(F.gelu(out, approximate="tanh"))
            elif act == 4:
                out.copy_(F.silu(out))
        what = ("torch.addmm (bias in the library epilogue)" if fused_bias else "torch.bmm / baddbmm" + (", then bias add" if w.has_bias else "")) + \
            " on the same buffers" + ({0: "", 1: ", then relu", 2: ", then gelu", 3: ", then gelu(tanh)", 4: ", then silu"}[act]) + \
            (" as a separate kernel" if act else "") + out_note
        return step, what

    def time_burst(self, n: int = 10):
        """`n` launches in a row, each between its own pair of events: the best one, in seconds."""
        torch = self.torch
        torch.cuda.synchronize()
        time.sleep(1.5)   # from a rested GPU, as a peak measurement would be taken
        for _ in range(3):
            self.step()
        pairs = []
        for _ in range(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            self.step()
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        return min(a.elapsed_time(b) for a, b in pairs) * 1e-3

    def time_isolated(self, n: int = 10):
        """Single launches, each on an idle GPU with a flushed L2 and bracketed by its own pair of events: (median, best) in
        seconds.  This is the situation of a launch under the profiler (nothing overlaps its set-up, caches are cold, the
        clocks start from idle), so it is the event-timed counterpart of the ncu durations in profiles/."""
        torch = self.torch
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=self.device)
        times = []
        for _ in range(n):
            flush.zero_()
            torch.cuda.synchronize()
            time.sleep(0.002)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            self.step()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) * 1e-3)
        return statistics.median(times), min(times)

    def time_sustained(self, seconds: float, step=None, sampler_index: int = 0):
        """Back-to-back steps for at least `seconds` (after one second of the same load), timed with CUDA events on the
        launching stream while the SM clock is sampled: what the configuration sustains under the power cap."""
        torch = self.torch
        step = step or self.step

        def spin(duration, chunk=20):
            n, t0 = 0, time.perf_counter()
            while time.perf_counter() - t0 < duration:
                for _ in range(chunk):
                    step()
                n += chunk
                if n % (8 * chunk) == 0:
                    torch.cuda.synchronize()   # keeps the launch queue short so that the loop ends on time
            return n

        spin(1.0)
        torch.cuda.synchronize()
        with ClockSampler(sampler_index) as clocks:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            n = spin(seconds)
            e1.record()
            torch.cuda.synchronize()
        sec = e0.elapsed_time(e1) * 1e-3
        c = clocks.summary()
        per_step = sec / n
        return {"value": round(metric_value(self.w, per_step), 2), "unit": "TFLOP/s", "seconds": round(sec, 2), "launches": n,
                "ms_per_step": round(per_step * 1e3, 5), "sm_mhz_median": c["sm_mhz"], "reasons": c["reasons"],
                # time x clock: SM cycles per step in millions; constant if the kernel is clock-bound, so run-to-run
                # differences in the power-capped clock can be told from differences in the kernel
                "mcycles_per_step": None if not c["sm_mhz"] else round(per_step * c["sm_mhz"], 3)}

    def time_e2e(self, steps: int, warmup: int):
        """Same metric with host-resident inputs and output, through gemm_host_run: every step copies A, B (and C_in,
        bias) from pinned host memory, multiplies, and copies D back, row panel by row panel on three streams.  The
        call returns when D is complete in host memory, so the steps are timed with the host clock between two
        device synchronisations.  Returns (seconds per step, h2d bytes, d2h bytes, row panels)."""
        torch, w, bg = self.torch, self.w, self.bg
        inp = self.host_inputs
        hA = _to_torch(torch, inp["A"], w.ab_dtype, pin=True)
        hB = _to_torch(torch, inp["B"], w.ab_dtype, pin=True)
        hbias = None if inp["bias"] is None else _to_torch(torch, inp["bias"], wl.F32, pin=True)
        C0 = self.sets[0][2]
        hC = (torch.empty(C0.shape, dtype=C0.dtype) if inp["C"] is None else _to_torch(torch, inp["C"], w.c_dtype)).pin_memory()
        h2d = hA.numel() * hA.element_size() + hB.numel() * hB.element_size()
        h2d += 0 if inp["C"] is None else hC.numel() * hC.element_size()
        h2d += 0 if hbias is None else hbias.numel() * 4
        d2h = w.M * w.N * hC.element_size()
        handle = bg.gemm_host_create(self.plan.desc, 0)
        try:
            args = (handle, hA.data_ptr(), hB.data_ptr(), hC.data_ptr(), 0 if hbias is None else hbias.data_ptr(),
                    float(w.alpha), float(w.beta))
            for _ in range(warmup):
                bg.gemm_host_run(*args)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(steps):
                bg.gemm_host_run(*args)
            torch.cuda.synchronize()
            sec = (time.perf_counter() - t0) / steps
            panels = bg.gemm_host_panels(handle)
        finally:
            bg.gemm_host_destroy(handle)
        return sec, h2d, d2h, panels

    def close(self):
        self.plan.close()
        self.sets = []


def max_over_ranks(x: float, device=None) -> float:
    """MAX of a per-rank scalar over the process group (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(w: wl.Workload, seconds_max_over_ranks: float, world: int) -> float:
    """Replicas: every rank runs the same problem, the job's throughput is world x flops over the slowest rank's time."""
    return world * w.flops / seconds_max_over_ranks / 1e12


def metric_value(w: wl.Workload, seconds: float) -> float:
    return w.flops / seconds / 1e12


def time_oracle_sample(w: wl.Workload, inputs: dict, target_seconds: float):
    """Time the oracle, as it stands, on the first rows of batch 0 of the workload; the row count
    is calibrated so the run takes about `target_seconds`.  Returns (TFLOP/s, cores, description)."""
    import oracle
    p = oracle.Problem(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, w.c_dtype, w.lda, w.ldb, w.ldc, w.batch,
                       w.stride_a, w.stride_b, w.stride_c, w.epilogue)
    cores = oracle.max_threads()
    cols = np.arange(w.N, dtype=np.int64)

    def run(nrows):
        rows = np.arange(nrows, dtype=np.int64)
        t0 = time.perf_counter()
        oracle.gemm(p, inputs["A"], inputs["B"], C_in=inputs["C"], bias=inputs["bias"], alpha=w.alpha, beta=w.beta,
                    batches=[0], rows=rows, cols=cols)
        return time.perf_counter() - t0

    probe_rows = min(w.M, 2)
    t_probe = max(run(probe_rows), 1e-4)
    nrows = int(max(probe_rows, min(w.M, round(probe_rows * target_seconds / t_probe))))
    t = run(nrows)
    flops = 2.0 * nrows * w.N * w.K
    return flops / t / 1e12, cores, f"rows 0..{nrows - 1} x all {w.N} columns of batch 0 ({flops / 1e9:.1f} GFLOP in {t:.1f} s)"


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2512_16465_b200 as bg

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    peaks, peak_kind = load_peaks()
    cfgs = wl.configs()
    flags = int(args.flags, 0)
    steps, warmup = args.steps, max(3, args.warmup)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over(x: float) -> float:
        return max_over_ranks(x, device)

    key = args.config
    w = cfgs[key]
    case = DeviceCase(torch, bg, key, w, flags, device)
    barrier()
    with ClockSampler(local_rank) as clocks:
        sec = case.time_steps(steps, warmup)
        barrier()
    sec = max_over(sec)
    warm_launches = case.warm_launches
    # context: the vendor library on the same buffers in the same loop, and the headline held for seconds
    library = sustained = None
    burst = case.time_burst() if args.all else None
    iso_med, iso_best = case.time_isolated() if args.all else (None, None)
    lib_step = None
    if args.all and world == 1:
        lib_step, lib_what = case.library_step()
        if lib_step is not None:
            time.sleep(1.0)
            lib_sec = case.time_steps(steps, warmup, step=lib_step)
            library = {"value": round(metric_value(w, lib_sec), 2), "unit": "TFLOP/s", "ms_per_step": round(lib_sec * 1e3, 5),
                       "what": lib_what + "; same rotating buffers, same event-timed loop; context only, no part of the product"}
        time.sleep(1.0)
    e2e_steps = max(2, min(steps, args.e2e_steps))
    barrier()
    if args.e2e_steps > 0:
        e2e_sec, h2d, d2h, e2e_panels = case.time_e2e(e2e_steps, 2)
    else:  # profiling runs skip the host-buffer leg
        e2e_sec, h2d, d2h, e2e_panels = float("nan"), 0, 0, 0
    barrier()
    e2e_sec = max_over(e2e_sec)

    out = {
        "metric": "GEMM TFLOP/s at 1 B200 and % of dense bf16 roofline (HBM GB/s for skinny)",
        "value": round(whole_job_value(w, sec, world), 2), "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "warmup_launches_actual": warm_launches,
        "ms_per_step": round(sec * 1e3, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 x bf16 -> fp32 accumulate", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "N": w.N, "K": w.K, "batch": w.batch,
                   "layout": "A row-major, B stored N x K", "out_dtype": ["bf16", "f16", "f32"][w.c_dtype],
                   "l2": f"inputs larger than L2: {case.nsets} rotating seeded sets of inputs and output, {w.min_bytes / 1e6:.0f} MB each",
                   "input_sets": case.nsets,
                   "multi_gpu": "replicas only (independent GEMMs, no collective)", "plan": case.plan.info},
        "e2e": None if args.e2e_steps <= 0 else {"value": round(metric_value(w, e2e_sec) * world, 3), "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_sec * 1e3, 3), "steps": e2e_steps,
                "path": f"gemm_host_run: pinned host buffers, {e2e_panels} row panels, H2D / GEMM / D2H overlapped on three streams; host clock around blocking calls"},
        "gpu_launches": steps,
        "clocks": clocks.summary(),
        "roofline": roofline_for(w, key, sec, peaks, peak_kind),
    }
    out["roofline"]["frac_of_sustained_peak"] = round(metric_value(w, sec) / peaks["bf16_tflops_sustained"], 4)
    if burst is not None:
        # ten launches in a row, each between its own pair of events, the best one: the protocol the measured dense peak
        # of this pool was taken with (best of ten single library launches), so this fraction compares like with like
        out["burst_best_of_10"] = {"ms": round(burst * 1e3, 5), "value": round(metric_value(w, burst), 2), "unit": "TFLOP/s",
                                   "frac_of_peak": round(roofline_for(w, key, burst, peaks, peak_kind)["frac"], 4)}
    if iso_med is not None:
        # single launches on an idle GPU with a flushed L2: what a launch under the profiler corresponds to
        out["isolated_launch"] = {"ms_median": round(iso_med * 1e3, 5), "ms_best_of_10": round(iso_best * 1e3, 5)}
    if library is not None:
        out["library_reference"] = library
    host_inputs = case.host_inputs

    if args.all:
        measured = []
        for k2, w2 in cfgs.items():
            if k2 == key:
                measured.append({"config": k2, "workload": w2.name, "ms_per_step": out["ms_per_step"], "tflops": out["value"] / world,
                                 "input_sets": out["config"]["input_sets"], "warmup_launches_actual": warm_launches,
                                 "ms_isolated_launch": None if iso_med is None else round(iso_med * 1e3, 5),
                                 "roofline": out["roofline"],
                                 "library_reference_ms_per_step": None if library is None else library["ms_per_step"]})
                continue
            c2 = DeviceCase(torch, bg, k2, w2, 0, device)
            torch.cuda.synchronize()
            time.sleep(1.5)  # let clocks and the power governor recover from the previous configuration's load
            s2 = max_over(c2.time_steps(steps, warmup))
            row = {"config": k2, "workload": w2.name, "ms_per_step": round(s2 * 1e3, 5),
                   "tflops": round(metric_value(w2, s2), 2), "gbs": round(w2.min_bytes / s2 / 1e9, 1),
                   "input_sets": c2.nsets, "warmup_launches_actual": c2.warm_launches, "plan": c2.plan.info,
                   "roofline": roofline_for(w2, k2, s2, peaks, peak_kind)}
            row["ms_isolated_launch"] = round(c2.time_isolated()[0] * 1e3, 5)
            if world == 1:
                lib2, lib2_what = c2.library_step()
                if lib2 is not None:     # the vendor library on the same buffers, same loop (context)
                    time.sleep(0.5)
                    row["library_reference_ms_per_step"] = round(c2.time_steps(steps, warmup, step=lib2) * 1e3, 5)
                    row["library_reference_what"] = lib2_what
                # the same plan launched without programmatic dependent launch: what the overlap of one kernel's set-up
                # with its predecessor's tail is worth in this back-to-back loop
                time.sleep(0.5)
                c2.use_plan(bg.make_flags(no_early_launch=True))
                row["ms_per_step_no_early_launch"] = round(c2.time_steps(steps, warmup) * 1e3, 5)
            measured.append(row)
            c2.close()
        out["configs_measured"] = measured

    # context only (library kernels, not part of the product): what plain streaming kernels reach on this GPU.
    # The copy figure in MEASURED_PEAKS.json mixes reads and writes; a write-dominated kernel (c4) cannot go faster
    # than a pure fill, a read-dominated one (c5) than a pure reduction.
    if args.all:
        xs = torch.empty(1 << 29, dtype=torch.float16, device=device)

        def rate(fn, nbytes, n=10):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(n):
                fn()
            b.record()
            torch.cuda.synchronize()
            return round(nbytes / (a.elapsed_time(b) * 1e-3 / n) / 1e9, 1)

        out["hbm_context"] = {"torch_fill_write_only_gbs": rate(lambda: xs.fill_(1.0), xs.numel() * 2),
                              "torch_sum_read_only_gbs": rate(lambda: xs.sum(), xs.numel() * 2)}
        del xs

    # last, so that the seconds of full load do not warm the GPU under the other measurements: the headline held for
    # `--sustained-seconds`, and the library reference point the same way
    if args.all and world == 1 and args.sustained_seconds > 0:
        time.sleep(1.0)
        sustained = case.time_sustained(args.sustained_seconds, sampler_index=local_rank)
        sustained["frac_of_sustained_peak"] = round(sustained["value"] / peaks["bf16_tflops_sustained"], 4)
        out["sustained"] = sustained
        if lib_step is not None:
            time.sleep(1.0)
            ls = case.time_sustained(args.sustained_seconds, step=lib_step, sampler_index=local_rank)
            out["library_reference"]["sustained"] = {k: ls[k] for k in ("value", "seconds", "launches", "sm_mhz_median", "mcycles_per_step")}
    case.close()

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample = time_oracle_sample(w, host_inputs, args.cpu_seconds)
        out["cpu_baseline"] = {"value": round(v, 6), "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def parse_shape(spec: str) -> wl.Workload:
    """'MxNxK' followed by optional ':key=value' fields: batch, ta, tb (1 = stored transposed), ab (bf16|f16|e4m3|e5m2), cd (bf16|f16|f32),
    epi (none|bias|relu|bias_relu|gelu|bias_gelu|gelu_tanh|bias_gelu_tanh|silu|bias_silu), rowbias (0|1), tri (lower|upper: op(A) triangular), btri (the same for op(B)), dtri (lower|upper: only that triangle of D wanted), mirror (0|1: copy it into the other triangle), alpha, beta,
    lda, ldb, ldc.  Example: 28672x8x8192:beta=1:cd=f32."""
    head, *fields = spec.split(":")
    M, N, K = (int(x) for x in head.lower().split("x"))
    dt = {"bf16": wl.BF16, "f16": wl.F16, "f32": wl.F32, "e4m3": wl.FP8_E4M3, "e5m2": wl.FP8_E5M2}
    epi = {"none": wl.EPI_NONE, "bias": wl.EPI_BIAS, "relu": wl.EPI_RELU, "bias_relu": wl.EPI_BIAS_RELU,
           "gelu": wl.EPI_GELU_ERF, "bias_gelu": wl.EPI_BIAS_GELU_ERF, "gelu_tanh": wl.EPI_GELU_TANH,
           "bias_gelu_tanh": wl.EPI_BIAS_GELU_TANH, "silu": wl.EPI_SILU, "bias_silu": wl.EPI_BIAS_SILU}
    kw = dict(c_dtype=wl.BF16, dist_a=wl.Dist("normal", 0.0, 0.02), dist_b=wl.Dist("normal", 0.0, 0.02))
    for f in fields:
        k, v = f.split("=")
        if k == "batch":
            kw["batch"] = int(v)
        elif k in ("ta", "tb"):
            kw["transa" if k == "ta" else "transb"] = int(v)
        elif k in ("ab", "cd"):
            kw["ab_dtype" if k == "ab" else "c_dtype"] = dt[v]
        elif k == "epi":
            kw["epilogue"] = epi[v]
        elif k in ("alpha", "beta"):
            kw[k] = float(v)
        elif k == "tri":
            kw["a_tri"] = {"lower": 1, "upper": 2}[v]
        elif k == "btri":
            kw["b_tri"] = {"lower": 1, "upper": 2}[v]
        elif k == "mirror":
            kw["d_mirror"] = bool(int(v))
        elif k == "dtri":
            kw["d_tri"] = {"lower": 1, "upper": 2}[v]
        elif k == "rowbias":
            kw["bias_per_row"] = bool(int(v))
        elif k in ("lda", "ldb", "ldc"):  # leading dimensions in elements (each must span a multiple of 16 bytes)
            kw[k] = int(v)
        else:
            raise SystemExit(f"unknown field {k!r} in --shapes")
    return wl.Workload(spec, M, N, K, **kw)


def run_shapes(args):
    """Time arbitrary problem shapes with the automatic plan (sweeps beyond the five configurations): one JSON line
    whose `shapes_measured` holds, per shape, the plan taken, the time per launch and the roofline entry."""
    import torch
    import paper_2512_16465_b200 as bg

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--shapes is a single-GPU sweep")
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    peaks, peak_kind = load_peaks()
    steps, warmup = args.steps, max(3, args.warmup)
    rows = []
    with ClockSampler(0) as clocks:
        for spec in args.shapes.split(";"):
            w = parse_shape(spec.strip())
            case = DeviceCase(torch, bg, spec, w, int(args.flags, 0), device)
            torch.cuda.synchronize()
            time.sleep(0.3)
            sec = case.time_steps(steps, warmup)
            row = {"shape": spec, "ms_per_step": round(sec * 1e3, 5), "tflops": round(metric_value(w, sec), 2),
                   "gbs": round(w.min_bytes / sec / 1e9, 1), "input_sets": case.nsets,
                   "plan": {k: case.plan.info[k] for k in ("variant", "tile_m", "tile_n", "stages", "cluster_size", "grid", "split")},
                   "roofline": roofline_for(w, spec, sec, peaks, peak_kind)}
            if args.library_reference:
                # context only: the vendor library on the same rotating buffers in the same loop (no part of the product)
                lib_step, lib_what = case.library_step()
                if lib_step is not None:
                    row["library_reference_ms"] = round(case.time_steps(steps, warmup, step=lib_step) * 1e3, 5)
                    row["library_reference_what"] = lib_what
            if args.tune:
                # measured plan selection on the first input set (its C is scratch from here on), then the same timing
                # loop again: the new plan picks the remembered choice up by itself
                A, B, C, bias = case.sets[0]
                tuned, rep = bg.Plan.tuned(case.plan.desc, A, B, C, bias, w.alpha, w.beta, iterations=10)
                tuned.close()
                case.close()
                case = DeviceCase(torch, bg, spec, w, 0, device)
                torch.cuda.synchronize()
                time.sleep(0.3)
                sec2 = case.time_steps(steps, warmup)
                row["tuned"] = {"ms_per_step": round(sec2 * 1e3, 5), "flags": hex(rep["best_flags"]),
                                "plan": {k: case.plan.info[k] for k in ("variant", "tile_m", "tile_n", "tile_k", "stages", "raster_group")},
                                "candidates_tried": rep["candidates_tried"], "candidates_skipped": rep["candidates_skipped"],
                                "tuner_auto_ms": round(rep["auto_ms"], 5), "tuner_best_ms": round(rep["best_ms"], 5),
                                "roofline_frac": roofline_for(w, spec, sec2, peaks, peak_kind)["frac"]}
                if not args.tune_file:
                    bg.gemm_tune_cache_clear()
            rows.append(row)
            case.close()
    if args.tune and args.tune_file:   # keep the measured choices: gemm_tune_cache_load brings them back in another process
        print(f"[bench] {bg.gemm_tune_cache_save(args.tune_file)} tuning results written to {args.tune_file}", file=sys.stderr)
        bg.gemm_tune_cache_clear()
    print(json.dumps({"shapes_measured": rows, "steps": steps, "warmup": warmup, "clocks": clocks.summary(),
                      "timing": "CUDA events around back-to-back launches; inputs rotate so that each step's footprint exceeds L2"}), flush=True)


def run_reference(args):
    """The reference arm of this build is the CPU oracle: K steps, each a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = wl.configs()[args.config]
    inputs = wl.make_inputs(w)
    steps, warmup = args.steps, args.warmup
    # size each step so that the whole run stays within a few minutes
    per_step = max(0.05, min(args.ref_step_seconds, 120.0 / max(1, steps + warmup)))
    p = oracle.Problem(w.M, w.N, w.K, w.transa, w.transb, w.ab_dtype, w.c_dtype, w.lda, w.ldb, w.ldc, w.batch,
                       w.stride_a, w.stride_b, w.stride_c, w.epilogue)
    cols = np.arange(w.N, dtype=np.int64)

    def run(nrows):
        t0 = time.perf_counter()
        oracle.gemm(p, inputs["A"], inputs["B"], C_in=inputs["C"], bias=inputs["bias"], alpha=w.alpha, beta=w.beta,
                    batches=[0], rows=np.arange(nrows, dtype=np.int64), cols=cols)
        return time.perf_counter() - t0

    t1 = max(run(1), 1e-4)
    nrows = int(max(1, min(w.M, round(per_step / t1))))
    for _ in range(warmup):
        run(nrows)
    t0 = time.perf_counter()
    for _ in range(steps):
        run(nrows)
    sec = (time.perf_counter() - t0) / steps
    flops = 2.0 * nrows * w.N * w.K
    v = flops / sec / 1e12
    cores = oracle.max_threads()
    sample = f"each step: rows 0..{nrows - 1} x all {w.N} columns of batch 0 ({flops / 1e9:.2f} GFLOP)"
    print(json.dumps({
        "impl": "reference", "metric": "GEMM TFLOP/s at 1 B200 and % of dense bf16 roofline (HBM GB/s for skinny)",
        "value": round(v, 6), "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": steps, "warmup": warmup,
        "ms_per_step": round(sec * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "N": w.N, "K": w.K, "batch": w.batch, "sample": sample},
        "cpu_baseline": {"value": round(v, 6), "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(v, 6), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default="c2", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--flags", default="0", help="gemm_desc_t.flags override for the headline config (tuning)")
    ap.add_argument("--all", dest="all", action="store_true", default=True)
    ap.add_argument("--only", dest="all", action="store_false", help="time only --config (used for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--sustained-seconds", type=float, default=4.0, help="length of the sustained leg of the headline config (0 = skip)")
    ap.add_argument("--ref-step-seconds", type=float, default=10.0, help="--impl reference: CPU time budget of one step")
    ap.add_argument("--shapes", default="", help="';'-separated MxNxK[:key=value...] problems to time instead of the five configurations")
    ap.add_argument("--tune-file", default="", help="--shapes --tune: write the measured choices to this file (gemm_tune_cache_save)")
    ap.add_argument("--tune", action="store_true", help="--shapes: also plan by measurement (gemm_tune) and time the tuned plan")
    ap.add_argument("--library-reference", action="store_true", help="--shapes: also time torch.matmul on the same operands (context)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.shapes:
        run_shapes(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
