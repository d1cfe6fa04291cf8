#!/usr/bin/env python
"""Benchmark of the FPROP convolution hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--kernel fp32|tf32|bf16]
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference ...      # the CPU oracle on the host cores

One step = one FPROP convolution of the named workload (patch gather, inner
product, alpha scaling and store — one kernel launch) on synthetic seeded
inputs.  Prints ONE JSON line on rank 0.  Throughput is the paper's FLOP count
C = 2 Nb Wo Ho (Nc Sk^2 + 1) No (Section 2) divided by time.  The default is the
largest single-GPU layer (large3x3) through the exact fp32 kernel (the paper's
arithmetic); the same line carries, under "tensor_cores", the TF32 and BF16
tensor-core kernels on the same layer, each with its own time, clocks and
roofline.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_1501_06633_b200 import workloads as wl  # noqa: E402

METRIC = "conv FPROP TFLOPS (paper's FLOP formula)"
UNIT = "TFLOP/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
                  "sm_max_mhz": 1965.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the committed ncu summaries
# under profiles/ (None = not captured).  Writes still sitting in L2 when the kernel ends
# are not in these figures, which is why they are below the algorithmic bytes.
NCU_TRAFFIC_BYTES = {
    # fp32 plans with a split tail: both launches of a step (whole tiles + split tail)
    ("first11x11s4", "fp32"): int((79.71 + 93.40) * 1e6),
    ("mid5x5", "fp32"): int((38.00 + 33.58 + 8.44 + 0.0) * 1e6),
    ("wide3x3", "fp32"): int((24.82 + 0.21 + 8.24 + 0.0) * 1e6),
    ("large3x3", "fp32"): int((104.0 + 151.3 + 3.21 + 0.0) * 1e6),
    ("large3x3", "bf16"): int((52.02 + 146.8) * 1e6),
    ("large3x3", "tf32"): int((104.0 + 149.8) * 1e6),
    ("mid5x5", "bf16"): int((19.17 + 37.60) * 1e6),
    ("first11x11s4", "bf16"): int((39.67 + 89.99) * 1e6),
}


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=300)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="large3x3", choices=wl.ORDER + wl.TABLE1_ORDER)
    p.add_argument("--kernel", default="fp32", choices=["fp32", "tf32", "bf16", "tf32x3"])
    p.add_argument("--op", default="fprop", choices=["fprop", "dgrad", "wgrad"],
                   help="fprop (the headline path) or one of its two adjoints (BPROP)")
    p.add_argument("--e2e-steps", type=int, default=10)
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--nb", type=int, default=0,
                   help="override the workload's minibatch (a count that is not a multiple of 4 "
                        "goes through maxdnn_conv_fprop_ragged)")
    p.add_argument("--no-tensor", action="store_true",
                   help="skip the tensor-core kernels timed beside the fp32 headline")
    p.add_argument("--min-seconds", type=float, default=0.6,
                   help="length of the extra 'sustained' region behind the clock record")
    p.add_argument("--cpu-seconds", type=float, default=12.0,
                   help="target wall time of the CPU-baseline sample")
    return p.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload_bytes(w, kernel, op="fprop"):
    """Algorithmic HBM bytes of one step: every operand element read once, every
    result element written once (results are fp32)."""
    eb = 2 if kernel == "bf16" else 4
    Ho = (w.Hi + 2 * w.pad - w.Sk) // w.stride + 1
    Wo = (w.Wi + 2 * w.pad - w.Sk) // w.stride + 1
    maps, filt, out = w.Nc * w.Hi * w.Wi * w.Nb, w.Nc * w.Sk * w.Sk * w.No, w.No * Ho * Wo * w.Nb
    if op == "dgrad":
        return out * eb + filt * eb + maps * 4, Ho, Wo
    if op == "wgrad":
        return maps * eb + out * eb + filt * 4, Ho, Wo
    return maps * eb + filt * eb + out * 4, Ho, Wo


def flops(w, Ho, Wo):
    return 2 * w.Nb * Wo * Ho * (w.Nc * w.Sk * w.Sk + 1) * w.No


# ----------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of our arm, and the whole --impl reference arm)
# ----------------------------------------------------------------------------
def oracle_sample(w, target_seconds):
    """Time the oracle, as it stands, on a band of output rows of the workload
    sized to take about `target_seconds` (the whole workload, repeated, if that is
    shorter).  Returns (tflops, seconds, rows, Ho, repeats, threads)."""
    import oracle
    inp, filt = wl.make_inputs(w)
    Ho = (w.Hi + 2 * w.pad - w.Sk) // w.stride + 1
    Wo = (w.Wi + 2 * w.pad - w.Sk) // w.stride + 1
    y_mid = Ho // 2
    t0 = time.perf_counter()
    oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, rows=(y_mid, y_mid + 1))
    t_row = max(time.perf_counter() - t0, 1e-6)
    rows = int(max(1, min(Ho, target_seconds / t_row)))
    y0 = max(0, min(Ho - rows, y_mid - rows // 2))
    repeats = int(max(1, min(50, round(target_seconds / (t_row * rows)))))
    t0 = time.perf_counter()
    for _ in range(repeats):
        oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, rows=(y0, y0 + rows))
    dt = time.perf_counter() - t0
    fl = flops(w, rows, Wo) * repeats
    return fl / dt / 1e12, dt, rows, Ho, repeats, oracle.num_threads()


def oracle_single_thread_tiny():
    """The oracle on ONE thread on the small config: the per-core rate behind `cores`."""
    import oracle
    w = wl.WORKLOADS["tiny3x3"]
    inp, filt = wl.make_inputs(w)
    Ho = (w.Hi + 2 * w.pad - w.Sk) // w.stride + 1
    oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, nthreads=1)
    reps, t0 = 0, time.perf_counter()
    while reps < 3 or time.perf_counter() - t0 < 0.5:
        oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, nthreads=1)
        reps += 1
    dt = time.perf_counter() - t0
    return {"value": flops(w, Ho, Ho) * reps / dt / 1e12, "unit": UNIT, "cores": 1,
            "sample": "tiny3x3 whole x %d passes" % reps}


def oracle_sample_bprop(w, op, target_seconds):
    """The BPROP oracle on the first `cs` channels of the workload (a gradient with respect
    to a subset of channels is that subset of the work), sized to about `target_seconds`."""
    import oracle
    inp, filt = wl.make_inputs(w)
    dout = wl.make_dout(w)

    def run(cs):
        t0 = time.perf_counter()
        if op == "dgrad":
            oracle.conv_bprop_data(dout, filt[:cs], (w.Hi, w.Wi), stride=w.stride, pad=w.pad, alpha=w.alpha)
        else:
            oracle.conv_bprop_filter(inp[:cs], dout, w.Sk, stride=w.stride, pad=w.pad, alpha=w.alpha)
        return max(time.perf_counter() - t0, 1e-6)

    t1 = run(1)
    cs = int(max(1, min(w.Nc, target_seconds / t1)))
    dt = run(cs) if cs > 1 else t1
    Ho = (w.Hi + 2 * w.pad - w.Sk) // w.stride + 1
    Wo = (w.Wi + 2 * w.pad - w.Sk) // w.stride + 1
    fl = flops(w, Ho, Wo) * cs / w.Nc
    return fl / dt / 1e12, dt, cs, oracle.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = wl.ALL[args.workload]
    inp, filt = wl.make_inputs(w)
    Ho = (w.Hi + 2 * w.pad - w.Sk) // w.stride + 1
    Wo = (w.Wi + 2 * w.pad - w.Sk) // w.stride + 1
    y_mid = Ho // 2
    t0 = time.perf_counter()
    oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, rows=(y_mid, y_mid + 1))
    t_row = max(time.perf_counter() - t0, 1e-6)
    total = max(1, args.steps + args.warmup)
    budget = 150.0 / total                      # whole run within a few minutes
    rows = int(max(1, min(Ho, budget / t_row)))
    y0 = max(0, min(Ho - rows, y_mid - rows // 2))
    for _ in range(args.warmup):
        oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, rows=(y0, y0 + rows))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.conv_fprop(inp, filt, stride=w.stride, pad=w.pad, alpha=w.alpha, rows=(y0, y0 + rows))
    dt = time.perf_counter() - t0
    value = flops(w, rows, Wo) * args.steps / dt / 1e12
    sample = "%d of %d output rows of %s per step" % (rows, Ho, w.name)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "kernel": "cpu oracle", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a
    timed region runs."""

    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
        0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
        0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, device_index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            self._nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {
            "sm_mhz": float(np.median(self.samples)) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# ----------------------------------------------------------------------------
# multi-rank plumbing (also exercised on CPU with gloo by the tests)
# ----------------------------------------------------------------------------
def rank_env():
    """(rank, local_rank, world) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(values, device, world):
    """Element-wise maximum of a list of floats over all ranks."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def shard_inputs(w, rank):
    """Rank `rank`'s batch shard: same recipe, its own independent draw."""
    return wl.make_inputs(w, seed_offset=rank)


def sum_gradient_over_ranks(t, world):
    """The one data-path collective of the sharded job: the filter gradient of a minibatch
    split over ranks is the sum of the ranks' filter gradients (in place, all ranks)."""
    import torch.distributed as dist
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def whole_job_tflops(flops_per_rank, world, ms_step):
    return world * flops_per_rank / (ms_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------
def measure_tf32_peak():
    """Dense TF32 throughput of the library GEMM on this GPU (the roofline's denominator for
    the TF32 kernel): torch.matmul 8192^3 with TF32 enabled, best of 10, CUDA events."""
    import torch
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        n = 8192
        a = torch.randn(n, n, device="cuda")
        b = torch.randn(n, n, device="cuda")
        c = torch.empty(n, n, device="cuda")
        for _ in range(3):
            torch.matmul(a, b, out=c)
        best = None
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch.matmul(a, b, out=c)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old


def peak_for(kernel, peaks, peaks_kind, sm_count, tf32_measured=None):
    """(peak TFLOP/s, bound, where the number comes from) of one kernel kind."""
    sm_max = float(peaks.get("sm_max_mhz") or 1965.0)
    if kernel == "fp32":
        # FP32 CUDA-core peak, Section 3.3's form: 2 FLOPs x 128 cores x SMs x clock
        return (2.0 * 128 * sm_count * sm_max * 1e6 / 1e12, "alu",
                "2*128*%d SMs*%.0f MHz (max SM clock, %s); context: a bare packed-FMA stream "
                "measures 92.3 %% of this figure, the denominator stays the nominal one"
                % (sm_count, sm_max, peaks_kind))
    bf16 = float(peaks["bf16_tflops"])
    if kernel == "bf16":
        return bf16, "tensor", "cuBLAS bf16 burst (%s)" % peaks_kind
    half = 0.5 * bf16
    if tf32_measured is None:
        peak, note = half, "half of cuBLAS bf16 burst (%s) = %.0f; tf32 GEMM not measured" % (peaks_kind, half)
    else:
        peak = max(half, tf32_measured)
        note = ("larger of: torch.matmul 8192^3 tf32 best of 10, measured in this run = %.0f; half of "
                "cuBLAS bf16 burst (%s) = %.0f" % (tf32_measured, peaks_kind, half))
    if kernel == "tf32x3":
        return peak / 3.0, "tensor", note + "; / 3 (three TF32 products per product counted)"
    return peak, "tensor", note


class Arm:
    """One kernel kind on one workload and operation: device buffers (rotated so that no step
    finds its operands in L2) and the call that runs one step."""

    def __init__(self, mx, w, kernel, op, rank, world):
        import torch
        self.torch, self.mx, self.w, self.kernel, self.op, self.world = torch, mx, w, kernel, op, world
        x3 = kernel == "tf32x3"            # three TF32 products: fp32 buffers, its own entry points
        kind = {"fp32": mx.KERNEL_FP32, "tf32": mx.KERNEL_TF32, "bf16": mx.KERNEL_BF16,
                "tf32x3": mx.KERNEL_TF32}[kernel]
        self.kind, self.x3 = kind, x3
        self.ragged = op == "fprop" and kernel == "fp32" and bool(w.Nb % 4 or w.No % 4)
        d = self.d = mx.ConvDesc.make(*w.dims)
        self.nbytes, self.Ho, self.Wo = workload_bytes(w, kernel, op)
        self.C = mx.conv_flops(d)          # the same bilinear form: all three operations cost C
        assert self.C == flops(w, self.Ho, self.Wo)
        # Each rank holds its own batch shard (same recipe, its own seed); neither FPROP nor
        # the map gradient needs an exchange between shards; the filter gradient of a sharded
        # batch is summed over ranks (all-reduce, inside the timed step).
        inp, filt = shard_inputs(w, rank)
        dout = wl.make_dout(w, seed_offset=rank) if op != "fprop" else None
        n_sets = self.n_sets = max(2, int(np.ceil(3.0 * L2_BYTES / self.nbytes)))
        if kernel == "bf16":
            to_host = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).reshape(-1)
            as_op = lambda t: t.view(torch.bfloat16)
        else:
            to_host = lambda a: torch.from_numpy(a).reshape(-1)
            as_op = lambda t: t
        # operands: (big streamed operand, second operand); result: fp32
        if op == "fprop":
            h_a, h_b, n_res = to_host(inp), to_host(filt), mx.conv_out_elems(d)
        elif op == "dgrad":
            h_a, h_b, n_res = to_host(dout), to_host(filt), mx.conv_in_elems(d)
        else:
            h_a, h_b, n_res = to_host(inp), to_host(dout), mx.conv_filt_elems(d)
        self.h_a, self.h_b, self.n_res = h_a.pin_memory(), h_b.pin_memory(), n_res
        self.d_as = [self.h_a.cuda() for _ in range(n_sets)]
        self.d_bs = [self.h_b.cuda() for _ in range(n_sets if op == "wgrad" else 2)]
        self.d_res = [torch.empty(n_res, dtype=torch.float32, device="cuda") for _ in range(n_sets)]
        ws = None
        if op == "dgrad":
            ws = torch.empty(mx.conv_bprop_data_workspace(d, kind), dtype=torch.uint8, device="cuda")
        elif op == "wgrad":
            ws = torch.empty(max(16, mx.conv_bprop_filter_workspace(d, kind)), dtype=torch.uint8,
                             device="cuda")
        fprop = {mx.KERNEL_FP32: mx.conv_fprop, mx.KERNEL_TF32: mx.conv_fprop_tf32,
                 mx.KERNEL_BF16: mx.conv_fprop_bf16}[kind]
        # one call of the operation: run(a, b, r, workspace, stream)
        if x3:
            size_fn, call_fn = {
                "fprop": (mx.conv_fprop_tf32x3_workspace, mx.conv_fprop_tf32x3),
                "dgrad": (mx.conv_bprop_data_tf32x3_workspace, mx.conv_bprop_data_tf32x3),
                "wgrad": (mx.conv_bprop_filter_tf32x3_workspace, mx.conv_bprop_filter_tf32x3)}[op]
            ws = torch.empty(max(16, size_fn(d)), dtype=torch.uint8, device="cuda")
            self.run = lambda a, b, r, wsp, stream=None: call_fn(d, a, b, r, wsp, stream=stream)
        elif op == "fprop" and kernel == "fp32" and (w.Nb % 4 or w.No % 4):
            # counts outside the 16-byte row rule: the ragged entry point (fp32: in-kernel staging)
            ws = torch.empty(max(16, mx.conv_fprop_ragged_workspace(d, kind)), dtype=torch.uint8,
                             device="cuda")
            self.run = lambda a, b, r, wsp, stream=None: mx.conv_fprop_ragged(d, a, b, r, wsp, kind,
                                                                              stream=stream)
        elif op == "fprop":
            self.run = lambda a, b, r, wsp, stream=None: fprop(d, as_op(a), as_op(b), r, stream=stream)
        elif op == "dgrad":
            self.run = lambda a, b, r, wsp, stream=None: mx.conv_bprop_data(
                d, as_op(a), as_op(b), r, wsp, kind, stream=stream)
        else:
            self.run = lambda a, b, r, wsp, stream=None: mx.conv_bprop_filter(
                d, as_op(a), as_op(b), r, wsp, kind, stream=stream)
        self.ws = ws

    def step(self, i):
        a, b, r = self.d_as[i % self.n_sets], self.d_bs[i % len(self.d_bs)], self.d_res[i % self.n_sets]
        self.run(a, b, r, self.ws)
        if self.op == "wgrad":
            sum_gradient_over_ranks(r, self.world)      # NCCL all-reduce over the batch shards

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def timed(self, steps, warmup, local_rank):
        """W warm-up steps, then EXACTLY `steps` steps between two events, a barrier and a
        synchronize on both sides.  Returns (ms of the region, clock record, launches)."""
        torch, mx = self.torch, self.mx
        for i in range(max(3, warmup)):
            self.step(i)
        self.barrier()
        sampler = ClockSampler(local_rank)
        launches0 = mx.launch_count()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.start()
        self.barrier()
        ev0.record()
        for i in range(steps):
            self.step(i)
        ev1.record()
        self.barrier()
        clocks = sampler.stop()
        launches = mx.launch_count() - launches0
        if mx.last_device_status() != mx.OK:
            raise SystemExit("a kernel reported a timed-out wait; results are not valid")
        return ev0.elapsed_time(ev1), clocks, launches

    def per_launch(self, n):
        """Events around each of `n` steps: (median ms, best ms)."""
        torch = self.torch
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(n)]
        self.barrier()
        for i, (e0, e1) in enumerate(evs):
            e0.record()
            self.step(i)
            e1.record()
        self.barrier()
        ms = sorted(e0.elapsed_time(e1) for e0, e1 in evs)
        return float(np.median(ms)), float(ms[0])

    def sustained(self, steps, seconds, local_rank):
        """The timed loop repeated until at least `seconds` have passed: a region long enough
        for the clock record (NVML samples every 2 ms) to mean something."""
        torch = self.torch
        sampler = ClockSampler(local_rank)
        sampler.start()
        self.barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        done = 0
        ev0.record()
        while True:
            for i in range(steps):
                self.step(i)
            done += steps
            torch.cuda.current_stream().synchronize()
            if time.perf_counter() - t0 >= seconds or done >= 200000:
                break
        ev1.record()
        self.barrier()
        clocks = sampler.stop()
        return ev0.elapsed_time(ev1) / done, done, clocks


def roofline_of(arm, ms_step, peak, bound, peak_note, peaks):
    per_gpu = arm.C / (ms_step * 1e-3) / 1e12
    t_compute = arm.C / (peak * 1e12)
    t_hbm = arm.nbytes / (float(peaks["hbm_gbs"]) * 1e9)
    return {
        "bound": bound, "achieved": per_gpu, "peak": peak, "unit": "TFLOP/s", "frac": per_gpu / peak,
        "traffic": NCU_TRAFFIC_BYTES.get((arm.w.name, arm.kernel)) if arm.op == "fprop" else None,
        "peak_source": peak_note,
        "roofline_time_us": max(t_compute, t_hbm) * 1e6,
        "frac_of_roofline_time": max(t_compute, t_hbm) / (ms_step * 1e-3),
        "achieved_hbm_gbs": arm.nbytes / (ms_step * 1e-3) / 1e9,
    }


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_1501_06633_b200 as mx

    rank, local_rank, world = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    peaks, peaks_kind = load_peaks()
    w = wl.ALL[args.workload]
    if args.nb > 0:
        w = w.scaled(Nb=args.nb)
    op = args.op
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    arm = Arm(mx, w, args.kernel, op, rank, world)
    d, C, n_sets, nbytes = arm.d, arm.C, arm.n_sets, arm.nbytes
    x3, kind = arm.x3, arm.kind

    ms_total, clocks, launches = arm.timed(args.steps, args.warmup, local_rank)

    # the same launches one by one (median / best beside the batch mean), then a region of
    # at least --min-seconds for the clock record
    pl_median, pl_best = arm.per_launch(max(3, min(args.steps, 50)))
    sus_ms, sus_steps, sus_clocks = arm.sustained(max(1, args.steps), args.min_seconds, local_rank)

    # Section 3.3's efficiency counts processor clocks: elapsed SM cycles measured inside the
    # kernel (maximum over its CTAs), fp32 FPROP only
    kernel_clock = None
    if args.kernel == "fp32" and op == "fprop":
        mx.set_option("KERNEL_CLOCK", 1)
        cyc = []
        for i in range(5):
            arm.step(i)
            cyc.append(mx.last_kernel_clock())
        mx.unset_option("KERNEL_CLOCK")
        cyc.sort()
        c_cycles, c_ns = cyc[len(cyc) // 2]
        if c_cycles > 0 and c_ns > 0:
            kernel_clock = {"sm_cycles": c_cycles, "ns": c_ns, "sm_mhz": c_cycles / c_ns * 1e3,
                            "ce_cycles": C / (2.0 * 128 * sm_count * c_cycles)}

    # end to end from pinned host buffers: host -> device copies of both operands, the
    # kernel(s), device -> host copy of the result, every step.  FPROP goes through
    # maxdnn_conv_fprop_host; the gradients through the same copies around their call.
    # Steps alternate between two streams, each with its own device and result buffers,
    # so that one step's result copy (device -> host) overlaps the next step's operand
    # copies (host -> device): the link is full duplex.  Every step still moves all its
    # bytes; the single-stream figure is reported beside it.
    h_a, h_b, n_res = arm.h_a, arm.h_b, arm.n_res
    d_as, d_bs, d_res, ws, run = arm.d_as, arm.d_bs, arm.d_res, arm.ws, arm.run
    barrier = arm.barrier
    h_outs = [torch.empty(n_res, dtype=torch.float32).pin_memory() for _ in range(2)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]

    def e2e_step(k, stream):
        a, b, r = d_as[k % n_sets], d_bs[k % len(d_bs)], d_res[k % n_sets]
        if op == "fprop" and not x3 and not arm.ragged:
            mx.conv_fprop_host(d, kind, h_a, h_b, h_outs[k], a, b, r, stream=stream)
        else:
            with torch.cuda.stream(stream):
                a.copy_(h_a, non_blocking=True)
                b.copy_(h_b, non_blocking=True)
                run(a, b, r, ws_e2e[k], stream=stream)
                h_outs[k].copy_(r, non_blocking=True)

    ws_e2e = [ws, None if ws is None else torch.empty_like(ws)]
    e2e_steps = max(1, min(args.steps, args.e2e_steps))

    def time_e2e(n_streams):
        cur = torch.cuda.current_stream()
        for k in range(2):
            e2e_step(k % n_streams, streams[k % n_streams])
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for st in streams[:n_streams]:
            st.wait_event(e0)
        for k in range(e2e_steps):
            e2e_step(k % n_streams, streams[k % n_streams])
        for st in streams[:n_streams]:
            cur.wait_stream(st)
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    e2e_ms_single = time_e2e(1)
    e2e_ms = time_e2e(2)
    if mx.last_device_status() != mx.OK:
        raise SystemExit("a kernel reported a timed-out wait; results are not valid")

    # Beside the exact fp32 headline: the same workload on the tensor cores (TF32 and BF16
    # operands, fp32 accumulate), each timed like the headline — W warm-ups, then the same
    # number of steps between two events — with its own clock record and roofline.
    tensor = None
    tf32_measured = None
    if world == 1 and op == "fprop" and args.kernel in ("fp32", "tf32", "tf32x3"):
        tf32_measured = measure_tf32_peak()
    if world == 1 and args.kernel == "fp32" and op == "fprop" and not args.no_tensor:
        del arm.d_as, arm.d_bs, arm.d_res
        d_as = d_bs = d_res = None
        torch.cuda.empty_cache()
        tensor = {}
        for k in ("tf32", "bf16"):
            try:
                t_arm = Arm(mx, w, k, "fprop", rank, world)
                t_ms, t_clocks, t_launches = t_arm.timed(args.steps, args.warmup, local_rank)
                t_med, t_best = t_arm.per_launch(max(3, min(args.steps, 50)))
                s_ms, s_steps, s_clocks = t_arm.sustained(max(1, args.steps), args.min_seconds, local_rank)
            except mx.MaxdnnError as e:
                tensor[k] = {"unavailable": str(e)}       # a shape this kernel does not take
                continue
            t_step = t_ms / args.steps
            peak, bound, note = peak_for(k, peaks, peaks_kind, sm_count, tf32_measured)
            tensor[k] = {
                "value": whole_job_tflops(C, 1, t_step), "unit": UNIT, "ms_per_step": t_step,
                "steps": args.steps, "warmup": max(3, args.warmup), "gpu_launches": int(t_launches),
                "per_launch": {"median_ms": t_med, "best_ms": t_best},
                "sustained": {"ms_per_step": s_ms, "steps": s_steps, "value": whole_job_tflops(C, 1, s_ms),
                              "clocks": s_clocks},
                "clocks": t_clocks,
                "roofline": roofline_of(t_arm, t_step, peak, bound, note, peaks),
            }
            del t_arm
            torch.cuda.empty_cache()

    ms_total, e2e_ms, e2e_ms_single = max_over_ranks([ms_total, e2e_ms, e2e_ms_single], "cuda", world)
    ms_step = ms_total / args.steps
    value = whole_job_tflops(C, world, ms_step)
    e2e_value = whole_job_tflops(C, world, e2e_ms / e2e_steps)

    if rank == 0:
        peak, bound, peak_note = peak_for(args.kernel, peaks, peaks_kind, sm_count, tf32_measured)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": {"fp32": "f32", "tf32": "tf32", "bf16": "bf16", "tf32x3": "tf32x3"}[args.kernel],
            "data": "synthetic",
            "config": {
                "workload": w.name, "op": op, "kernel": args.kernel, "Nb": w.Nb, "Wi": w.Wi, "Hi": w.Hi,
                "Nc": w.Nc, "No": w.No, "Sk": w.Sk, "stride": w.stride, "pad": w.pad,
                "alpha": w.alpha, "flops_per_step": C, "algorithmic_bytes_per_step": nbytes,
                "l2": "rotating %d buffer sets (%.0f MB) > L2 (126 MB)" % (n_sets, n_sets * nbytes / 1e6),
                "parallelism": ("single GPU" if world == 1 else
                                "batch shards, filter gradient all-reduced" if op == "wgrad" else
                                "batch shards, no collective"),
            },
            "clocks": clocks,
            "per_launch": {"median_ms": pl_median, "best_ms": pl_best,
                           "best_value": whole_job_tflops(C, world, pl_best)},
            "sustained": {"ms_per_step": sus_ms, "steps": sus_steps,
                          "value": whole_job_tflops(C, world, sus_ms), "clocks": sus_clocks,
                          "note": "the timed loop repeated for at least %.1f s" % args.min_seconds},
            "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps, "streams": 2,
                    "value_single_stream": whole_job_tflops(C, world, e2e_ms_single / e2e_steps),
                    "h2d_bytes_per_step": int(h_a.numel() * h_a.element_size()
                                              + h_b.numel() * h_b.element_size()),
                    "d2h_bytes_per_step": int(n_res * 4)},
            "gpu_launches": int(launches),
            "roofline": roofline_of(arm, ms_step, peak, bound, peak_note, peaks),
        }
        if (clocks.get("samples") or 0) < 50:
            line["clocks"]["note"] = ("fewer than 50 clock samples in the %d-step region; see "
                                      "sustained.clocks" % args.steps)
        if tensor is not None:
            line["tensor_cores"] = tensor
        if kernel_clock is not None:
            # the paper's clock-independent efficiency: C / (2*128*SMs*elapsed SM cycles)
            line["roofline"]["ce_cycles"] = kernel_clock["ce_cycles"]
            line["roofline"]["kernel_clock"] = kernel_clock
        if clocks.get("sm_mhz"):
            cycles = ms_step * 1e-3 * clocks["sm_mhz"] * 1e6
            line["roofline"]["ce_at_sampled_clock"] = C / (2.0 * 128 * sm_count * cycles)
        if world == 1 and not args.no_cpu_baseline and op != "fprop":
            tf, secs, cs, threads = oracle_sample_bprop(w, op, args.cpu_seconds)
            line["cpu_baseline"] = {
                "value": tf, "unit": UNIT, "cores": threads, "kind": "oracle",
                "sample": "%s of %s restricted to %d of %d channels, %.1f s" % (op, w.name, cs, w.Nc, secs)}
        elif world == 1 and not args.no_cpu_baseline:
            tf, secs, rows, Ho_, reps, threads = oracle_sample(w, args.cpu_seconds)
            line["cpu_baseline"] = {
                "value": tf, "unit": UNIT, "cores": threads, "kind": "oracle",
                "sample": "%d of %d output rows of %s x %d passes, %.1f s" % (rows, Ho_, w.name,
                                                                            reps, secs),
                "single_thread_tiny3x3": oracle_single_thread_tiny()}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
