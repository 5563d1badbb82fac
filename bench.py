#!/usr/bin/env python
"""Throughput of the MMSE quantization search on the ResNet-50-shaped weight set.

One step = the whole hot path over one batch of synthetic input: every one of the 54 weight
tensors goes through omse_quantize_weights_batched (stage, max, 1024-candidate sweep, argmin,
3 polish steps, codes, INT4 packing; one launch for the set).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

--workload selects one of the other configurations (c1, c3, c4, c5:K:bits) for measurement and
profiling; the default c2 is the one the metric is quoted on.

With N > 1 (launched under torch.distributed.run) every rank quantizes its own copy of the
weight set (different seed): kernels of different tensors are independent, so there is no
data-path collective; only the timing is reduced (max over ranks).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

N_CAND, BITS, REFINE, HI_FRAC = 1024, 4, 3, 1.0
METRIC = "elements quantized/sec (4-bit MMSE search)"
INSTR_PER_EVAL = 6            # reference FP32 sequence per (element, candidate): 3 fma + 2 min/max + 1 add
LANE_OPS_PER_EVAL = 4         # FMA-pipe lane operations of an evaluation the kernels execute: fma, add, fma, fma
# dram__bytes_read.sum + dram__bytes_write.sum of one step of the default workload (its two launches of the row kernel:
# rows of up to 640 elements, and the longer ones beside them) from an ncu capture; None whenever the kernels have changed
# since the capture
NCU_TRAFFIC_BYTES = 105_624_064
E2E_CHUNKS = 12               # batched launches per end-to-end step (copies of later chunks overlap earlier searches)
N_SM, LANES_PER_SM = 148, 128
WORKLOAD = "resnet50_weight_set_54_tensors_25.5M_params_signed4bit_kernelwise_1024cand_3refine_packed"


def _hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        if d.get("hbm_gbs"):
            return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json: copy bandwidth)"
    return 6650.0, "fallback (6.65 TB/s, an earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi sampler running beside the timed region."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        clocks, reasons, mx, power = [], set(), None, []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                clocks.append(float(parts[0]))
                mx = float(parts[1])
                power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        if clocks:
            busy = [c for c, p in zip(clocks, power) if p > 0.5 * max(power)] or clocks
            out.update(sm_mhz=float(np.median(busy)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(clocks),
                       power_w_max=max(power))
        return out


def max_over_ranks(ms_local: float, dist, device) -> float:
    """Slowest rank's time (every multi-GPU number is the max over ranks); identity without a process group."""
    if dist is None:
        return ms_local
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(n_per_rank: int, world: int, ms_total: float, steps: int) -> float:
    """Elements per second over all ranks: each rank quantizes its own copy of the set (weak scaling)."""
    return world * n_per_rank / (ms_total * 1e-3 / steps)


def rank_seed(rank: int) -> int:
    return 2 + 1000 * rank


# --------------------------------------------------------------------------------------------------
# Workloads.  "c2" (the ResNet-50-shaped weight set) is the one the metric is quoted on and the
# default; the others are the remaining configurations, selectable for measurement and profiling.
# Every workload gives: device-resident step, end-to-end step (host buffers), byte counts, and a
# bounded sample for the oracle.
# --------------------------------------------------------------------------------------------------
def _time_oracle_rows(samples, bits, n_cand, packed=True):
    from oracle import omse_oracle as orc
    orc.build()
    t0 = time.perf_counter()
    for w in samples:
        r = orc.quantize_rows(w, bits, True, n_cand, HI_FRAC, REFINE)
        if packed:
            orc.pack_int4(r.codes)
    dt = time.perf_counter() - t0
    n = sum(w.size for w in samples)
    return n / dt, dt, n, orc.max_threads()


class Workload:
    name = ""
    n_cand = N_CAND
    evals_per_element = 1        # quantized tensors searched per element
    kernel = "rows_kernel<8>"

    def host_arrays(self):       # list of numpy inputs
        raise NotImplementedError

    def algorithmic_bytes(self):  # HBM bytes one step has to move: inputs read once, outputs written once
        return self.h2d + self.d2h

    def release(self):           # drop device and pinned buffers
        for k in list(self.__dict__):
            if k not in ("name", "n_cand", "n_total", "h2d", "d2h", "evals_per_element"):
                delattr(self, k)


class WeightSet(Workload):
    """One or more weight tensors through the batched kernel-wise call."""

    def __init__(self, name, tensors, bits, n_cand, packed, sample_stride, sample_desc):
        self.name, self.tensors, self.bits, self.n_cand, self.packed = name, tensors, bits, n_cand, packed
        self.sample_stride, self.sample_desc = sample_stride, sample_desc

    def host_arrays(self):
        return self.tensors

    def setup(self, ctx, torch, dev):
        self.host_in = [torch.from_numpy(w).pin_memory() for w in self.tensors]
        self.d_w = [h.to(dev) for h in self.host_in]
        self.outs = []
        for w in self.tensors:
            s, k = w.shape
            code = (torch.empty((s * k + 1) // 2, dtype=torch.uint8, device=dev) if self.packed
                    else torch.empty(s * k, dtype=torch.int8, device=dev))
            self.outs.append((torch.empty(s, device=dev), torch.empty(s, device=dev), code))
        self.host_out = [tuple(t.cpu().pin_memory() for t in o) for o in self.outs]
        key = "packed" if self.packed else "codes"
        descs = [dict(w=dw, n_kernels=w.shape[0], kernel_len=w.shape[1], alpha=a, sse=e, **{key: c})
                 for w, dw, (a, e, c) in zip(self.tensors, self.d_w, self.outs)]
        self.n_total = sum(w.size for w in self.tensors)
        self.h2d = 4 * self.n_total
        self.d2h = sum(a.numel() * 4 + e.numel() * 4 + c.numel() for a, e, c in self.outs)

        def step():   # every tensor in one launch: kernels of all layers are handed out longest first
            ctx.omse_quantize_weights_batched(descs, self.bits, True, self.n_cand, HI_FRAC, REFINE)
        self.step = step

        # End-to-end: the host->device copies of later tensors run under the search of earlier ones.
        # Tensors go longest rows first in E2E_CHUNKS chunks of equal bytes; each chunk is one batched launch.
        order = sorted(range(len(descs)), key=lambda i: -self.tensors[i].shape[1])
        n_chunks = min(E2E_CHUNKS, len(descs))
        target, acc, self.chunks, cur = self.n_total / n_chunks, 0, [], []
        for i in order:
            cur.append(i)
            acc += self.tensors[i].size
            if acc >= target * (len(self.chunks) + 1) and len(self.chunks) < n_chunks - 1:
                self.chunks.append(cur)
                cur = []
        if cur:
            self.chunks.append(cur)
        self.h2d_stream, self.d2h_stream = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        self._torch, self._ctx, self._descs = torch, ctx, descs

    def step_e2e(self):
        torch, ctx = self._torch, self._ctx
        main = torch.cuda.current_stream()
        self.h2d_stream.wait_stream(main)          # inputs of the previous step are no longer in use
        self.d2h_stream.wait_stream(main)
        ready = []
        with torch.cuda.stream(self.h2d_stream):
            for ch in self.chunks:
                for i in ch:
                    self.d_w[i].copy_(self.host_in[i], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(self.h2d_stream)
                ready.append(ev)
        for ch, ev in zip(self.chunks, ready):
            main.wait_event(ev)
            ctx.omse_quantize_weights_batched([self._descs[i] for i in ch], self.bits, True, self.n_cand, HI_FRAC,
                                              REFINE)
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(self.d2h_stream):
                self.d2h_stream.wait_event(done)
                for i in ch:
                    for t, h in zip(self.outs[i], self.host_out[i]):
                        h.copy_(t, non_blocking=True)
        main.wait_stream(self.d2h_stream)          # the step ends when its results are on the host

    def cpu(self):
        samples = [np.ascontiguousarray(w[::self.sample_stride]) for w in self.tensors]
        v, dt, n, cores = _time_oracle_rows(samples, self.bits, self.n_cand, self.packed)
        return v, cores, f"{self.sample_desc} ({n} elements, {dt:.1f} s)", n


class Activation(Workload):
    kernel = "tensor_sweep_kernel<8>"

    def __init__(self, name, x, n_cand):
        self.name, self.x, self.n_cand = name, x, n_cand

    def host_arrays(self):
        return [self.x]

    def algorithmic_bytes(self):  # maximum, sweep, polish steps and the final error each read the tensor once
        return 4 * self.n_total * (3 + REFINE)

    def setup(self, ctx, torch, dev):
        self.host_in = torch.from_numpy(self.x).pin_memory()
        self.d_x = self.host_in.to(dev)
        self.out = (torch.empty(1, device=dev), torch.empty(1, device=dev))
        self.host_out = tuple(t.cpu().pin_memory() for t in self.out)
        self.n_total = self.x.size
        self.h2d, self.d2h = 4 * self.n_total, 8

        def step():
            ctx.omse_activation_scale(self.d_x, self.n_total, BITS, False, self.n_cand, HI_FRAC, REFINE, *self.out)
        self.step = step

    def step_e2e(self):
        self.d_x.copy_(self.host_in, non_blocking=True)
        self.step()
        for t, h in zip(self.out, self.host_out):
            h.copy_(t, non_blocking=True)

    def cpu(self):
        from oracle import omse_oracle as orc
        sub = np.ascontiguousarray(self.x[: 1 << 21])       # the per-tensor search on the first 2M elements
        t0 = time.perf_counter()
        orc.activation_scale(sub, BITS, False, self.n_cand, HI_FRAC, REFINE)
        dt = time.perf_counter() - t0
        return (sub.size / dt, orc.max_threads(),
                f"first {sub.size} elements of the tensor, all {self.n_cand} candidates ({dt:.1f} s)", sub.size)


class Residual(Workload):
    evals_per_element = 2

    def __init__(self, name, t, n_cand):
        self.name, self.t, self.n_cand = name, t, n_cand

    def host_arrays(self):
        return [self.t]

    def setup(self, ctx, torch, dev):
        s, k = self.t.shape
        self.host_in = torch.from_numpy(self.t).pin_memory()
        self.d_t = self.host_in.to(dev)
        self.out = (torch.empty(2, s, device=dev), torch.empty(2, s, device=dev),
                    torch.empty(2, (s * k + 1) // 2, dtype=torch.uint8, device=dev))
        self.host_out = tuple(t.cpu().pin_memory() for t in self.out)
        self.n_total = s * k
        self.h2d, self.d2h = 4 * self.n_total, sum(t.numel() * t.element_size() for t in self.out)

        def step():
            ctx.omse_residual_quantize(self.d_t, s, k, [BITS, BITS], True, self.n_cand, HI_FRAC, REFINE, 1,
                                       self.out[0], self.out[1], None, self.out[2])
        self.step = step

    def step_e2e(self):
        self.d_t.copy_(self.host_in, non_blocking=True)
        self.step()
        for t, h in zip(self.out, self.host_out):
            h.copy_(t, non_blocking=True)

    def cpu(self):
        from oracle import omse_oracle as orc
        sub = np.ascontiguousarray(self.t[::64])
        t0 = time.perf_counter()
        orc.residual_rows(sub, (BITS, BITS), True, self.n_cand, HI_FRAC, REFINE, 1)
        dt = time.perf_counter() - t0
        return sub.size / dt, orc.max_threads(), f"every 64th kernel ({sub.size} elements, {dt:.1f} s)", sub.size


class Dual(Workload):
    """Dual line search (Section 3.5, n = 2) on one convolution-shaped tensor."""
    kernel = "dual_kernel"
    instr_per_eval = 7           # per (element, pair, first code): fma, fma, max, min, add, fma, mul+min
    C1 = C2 = 32
    HF2 = 0.25

    def __init__(self, name, t):
        self.name, self.t = name, t
        self.n_cand = self.C1 * self.C2
        self.evals_per_element = 1 << BITS          # first codes enumerated per pair

    def host_arrays(self):
        return [self.t]

    def setup(self, ctx, torch, dev):
        s, k = self.t.shape
        self.host_in = torch.from_numpy(self.t).pin_memory()
        self.d_t = self.host_in.to(dev)
        self.out = (torch.empty(2, s, device=dev), torch.empty(s, device=dev),
                    torch.empty(2, (s * k + 1) // 2, dtype=torch.uint8, device=dev))
        self.host_out = tuple(t.cpu().pin_memory() for t in self.out)
        self.n_total = s * k
        self.h2d, self.d2h = 4 * self.n_total, sum(t.numel() * t.element_size() for t in self.out)

        def step():
            ctx.omse_dual_quantize(self.d_t, s, k, BITS, BITS, True, self.C1, self.C2, HI_FRAC, self.HF2,
                                   self.out[0], self.out[1], None, None, self.out[2])
        self.step = step

    def step_e2e(self):
        self.d_t.copy_(self.host_in, non_blocking=True)
        self.step()
        for t, h in zip(self.out, self.host_out):
            h.copy_(t, non_blocking=True)

    def cpu(self):
        from oracle import omse_oracle as orc
        sub = np.ascontiguousarray(self.t[::32])
        t0 = time.perf_counter()
        orc.dual_rows(sub, BITS, BITS, True, self.C1, self.C2, HI_FRAC, self.HF2)
        dt = time.perf_counter() - t0
        return sub.size / dt, orc.max_threads(), f"every 32nd kernel ({sub.size} elements, {dt:.1f} s)", sub.size


def make_workload(spec: str, rank: int):
    from paper_1902_06822_b200 import synth
    if spec == "c2":
        ws = [w for _, w in synth.resnet50_weights(seed=rank_seed(rank))]
        return WeightSet(WORKLOAD, ws, BITS, N_CAND, True, 4, "every 4th kernel of each of the 54 tensors")
    if spec == "c1":
        return WeightSet("single_conv_layer_64x576_signed4bit_256cand_3refine_int8", [synth.conv_layer(1 + rank)],
                         BITS, 256, False, 1, "all 64 kernels")
    if spec == "c1x64":
        ws = [synth.conv_layer(100 + 64 * rank + i) for i in range(64)]
        return WeightSet("64_conv_layers_64x576_signed4bit_256cand_3refine_int8_one_batched_launch", ws, BITS, 256, False,
                         4, "every 4th kernel of each of the 64 tensors")
    if spec == "c3":
        return Activation("activation_64x256x56x56_unsigned4bit_per_tensor_2048cand_3refine",
                          synth.activation_tensor(seed=3 + 1000 * rank), 2048)
    if spec == "c4":
        return Residual("vgg16_fc6_4096x25088_residual_two_tensors_signed4bit_1024cand_3refine_packed",
                        synth.fc6_weights(seed=4 + 1000 * rank), N_CAND)
    if spec.startswith("c5"):          # c5:K:bits
        _, k, bits = spec.split(":")
        k, bits = int(k), int(bits)
        w = synth.sweep_tensor(k, seed=5 + 1000 * rank)
        stride = max(1, w.shape[0] // max(1, (6_000_000 // k)))
        return WeightSet(f"sweep_64M_student_t_K{k}_signed{bits}bit_1024cand_3refine", [w], bits, N_CAND, bits <= 4,
                         stride, f"every {stride}th kernel")
    if spec == "dual":
        w = synth.laplace(512 * 4608, 1.0 / np.sqrt(4608.0), 6 + 1000 * rank).reshape(512, 4608)
        return Dual("dual_line_search_512x4608_conv_signed4bit_x2_32x32_grid_packed", w)
    raise SystemExit(f"unknown workload {spec}")


def base_config(wl, n_total):
    """The keys both arms print under "config"."""
    return {"workload": wl.name, "elements_per_gpu": n_total, "n_cand": wl.n_cand, "refine_iters": REFINE,
            "l2": "flushed between timed steps (256 MB write)"}


def run_reference(args, rank):
    """The oracle, as it stands, on the host cores; each step is the workload's bounded sample."""
    if rank != 0:
        return
    wl = make_workload(args.workload, 0)
    n_total = sum(a.size for a in wl.host_arrays())
    # Size the per-step sample so that all the steps together take about a minute on this host: one
    # calibration call on the standard sample, then a coarser row stride if the run would be longer.
    if hasattr(wl, "sample_stride"):
        t0 = time.perf_counter()
        wl.cpu()
        t_step = time.perf_counter() - t0
        budget_s = 60.0
        if t_step * args.steps > budget_s:
            factor = int(np.ceil(t_step * args.steps / budget_s))
            wl.sample_stride *= factor
            wl.sample_desc = wl.sample_desc.replace("every 4th", f"every {wl.sample_stride}th")
    total_t, n = 0.0, 0
    for _ in range(args.steps):
        t0 = time.perf_counter()
        _, cores, desc, n = wl.cpu()
        total_t += time.perf_counter() - t0
    value = n * args.steps / total_t
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value,
        "unit": "elements/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": base_config(wl, n_total),
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Timer:
    """CUDA-event timing of `steps` calls with an L2 flush before each (the flush is not timed)."""

    def __init__(self, torch, stream, dev, dist):
        self.torch, self.stream, self.dev, self.dist = torch, stream, dev, dist
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def run(self, fn, steps):
        torch = self.torch
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        self.barrier()
        for s0, s1 in ev:
            self.flush.fill_(1)         # evict the inputs from L2 between timed steps
            s0.record(self.stream)
            fn()
            s1.record(self.stream)
        self.barrier()
        return max_over_ranks(sum(s0.elapsed_time(s1) for s0, s1 in ev), self.dist, self.dev)


def roofline_of(wl, n_total, per_step_s, executed, fma_peak, hbm_gbs):
    """Executed work against the two roofs: FP32 lane operations of the FMA pipe (4 per executed evaluation:
    fma, add, fma, fma) and algorithmic HBM bytes; the fraction is the larger of the two, i.e. roof time / time."""
    evals = wl.n_cand * wl.evals_per_element * n_total                      # all (element, candidate) pairs
    ipe = getattr(wl, "instr_per_eval", INSTR_PER_EVAL)
    lane_ops = LANE_OPS_PER_EVAL * executed
    bytes_algo = wl.algorithmic_bytes()
    frac_fma = lane_ops / per_step_s / fma_peak
    frac_hbm = bytes_algo / per_step_s / (hbm_gbs * 1e9)
    return {"bound": "alu", "achieved": lane_ops / per_step_s / 1e12, "peak": fma_peak / 1e12,
            "unit": "T FP32 lane-op/s", "frac": max(frac_fma, frac_hbm), "frac_fma_pipe": frac_fma, "frac_hbm": frac_hbm,
            "kernel": wl.kernel, "lane_ops_per_executed_evaluation": LANE_OPS_PER_EVAL,
            "executed_evaluations_per_step": executed, "executed_share": executed / evals,
            "algorithmic_bytes_per_step": bytes_algo,
            # speed against a kernel that evaluates every pair with the 6-instruction reference sequence at this peak
            "speed_vs_exhaustive": ipe * evals / per_step_s / fma_peak}


def measure(wl, ctx, timer, steps, warmup):
    """Device-resident timing of one workload: ms per step and executed evaluations per step."""
    for _ in range(max(warmup, 3)):
        wl.step()
    timer.torch.cuda.synchronize()
    ctx.omse_read_evaluations()                     # clear the instrumentation counters
    ctx.omse_read_launches()
    ms = timer.run(wl.step, steps)
    executed = ctx.omse_read_evaluations() / steps
    wl.launches_timed = ctx.omse_read_launches()    # kernels of this library launched inside the timed region
    return ms, executed


PER_CONFIG = ["c1", "c1x64", "c3", "c4", "c5:27:4", "c5:576:4", "c5:4608:4", "c5:25088:4", "dual"]


def run_ours(args, rank, world):
    import torch
    from paper_1902_06822_b200 import binding, build
    build.build()
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    wl = make_workload(args.workload, rank)
    ctx = binding.Context(local)
    stream = torch.cuda.current_stream(dev)
    timer = Timer(torch, stream, dev, dist)
    wl.setup(ctx, torch, dev)
    n_total = wl.n_total
    hbm_gbs, hbm_src = _hbm_peak()

    # ---- the FP32 roof, measured in this process on this GPU (packed fma loop on every SM), clocks sampled beside it
    peak_sampler = ClockSampler(local) if rank == 0 else None
    ctx.omse_measure_fp32_peak(50)
    fma_peak = ctx.omse_measure_fp32_peak(400)
    peak_clocks = peak_sampler.stop() if peak_sampler else None

    # ---- the timed region proper
    sampler = ClockSampler(local) if rank == 0 else None
    ms, executed = measure(wl, ctx, timer, args.steps, args.warmup)
    clocks = sampler.stop() if sampler else None
    wl.step_e2e()
    ms_e2e = timer.run(wl.step_e2e, args.steps)
    status = ctx.omse_last_device_status()

    # ---- the same step repeated for seconds: does the clock hold under this kernel?
    sustained = None
    if world == 1 and not args.quick:
        n_long = int(min(20000, max(args.steps, np.ceil(2000.0 / (ms / args.steps)))))
        long_sampler = ClockSampler(local)
        ms_long = timer.run(wl.step, n_long)
        lc = long_sampler.stop()
        sustained = {"steps": n_long, "ms_per_step": ms_long / n_long, "value": n_total / (ms_long * 1e-3 / n_long),
                     "clocks": lc}

    # ---- the other configurations, a few steps each (the default line stays the one the metric is quoted on)
    per_config = None
    if world == 1 and not args.quick and args.workload == "c2":
        per_config = {}
        for spec in PER_CONFIG:
            w2 = make_workload(spec, rank)
            w2.setup(ctx, torch, dev)
            s2 = 5
            ms2, ex2 = measure(w2, ctx, timer, s2, 3)
            r2 = roofline_of(w2, w2.n_total, ms2 * 1e-3 / s2, ex2, fma_peak, hbm_gbs)
            per_config[spec] = {"workload": w2.name, "elements": w2.n_total, "steps": s2, "ms_per_step": ms2 / s2,
                                "value": w2.n_total / (ms2 * 1e-3 / s2), "executed_share": r2["executed_share"],
                                "frac": r2["frac"], "frac_fma_pipe": r2["frac_fma_pipe"], "frac_hbm": r2["frac_hbm"],
                                "speed_vs_exhaustive": r2["speed_vs_exhaustive"], "kernel": w2.kernel,
                                "gpu_launches": w2.launches_timed}
            w2.release()
            del w2
            torch.cuda.empty_cache()

    if rank == 0:
        per_step_s = ms * 1e-3 / args.steps
        value = whole_job_value(n_total, world, ms, args.steps)
        roof = roofline_of(wl, n_total, per_step_s, executed, fma_peak, hbm_gbs)
        roof["traffic"] = NCU_TRAFFIC_BYTES if args.workload == "c2" else None
        roof["peak_source"] = ("measured in this run: packed fma.rn.f32x2 loop on all SMs, "
                               f"{fma_peak / (N_SM * LANES_PER_SM) / 1e6:.0f} MHz-equivalent per lane")
        roof["peak_clocks"] = peak_clocks
        roof["hbm_peak_gbs"] = hbm_gbs
        roof["hbm_peak_source"] = hbm_src
        out = {
            "metric": METRIC, "value": value, "unit": "elements/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": base_config(wl, n_total), "device_status": status,
            "clocks": clocks,
            "e2e": {"value": whole_job_value(n_total, world, ms_e2e, args.steps), "unit": "elements/s",
                    "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h},
            "gpu_launches": wl.launches_timed,
            "roofline": roof,
        }
        if sustained is not None:
            out["sustained"] = sustained
        if per_config is not None:
            out["per_config"] = per_config
        if world == 1 and not args.no_cpu_baseline:
            v, cores, desc, _ = wl.cpu()
            out["cpu_baseline"] = {"value": v, "unit": "elements/s", "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true",
                    help="only the timed region of the selected workload: no seconds-long loop, no per_config block")
    ap.add_argument("--workload", default="c2",
                    help="c2 (default: the ResNet-50 weight set the metric is quoted on), c1, c1x64, c3, c4, c5:K:bits, dual")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
