#!/usr/bin/env python
"""Throughput of the MMSE quantization search on the ResNet-50-shaped weight set.

One step = the whole hot path over one batch of synthetic input: every one of the 54 weight
tensors goes through omse_quantize_weights_batched (stage, max, 1024-candidate sweep, argmin,
3 polish steps, codes, INT4 packing; one launch for the set).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

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
INSTR_PER_EVAL = 6            # reference FP32 sequence per (element, candidate): 3 fma + 2 min/max + 1 add
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the timed kernel, from the ncu capture summarised
# in profiles/rows_kernel_resnet50_weight_set.md; set to None whenever the kernel changes after the capture
NCU_TRAFFIC_BYTES = None
N_SM, LANES_PER_SM = 148, 128
WORKLOAD = "resnet50_weight_set_54_tensors_25.5M_params_signed4bit_kernelwise_1024cand_3refine_packed"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d.get("sm_max_mhz", 1965.0), "measured"
    return 1965.0, "fallback"


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


def _cpu_sample(weights):
    """Every fourth kernel of every tensor: the bounded sample the oracle is timed on."""
    return [np.ascontiguousarray(w[::4]) for _, w in weights]


def _time_oracle(sample):
    from oracle import omse_oracle as orc
    orc.build()
    t0 = time.perf_counter()
    for w in sample:
        r = orc.quantize_rows(w, BITS, True, N_CAND, HI_FRAC, REFINE)
        orc.pack_int4(r.codes)
    dt = time.perf_counter() - t0
    n = sum(w.size for w in sample)
    return n / dt, dt, n, orc.max_threads()


def run_reference(args, rank):
    """The oracle, as it stands, on the host cores; each step is the bounded sample."""
    if rank != 0:
        return
    from paper_1902_06822_b200 import synth
    sample = _cpu_sample(synth.resnet50_weights(seed=2))
    for _ in range(min(args.warmup, 1)):
        _time_oracle(sample[:4])
    total_t, n = 0.0, 0
    for _ in range(args.steps):
        _, dt, n, cores = _time_oracle(sample)
        total_t += dt
    value = n * args.steps / total_t
    desc = f"every 4th kernel of each of the 54 tensors ({n} elements per step)"
    print(json.dumps({
        "impl": "reference", "metric": "elements quantized/sec (4-bit MMSE search)", "value": value,
        "unit": "elements/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args, rank, world):
    import torch
    from paper_1902_06822_b200 import binding, build, synth
    build.build()
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    weights = synth.resnet50_weights(seed=rank_seed(rank))
    n_total = sum(w.size for _, w in weights)
    ctx = binding.Context(local)
    stream = torch.cuda.current_stream(dev)

    host_in = [torch.from_numpy(w).pin_memory() for _, w in weights]
    d_w = [h.to(dev) for h in host_in]
    outs = []
    for _, w in weights:
        s, k = w.shape
        outs.append((torch.empty(s, dtype=torch.float32, device=dev), torch.empty(s, dtype=torch.float32, device=dev),
                     torch.empty((s * k + 1) // 2, dtype=torch.uint8, device=dev)))
    host_out = [(a.cpu().pin_memory(), e.cpu().pin_memory(), p.cpu().pin_memory()) for a, e, p in outs]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2

    descs = [dict(w=dw, n_kernels=w.shape[0], kernel_len=w.shape[1], alpha=a, sse=e, packed=p)
             for (name, w), dw, (a, e, p) in zip(weights, d_w, outs)]

    def step():
        # all 54 tensors in one launch: kernels of every layer are handed out longest first
        ctx.omse_quantize_weights_batched(descs, BITS, True, N_CAND, HI_FRAC, REFINE)

    def step_e2e():
        for hin, dw in zip(host_in, d_w):
            dw.copy_(hin, non_blocking=True)
        ctx.omse_quantize_weights_batched(descs, BITS, True, N_CAND, HI_FRAC, REFINE)
        for (a, e, p), (ha, he, hp) in zip(outs, host_out):
            ha.copy_(a, non_blocking=True)
            he.copy_(e, non_blocking=True)
            hp.copy_(p, non_blocking=True)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for s0, s1 in ev:
            flush.fill_(1)          # evict the inputs from L2 between timed steps (not timed)
            s0.record(stream)
            fn()
            s1.record(stream)
        barrier()
        return max_over_ranks(sum(s0.elapsed_time(s1) for s0, s1 in ev), dist, dev)

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    ms = timed(step, args.steps)
    clocks = sampler.stop() if sampler else None
    step_e2e()
    ms_e2e = timed(step_e2e, args.steps)
    status = ctx.omse_last_device_status()

    if rank == 0:
        sm_max_mhz, peak_src = _peaks()
        per_step_s = ms * 1e-3 / args.steps
        value = whole_job_value(n_total, world, ms, args.steps)
        peak = N_SM * LANES_PER_SM * sm_max_mhz * 1e6                     # FP32 lane-instructions per second
        achieved = INSTR_PER_EVAL * N_CAND * n_total / per_step_s          # algorithmic instructions per second
        h2d = sum(h.numel() * 4 for h in host_in)
        d2h = sum(a.numel() * 4 + e.numel() * 4 + p.numel() for a, e, p in outs)
        out = {
            "metric": "elements quantized/sec (4-bit MMSE search)", "value": value, "unit": "elements/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "elements_per_gpu": n_total, "n_cand": N_CAND, "bits": BITS,
                       "refine_iters": REFINE, "l2": "flushed between timed steps (256 MB write)",
                       "device_status": status},
            "clocks": clocks,
            "e2e": {"value": whole_job_value(n_total, world, ms_e2e, args.steps), "unit": "elements/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": args.steps,
            "roofline": {"bound": "alu", "achieved": achieved / 1e12, "peak": peak / 1e12,
                         "unit": "T FP32-instr/s", "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES,
                         "kernel": "rows_kernel<8>", "peak_source": f"148 SMs x 128 lanes x {sm_max_mhz:.0f} MHz ({peak_src} max clock)",
                         "instr_per_eval": INSTR_PER_EVAL},
        }
        if world == 1 and not args.no_cpu_baseline:
            v, dt, n, cores = _time_oracle(_cpu_sample(weights))
            out["cpu_baseline"] = {"value": v, "unit": "elements/s", "cores": cores, "kind": "oracle",
                                   "sample": f"every 4th kernel of each of the 54 tensors ({n} elements, {dt:.1f} s)"}
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
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
