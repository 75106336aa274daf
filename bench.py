#!/usr/bin/env python
"""Throughput of the M2RNN scan library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the scan over one batch of synthetic input of the named workload
(default: the bf16 forward configuration B=8, N=16, K=V=64, T=2048).  Prints ONE JSON line:
tokens/s with inputs resident in HBM (`value`), the same through host buffers (`e2e`), the
achieved fraction of the tensor-core roofline for the scan kernel (`roofline`), the CPU oracle
timed on this host (`cpu_baseline`) and the GPU clocks seen while timing.

With N > 1 (torchrun) every rank scans its own batch of the same shape (units are independent:
no collective on the data path); the value is all ranks' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_14360_b200 import inputs  # noqa: E402
from paper_2603_14360_b200.inputs import CONFIGS  # noqa: E402

METRIC = "m2rnn_scan_tokens_per_s"
ROTATE = 4  # input sets cycled through so that no step finds its inputs in L2


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:  # NVML missing: clocks are reported as unknown
            self.nv = None

    def _once(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        for k, bit in names.items():
            if r & bit:
                self.reasons.add(k)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                return
            time.sleep(self.period)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()
            try:
                self._once()
            except Exception:
                pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def oracle_sample_rate(cfg, seconds_target=12.0):
    """Times the fp64 oracle (one thread) on whole (b,n) units of the workload and scales by the
    exact ratio of units (they are independent).  Returns (tokens/s, description, seconds)."""
    import oracle
    oracle.build()
    d = inputs.make_inputs(cfg.with_(B=1, N=min(cfg.N, 2), Nq=0, Nk=0))
    f = inputs.to_f64
    args = [f(d[x]) for x in ("q", "k", "v", "gate", "W", "h0")]
    t0 = time.perf_counter()
    oracle.fwd(*[a[:, :64] if i < 4 else a for i, a in enumerate(args)])
    per_unit_step = (time.perf_counter() - t0) / (64 * args[2].shape[2])
    # whole units, full T, as many as fit the budget
    units = max(1, min(args[2].shape[2], int(seconds_target / (per_unit_step * cfg.T))))
    sub = [a[:, :, :units] if i < 4 else (a[:units] if i == 4 else (None if a is None else a[:, :units]))
           for i, a in enumerate(args)]
    t0 = time.perf_counter()
    oracle.fwd(*sub)
    dt = time.perf_counter() - t0
    full_time = dt * (cfg.B * cfg.N) / units
    return cfg.tokens / full_time, f"{units} of {cfg.B * cfg.N} (b,n) units x T={cfg.T}, fp64, 1 thread, scaled by unit count", dt


def run_reference(args, cfg):
    """The reference arm: the CPU oracle as it stands, on this host's cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rates, dts = [], []
    for i in range(args.warmup + args.steps):
        r, desc, dt = oracle_sample_rate(cfg, seconds_target=4.0)
        if i >= args.warmup:
            rates.append(r); dts.append(dt)
    value = sum(rates) / len(rates)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cfg.tokens / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "T": cfg.T, "N": cfg.N, "K": cfg.K, "V": cfg.V,
                       "pass": "fwd"},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="fwd_bf16", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    cfg = CONFIGS[args.workload]
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        args.steps, args.warmup = min(args.steps, 5), min(args.warmup, 1)
        run_reference(args, cfg)
        return

    from paper_2603_14360_b200 import binding
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the scan has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ROTATE seeded input sets per rank, resident in HBM; the same sets pinned on the host for e2e
    host_sets = []
    for r in range(ROTATE):
        d = inputs.make_inputs(cfg, seed=cfg.seed + 1000 * rank + 17 * r)
        host_sets.append({k: (v.pin_memory() if isinstance(v, torch.Tensor) else v) for k, v in d.items()})
    dev_sets = [{k: (v.to(dev) if isinstance(v, torch.Tensor) else v) for k, v in hs.items()} for hs in host_sets]
    W = dev_sets[0]["W"]
    io = inputs.torch_dtype(cfg.dtype)
    outs = [dict(y=torch.empty((cfg.B, cfg.T, cfg.N, cfg.V), dtype=io, device=dev),
                 hT=torch.empty((cfg.B, cfg.N, cfg.K, cfg.V), dtype=torch.float32, device=dev)) for _ in range(ROTATE)]
    stream = torch.cuda.current_stream()

    def step(i):
        s = dev_sets[i % ROTATE]
        binding.m2rnn_fwd(s["q"], s["k"], s["v"], s["gate"], W, s["h0"], gate_kind=cfg.gate_kind,
                          out=outs[i % ROTATE], stream=stream)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    binding.check_device_status()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    with ClockSampler(local) as clocks:
        barrier()
        ev[0].record(stream)
        for i in range(args.steps):
            step(i)
        ev[1].record(stream)
        barrier()
    ms_total = ev[0].elapsed_time(ev[1])
    binding.check_device_status()

    # end to end: host buffers in, host buffers out, every step
    host_out = dict(y=torch.empty((cfg.B, cfg.T, cfg.N, cfg.V), dtype=io).pin_memory(),
                    hT=torch.empty((cfg.B, cfg.N, cfg.K, cfg.V), dtype=torch.float32).pin_memory())
    stage = {k: torch.empty_like(v) for k, v in dev_sets[0].items() if isinstance(v, torch.Tensor) and k != "W"}
    h2d = sum(t.numel() * t.element_size() for t in stage.values())
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())

    def e2e_step(i):
        hs = host_sets[i % ROTATE]
        for k, t in stage.items():
            t.copy_(hs[k], non_blocking=True)
        binding.m2rnn_fwd(stage["q"], stage["k"], stage["v"], stage["gate"], W, stage.get("h0"),
                          gate_kind=cfg.gate_kind, out=outs[0], stream=stream)
        host_out["y"].copy_(outs[0]["y"], non_blocking=True)
        host_out["hT"].copy_(outs[0]["hT"], non_blocking=True)

    e2e_steps = max(3, min(args.steps, 50))
    for i in range(3):
        e2e_step(i)
    barrier()
    ev2 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev2[0].record(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    ev2[1].record(stream)
    barrier()
    ms_e2e = ev2[0].elapsed_time(ev2[1])

    times = torch.tensor([ms_total, ms_e2e], dtype=torch.float64, device=dev)
    if dist:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms_total, ms_e2e = (float(x) for x in times.tolist())
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    ms_step = ms_total / args.steps
    tokens = cfg.tokens * world
    value = tokens / (ms_step * 1e-3)
    peaks = measured_peaks()
    th = cfg.B * cfg.T * cfg.N                                   # token-heads per launch
    flops = 2.0 * cfg.K * cfg.V * cfg.V * th                     # the state x W contraction
    esz = 2 if cfg.dtype == "bf16" else 4
    bt = cfg.B * cfg.T
    stream_bytes = (bt * (cfg.nq + cfg.nk) * cfg.K * esz + 2 * th * cfg.V * esz + th * 4      # q,k | v,y | gate
                    + 2 * cfg.B * cfg.N * cfg.K * cfg.V * 4)                                   # h0 in, hT out
    t_tensor = flops / (peaks["tflops_burst"] * 1e12)
    t_hbm = stream_bytes / (peaks["hbm_gbs"] * 1e9)
    achieved = flops / (ms_step * 1e-3) / 1e12
    sm_clock = 1.965e9
    mufu_s = th * cfg.K * cfg.V / (16 * 148 * sm_clock)          # one tanh per state element per step
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "pass": "fwd", "B": cfg.B, "T": cfg.T, "N": cfg.N, "K": cfg.K, "V": cfg.V,
                   "Nq": cfg.nq, "Nk": cfg.nk, "gate": "logit", "state": "fp32", "accumulate": "fp32",
                   "per_gpu_batch": cfg.B,
                   "l2": f"{ROTATE} input/output sets cycled ({ROTATE} x {int((h2d + d2h) / 1e6)} MB > 126 MB L2)"},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peaks["tflops_burst"], "unit": "TFLOP/s",
                     "frac": achieved / peaks["tflops_burst"], "traffic": None,
                     "peak_source": f"{peaks['source']} cuBLAS bf16 burst",
                     "t_tensor_ms": t_tensor * 1e3, "t_hbm_ms": t_hbm * 1e3,
                     "t_mufu_ms": mufu_s * 1e3, "frac_of_mufu_ceiling": mufu_s / (ms_step * 1e-3),
                     "ns_per_scan_step": ms_step * 1e6 / cfg.T},
        "e2e": {"value": tokens / (ms_e2e / e2e_steps * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": args.steps,
        "clocks": clocks.summary(),
    }
    if not args.no_cpu_baseline:
        rate, desc, dt = oracle_sample_rate(cfg)
        line["cpu_baseline"] = {"value": rate, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": desc,
                                "seconds": dt}
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
