#!/usr/bin/env python
"""Throughput of the M2RNN scan library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the scan over one batch of synthetic input of the named workload:
a forward scan (`fwd_bf16`, the default: B=8, N=16, K=V=64, T=2048; also `long_ctx`,
`paper_layer`, `tiny_f32`), a forward + backward scan (`bptt_bf16`, `sweep16..128`), one decoding
step (`decode`), or the output path after the scan (`out_norm`: gated RMSNorm forward + backward on
fwd_bf16's y).  `--multi-value` runs a scan workload in the paper's shared q/k head layout.
Prints ONE JSON line: tokens/s with inputs resident in HBM (`value`), the same
through host buffers (`e2e`: copy-in, step and copy-out as a three-stream pipeline), the achieved fraction of the roofline of the dominant call
(`roofline`), the CPU oracle timed on this host (`cpu_baseline`) and the GPU clocks seen while
timing.

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
PASS_OF = {"fwd_bf16": "fwd", "long_ctx": "fwd", "paper_layer": "fwd", "tiny_f32": "fwd", "decode": "decode"}   # others: fwd+bwd
SM_COUNT, SM_HZ = 148, 1.965e9
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic.txt")
CSRC = os.path.join(ROOT, "paper_2603_14360_b200", "csrc")


def kernel_source_digest(cu_file: str) -> str:
    """Digest of a kernel's translation unit and the headers of its directory: the table's rows are
    valid for the sources they were captured from, not after a change."""
    import hashlib
    h = hashlib.sha256()
    names = [cu_file] + sorted(f for f in os.listdir(CSRC) if f.endswith((".cuh", ".h")))
    for f in names:
        h.update(open(os.path.join(CSRC, f), "rb").read())
    return h.hexdigest()[:16]


def profiled_traffic(workload: str, units: int):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the workload's
    dominant kernel, from the table that `python -m paper_2603_14360_b200.ncu_traffic` writes out of
    an ncu capture.  A row captured at another sequence length is scaled by the token-heads of a
    full launch (traffic is per token-head).  None when there is no row, or when the kernel's
    sources have changed since the capture."""
    if not os.path.exists(TRAFFIC_TABLE):
        return None
    for ln in open(TRAFFIC_TABLE):
        f = ln.split()
        if len(f) < 6 or f[0].startswith("#") or f[0] != workload:
            continue
        _, kernel, cu_file, bytes_per_launch, units_captured, digest = f[:6]
        if digest != kernel_source_digest(cu_file):
            return None
        scale = units / float(units_captured)
        return {"bytes": float(bytes_per_launch) * scale,
                "source": f"profiles/dram_traffic.txt: {kernel}, captured on {units_captured} token-heads"
                          + ("" if scale == 1 else f", scaled x{scale:g}")}
    return None


def profiled_traffic_sum(workload: str, parts, units: int):
    """The same for a step made of several kernels: rows `workload:part`, added; None if one is
    missing or stale."""
    rows = [profiled_traffic(f"{workload}:{p}", units) for p in parts]
    if any(r is None for r in rows):
        return None
    return {"bytes": sum(r["bytes"] for r in rows), "source": "; ".join(r["source"] for r in rows)}


def workload_pass(name: str) -> str:
    return PASS_OF.get(name, "fwd+bwd")


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


# ------------------------------------------------------------------------------ CPU oracle leg
def oracle_sample_rate(cfg, pas, seconds_target=12.0):
    """Times the fp64 oracle (one thread) on whole (b,n) units of the workload and scales by the
    exact ratio of units (they are independent).  Returns (tokens/s, description, seconds)."""
    import oracle
    oracle.build()
    f = inputs.to_f64
    nmax, bmax = min(cfg.N, 16), min(cfg.B, 4)
    small = cfg.with_(B=bmax, N=nmax, Nq=0, Nk=0)
    if pas == "decode":
        d = inputs.make_inputs(small.with_(T=1))
        args = [f(d[x][:, 0]) for x in ("q", "k", "v", "gate")] + [f(d["W"]), f(d["h0"])]
        oracle.decode_step(*args)
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < seconds_target:
            oracle.decode_step(*args)
            reps += 1
        dt = time.perf_counter() - t0
        per_unit = dt / (reps * bmax * nmax)
        full = per_unit * cfg.B * cfg.N
        return cfg.B / full, (f"{reps} decode steps of {bmax * nmax} of {cfg.B * cfg.N} (b,n) units, fp64, 1 thread, "
                              "scaled by unit count"), dt
    d = inputs.make_inputs(small, backward=(pas == "fwd+bwd"))
    names = ("q", "k", "v", "gate", "W", "h0") + (("dy",) if pas == "fwd+bwd" else ())
    args = {x: f(d[x]) for x in names}

    def run(sub):
        oracle.fwd(sub["q"], sub["k"], sub["v"], sub["gate"], sub["W"], sub["h0"])
        if pas == "fwd+bwd":
            oracle.bwd(sub["q"], sub["k"], sub["v"], sub["gate"], sub["W"], sub["h0"], sub["dy"])

    def cut(nb, nn, T):
        out = {}
        for x, a in args.items():
            if x == "W":
                out[x] = a[:nn]
            elif x == "h0":
                out[x] = None if a is None else a[:nb, :nn]
            else:
                out[x] = a[:nb, :T, :nn]
        return out

    probe_T = min(cfg.T, 64)
    t0 = time.perf_counter()
    run(cut(1, min(nmax, 2), probe_T))
    per_unit_step = (time.perf_counter() - t0) / (probe_T * min(nmax, 2))
    # whole units where a unit fits the budget, else one unit over a prefix of the sequence
    T_use = cfg.T
    budget_units = seconds_target / (per_unit_step * cfg.T)
    if budget_units < 1:
        nb, nn = 1, 1
        T_use = max(probe_T, int(seconds_target / per_unit_step))
    elif budget_units < nmax:
        nb, nn = 1, max(1, int(budget_units))
    else:
        nn = nmax
        nb = max(1, min(bmax, int(budget_units / nmax)))
    t0 = time.perf_counter()
    run(cut(nb, nn, T_use))
    dt = time.perf_counter() - t0
    units = nb * nn
    full_time = dt * (cfg.B * cfg.N) / units * (cfg.T / T_use)
    what = f"{units} of {cfg.B * cfg.N} (b,n) units x T={T_use}" + ("" if T_use == cfg.T else f" of {cfg.T}")
    return cfg.tokens / full_time, f"{what}, {pas}, fp64, 1 thread, scaled by unit (and step) count", dt


def oracle_all_cores_rate(cfg, pas, seconds_target=10.0):
    """The fp32 build of the oracle's loops on every core of this host: whole (b,n) units of the
    workload handed to a thread pool (units are independent; the C loops run outside the
    interpreter lock), scaled by the exact ratio of units (and of steps, when one unit alone
    exceeds the budget).  Returns (tokens/s, cores, description, seconds)."""
    import concurrent.futures
    import oracle
    oracle.build_f32()
    cores = os.cpu_count() or 1
    bwd = pas == "fwd+bwd"
    nb, nn = min(cfg.B, 4), min(cfg.N, max(1, 64 // min(cfg.B, 4)))
    small = cfg.with_(B=nb, N=nn, Nq=0, Nk=0)
    d = inputs.make_inputs(small, backward=bwd)
    names = ("q", "k", "v", "gate", "W", "h0") + (("dy",) if bwd else ())
    f32 = {x: (None if d[x] is None else d[x].float().numpy()) for x in names}

    def unit_args(b, n, T):
        out = [f32[x][b:b + 1, :T, n:n + 1] for x in ("q", "k", "v", "gate")]
        out += [f32["W"][n:n + 1], None if f32["h0"] is None else f32["h0"][b:b + 1, n:n + 1]]
        return out + ([f32["dy"][b:b + 1, :T, n:n + 1]] if bwd else [])

    def run(a):
        oracle.fwd_f32(*a[:6])
        if bwd:
            oracle.bwd_f32(*a)

    probe_T = min(cfg.T, 64)
    t0 = time.perf_counter()
    run(unit_args(0, 0, probe_T))
    per_step = (time.perf_counter() - t0) / probe_T
    T_use = cfg.T if per_step * cfg.T <= seconds_target else max(probe_T, int(seconds_target / per_step))
    rounds = max(1, int(seconds_target / (per_step * T_use)))
    units = [(u // nn % nb, u % nn) for u in range(min(nb * nn, cores * rounds))]
    work = [unit_args(b, n, T_use) for (b, n) in units]
    t0 = time.perf_counter()
    with concurrent.futures.ThreadPoolExecutor(max_workers=cores) as ex:
        list(ex.map(run, work))
    dt = time.perf_counter() - t0
    full_time = dt * (cfg.B * cfg.N) / len(units) * (cfg.T / T_use)
    what = f"{len(units)} of {cfg.B * cfg.N} (b,n) units x T={T_use}" + ("" if T_use == cfg.T else f" of {cfg.T}")
    return cfg.tokens / full_time, min(cores, len(units)), f"{what}, {pas}, fp32 build of the same loops, one unit per thread, scaled by unit (and step) count", dt


def run_reference(args, cfg, pas):
    """The reference arm: the CPU oracle as it stands, on this host's cores."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    rates = []
    desc = ""
    for i in range(args.warmup + args.steps):
        r, desc, _ = oracle_sample_rate(cfg, pas, seconds_target=4.0)
        if i >= args.warmup:
            rates.append(r)
    value = sum(rates) / len(rates)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cfg.tokens / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "T": cfg.T, "N": cfg.N, "K": cfg.K, "V": cfg.V, "pass": pas},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ multi-rank plumbing
# The scan has no exchange step: with N ranks every rank scans its own batch (replicas), and the
# only communication is the barrier around the timed region and the max of the ranks' timings.
def rank_input_seed(base_seed: int, rank: int, rotation: int) -> int:
    """Seed of input set `rotation` on `rank`: distinct per rank so the replicas do not share data."""
    return base_seed + 1000 * rank + 17 * rotation


def max_over_ranks(values, dist, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_step: float) -> float:
    """All ranks' tokens over the slowest rank's time per step."""
    return tokens_per_rank * world / (ms_step * 1e-3)


# ------------------------------------------------------------------------------ GPU leg
def nbytes(t):
    return 0 if t is None else t.numel() * t.element_size()


def e2e_pipeline(stream, dev, n, copy_in, compute, copy_out):
    """n steps as a three-stream pipeline with two device buffers each way: copy_in(i, b) brings the
    inputs of step i into buffer b on a copy stream, compute(i, b) runs the step on `stream`,
    copy_out(b) takes the results of buffer b back on a third stream.  Returns (start, stop) events on
    `stream`; the first copy-in and the last copy-out are not overlapped and lie between them."""
    copy_stream = torch.cuda.Stream(device=dev)
    back_stream = torch.cuda.Stream(device=dev)
    landed = [torch.cuda.Event() for _ in range(2)]        # the buffer's inputs are on the device
    consumed = [torch.cuda.Event() for _ in range(2)]      # the step that read the buffer is done
    computed = [torch.cuda.Event() for _ in range(2)]      # the step's results are in their buffers
    copied_back = [torch.cuda.Event() for _ in range(2)]   # ... and have left them

    def issue_h2d(i):
        b = i % 2
        with torch.cuda.stream(copy_stream):
            if i >= 2:
                copy_stream.wait_event(consumed[b])
            copy_in(i, b)
            landed[b].record(copy_stream)

    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    start.record(stream)
    copy_stream.wait_event(start)
    issue_h2d(0)
    for i in range(n):
        b = i % 2
        if i + 1 < n:
            issue_h2d(i + 1)
        stream.wait_event(landed[b])
        if i >= 2:
            stream.wait_event(copied_back[b])
        compute(i, b)
        consumed[b].record(stream)
        computed[b].record(stream)
        with torch.cuda.stream(back_stream):
            back_stream.wait_event(computed[b])
            copy_out(b)
            copied_back[b].record(back_stream)
    stream.wait_stream(back_stream)
    stop.record(stream)
    return start, stop


def main_out_norm(args):
    """`--workload out_norm`: the output path after the scan (y (.) SiLU(g) -> RMSNorm over the
    concatenated heads), forward + backward, on the y of the fwd_bf16 workload (B=8, T=2048, N=16,
    V=64, bf16).  HBM-bound: 6d+4 bytes per token forward, 10d+4 backward (d = N V)."""
    from paper_2603_14360_b200 import binding
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist_.init_process_group("nccl", device_id=dev)
        dist = dist_
    base = CONFIGS["fwd_bf16"]
    B, T, N, V = base.B, base.T, base.N, base.V
    d = N * V
    tokens = B * T
    args.steps = args.steps or 200
    args.warmup = max(args.warmup or 10, 3)
    R = 8                                              # 8 x 168 MB of inputs and outputs cycled: far above L2
    host = [{k: v.pin_memory() for k, v in inputs.make_gated_norm_inputs(B, T, N, V, "bf16",
                                                                         seed=rank_input_seed(7, rank, r)).items()}
            for r in range(R)]
    sets = [{k: v.to(dev) for k, v in h.items()} for h in host]
    outs = [dict(out=torch.empty_like(s["y"]), rstd=torch.empty((B, T), dtype=torch.float32, device=dev),
                 dy=torch.empty_like(s["y"]), dg=torch.empty_like(s["y"]),
                 dw=torch.empty((d,), dtype=torch.float32, device=dev)) for s in sets[:2]]
    ws = torch.empty(max(1, binding.m2rnn_gated_norm_bwd_workspace_bytes(tokens, d)), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def launch(s, o, st):
        binding.m2rnn_gated_norm_fwd(s["y"], s["g_in"], s["w"], eps=1e-6, out=o["out"], rstd=o["rstd"], stream=st)
        binding.m2rnn_gated_norm_bwd(s["y"], s["g_in"], s["w"], o["rstd"], s["dout"], workspace=ws, out=o, stream=st)

    # the three launches of a step are short (tens of microseconds): one CUDA graph per input set
    # replays them without the per-launch host work
    for s_ in sets:
        launch(s_, outs[0], stream)
    torch.cuda.synchronize()
    graphs = []
    for s_ in sets:
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            launch(s_, outs[0], torch.cuda.current_stream())
        graphs.append(gr)

    def step(i, s=None, ob=0):
        if s is None:
            graphs[i % R].replay()
        else:
            launch(s, outs[ob], stream)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    with ClockSampler(local) as clocks:
        barrier()
        ev[0].record(stream)
        for i in range(args.steps):
            step(i)
        ev[1].record(stream)
        barrier()
    ms_total = ev[0].elapsed_time(ev[1])
    # end to end: y, g, dout in from pinned host memory, out, dy, dg, dw back, every step, as the
    # same three-stream pipeline as the scan workloads
    ms_e2e, e2e_steps, h2d, d2h = 0.0, 0, 0, 0
    if not args.no_e2e:
        stages = [{k: torch.empty_like(v) for k, v in sets[0].items()} for _ in range(2)]
        hout = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in outs[0].items() if k != "rstd"}
        h2d = sum(nbytes(t) for t in stages[0].values())
        d2h = sum(nbytes(t) for t in hout.values())
        e2e_steps = 20

        def copy_in(i, b):
            for k, t in stages[b].items():
                t.copy_(host[i % R][k], non_blocking=True)

        def compute(i, b):
            step(i, s=stages[b], ob=b)

        def copy_out(b):
            for k, t in hout.items():
                t.copy_(outs[b][k], non_blocking=True)

        e2e_pipeline(stream, dev, 3, copy_in, compute, copy_out)
        barrier()
        ev2 = e2e_pipeline(stream, dev, e2e_steps, copy_in, compute, copy_out)
        barrier()
        ms_e2e = ev2[0].elapsed_time(ev2[1])
    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dist, dev)
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    ms_step = ms_total / args.steps
    peaks = measured_peaks()
    alg_bytes = tokens * ((6 * d + 4) + (10 * d + 4)) + 2 * d * 2 + d * 4
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    traffic = profiled_traffic_sum("out_norm", ("fwd", "bwd"), tokens)
    line = {
        "metric": METRIC, "value": whole_job_tokens_per_s(tokens, world, ms_step), "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "out_norm", "pass": "fwd+bwd of RMSNorm(y * SiLU(g))", "B": B, "T": T, "N": N, "V": V, "d": d,
                   "per_gpu_batch": B, "l2": f"{R} input sets cycled; bytes touched per step {int(alg_bytes / 1e6)} MB vs 126 MB L2"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"],
                     # dram bytes of the two kernels of a step (part of the results is still in L2 when a
                     # kernel ends, so this is below the algorithmic bytes)
                     "traffic": traffic and traffic["bytes"], "traffic_source": traffic and traffic["source"],
                     "call": "m2rnn_gated_norm_fwd + m2rnn_gated_norm_bwd",
                     "peak_source": f"{peaks['source']} HBM copy", "algorithmic_bytes_per_step": alg_bytes},
        "gpu_launches": args.steps * 3,
        "clocks": clocks.summary(),
    }
    if not args.no_e2e:
        line["e2e"] = {"value": tokens * world / (ms_e2e / e2e_steps * 1e-3), "unit": "tokens/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    if not args.no_cpu_baseline:
        import oracle
        f = inputs.to_f64
        n_tok = 1024                                    # a bounded sample: the first tokens of the first set
        hs = {k: (v.reshape(tokens, N, V)[:n_tok] if v.dim() == 4 else v) for k, v in host[0].items()}
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            oracle.gated_norm_fwd(f(hs["y"]), f(hs["g_in"]), f(hs["w"]), eps=1e-6)
            oracle.gated_norm_bwd(f(hs["y"]), f(hs["g_in"]), f(hs["w"]), f(hs["dout"]), eps=1e-6)
            reps += 1
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": reps * n_tok / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                                "sample": f"{reps} x the first {n_tok} tokens of one input set, forward + backward", "seconds": dt}
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def main_in_conv(args):
    """`--workload in_conv`: the input path before the scan (SiLU of a depthwise causal conv1d of width
    4), forward + backward, on the fused q/k/v projection of the fwd_bf16 workload (B=8, T=2048,
    C = Nq K + Nk K + N V = 3072, bf16).  HBM-bound: 4C bytes per token forward (x in, out), 6C backward
    (x, dout in, dx out)."""
    from paper_2603_14360_b200 import binding
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist_.init_process_group("nccl", device_id=dev)
        dist = dist_
    base = CONFIGS["fwd_bf16"]
    B, T = base.B, base.T
    C = (base.nq + base.nk) * base.K + base.N * base.V
    tokens = B * T
    steps = args.steps or 200
    warmup = max(args.warmup or 10, 3)
    R = 4                                              # 4 x 200 MB of inputs cycled: above L2
    host = [{k: v.pin_memory() for k, v in inputs.make_conv_inputs(B, T, C, "bf16", seed=rank_input_seed(11, rank, r), prev=False).items()
             if v is not None} for r in range(R)]
    sets = [{k: v.to(dev) for k, v in h.items()} for h in host]
    outs = [dict(out=torch.empty_like(sets[0]["x"]), dx=torch.empty_like(sets[0]["x"]),
                 dw=torch.empty((C, 4), dtype=torch.float32, device=dev), dbias=torch.empty((C,), dtype=torch.float32, device=dev))
            for _ in range(2)]
    ws = torch.empty(max(1, binding._lib().m2rnn_conv_silu_bwd_workspace_bytes(B, T, C)), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step(i, s=None, ob=0):
        s = s or sets[i % R]
        o = outs[ob]
        binding.m2rnn_conv_silu_fwd(s["x"], s["w"], s["bias"], out=o["out"], stream=stream)
        binding.m2rnn_conv_silu_bwd(s["x"], s["w"], s["dout"], s["bias"], out=o, workspace=ws, stream=stream)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(warmup):
        step(i)
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    with ClockSampler(local) as clocks:
        barrier()
        ev[0].record(stream)
        for i in range(steps):
            step(i)
        ev[1].record(stream)
        barrier()
    ms_total = ev[0].elapsed_time(ev[1])
    ms_e2e, e2e_steps, h2d, d2h = 0.0, 0, 0, 0
    if not args.no_e2e:
        stages = [{k: torch.empty_like(v) for k, v in sets[0].items()} for _ in range(2)]
        hout = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in outs[0].items()}
        h2d = sum(nbytes(t) for t in stages[0].values())
        d2h = sum(nbytes(t) for t in hout.values())
        e2e_steps = 20

        def copy_in(i, b):
            for k, t in stages[b].items():
                t.copy_(host[i % R][k], non_blocking=True)

        def copy_out(b):
            for k, t in hout.items():
                t.copy_(outs[b][k], non_blocking=True)

        e2e_pipeline(stream, dev, 3, copy_in, lambda i, b: step(i, s=stages[b], ob=b), copy_out)
        barrier()
        ev2 = e2e_pipeline(stream, dev, e2e_steps, copy_in, lambda i, b: step(i, s=stages[b], ob=b), copy_out)
        barrier()
        ms_e2e = ev2[0].elapsed_time(ev2[1])
    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dist, dev)
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    ms_step = ms_total / steps
    peaks = measured_peaks()
    alg_bytes = tokens * C * 2 * (2 + 3)               # x, out | x, dout, dx (bf16)
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    traffic = profiled_traffic_sum("in_conv", ("fwd", "bwd", "reduce"), tokens)
    line = {
        "metric": METRIC, "value": whole_job_tokens_per_s(tokens, world, ms_step), "unit": "tokens/s", "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "in_conv", "pass": "fwd+bwd of SiLU(conv1d) on the fused q/k/v projection", "B": B, "T": T, "C": C,
                   "per_gpu_batch": B, "l2": f"{R} input sets cycled; bytes touched per step {int(alg_bytes / 1e6)} MB vs 126 MB L2"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "traffic": traffic and traffic["bytes"],
                     "traffic_source": traffic and traffic["source"], "call": "m2rnn_conv_silu_fwd + m2rnn_conv_silu_bwd",
                     "peak_source": f"{peaks['source']} HBM copy", "algorithmic_bytes_per_step": alg_bytes},
        "gpu_launches": steps * 3,
        "clocks": clocks.summary(),
    }
    if not args.no_e2e:
        line["e2e"] = {"value": tokens * world / (ms_e2e / e2e_steps * 1e-3), "unit": "tokens/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    if not args.no_cpu_baseline:
        import oracle
        f = inputs.to_f64
        n_t = 64                                        # a bounded sample: the first steps of every batch entry
        hs = {k: (v[:, :n_t] if v.dim() == 3 else v) for k, v in host[0].items()}
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            oracle.conv_silu_fwd(f(hs["x"]), f(hs["w"]), f(hs["bias"]))
            oracle.conv_silu_bwd(f(hs["x"]), f(hs["w"]), f(hs["dout"]), f(hs["bias"]))
            reps += 1
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": reps * B * n_t / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                                "sample": f"{reps} x the first {n_t} steps of the {B} batch entries, forward + backward", "seconds": dt}
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def pick_config(args, workload):
    cfg = CONFIGS["paper_layer" if workload == "paper_layer_bptt" else workload]
    if workload == "paper_layer_bptt":
        cfg = cfg.with_(name="paper_layer_bptt")
    if args.seq_len and workload != "decode":
        cfg = cfg.with_(T=args.seq_len, name=f"{cfg.name}@T={args.seq_len}")
    if args.multi_value:   # the paper's layout: one q and one k head shared by all N value heads
        cfg = cfg.with_(Nq=1, Nk=1, name=f"{cfg.name}+multi_value")
    return cfg, workload_pass(workload)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="0: a default per workload")
    ap.add_argument("--warmup", type=int, default=0)
    ap.add_argument("--workload", default=None, choices=sorted(CONFIGS) + ["paper_layer_bptt", "out_norm", "in_conv"],
                    help="default: fwd_bf16 as the line's value, with bptt_bf16 (forward + backward) as the sub-object 'bptt'")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-bptt", action="store_true", help="default run: leave the forward + backward sub-object out")
    ap.add_argument("--multi-value", action="store_true",
                    help="run the workload in the multi-value layout (Nq = Nk = 1) instead of multi-head")
    ap.add_argument("--seq-len", type=int, default=0,
                    help="shorten (or lengthen) the workload's T, for profiler captures; the line's workload name says so")
    args = ap.parse_args()
    both_halves = args.workload is None and not args.no_bptt and not args.seq_len
    workload = args.workload or "fwd_bf16"
    if workload in ("out_norm", "in_conv") and args.impl == "ours":
        (main_out_norm if workload == "out_norm" else main_in_conv)(args)
        return
    if workload in ("out_norm", "in_conv"):
        raise SystemExit("--impl reference times the scan workloads; the out_norm and in_conv lines carry their own cpu_baseline")
    cfg, pas = pick_config(args, workload)

    if args.impl == "reference":
        args.steps, args.warmup = min(args.steps or 3, 5), min(args.warmup or 1, 1)
        run_reference(args, cfg, pas)
        return
    steps = args.steps or {"fwd_bf16": 300, "decode": 1000, "tiny_f32": 300}.get(workload, 20)
    warmup = max(args.warmup or (20 if pas != "fwd+bwd" else 3), 3)

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
    env = dict(binding=binding, world=world, rank=rank, local=local, dev=dev, dist=dist)

    line = run_scan_workload(args, workload, cfg, pas, steps, warmup, env)
    if both_halves:
        # the other half of the metric: forward + backward through time on the BPTT configuration,
        # measured the same way (its own roofline, end-to-end and CPU legs), fewer steps
        cfg2, pas2 = pick_config(args, "bptt_bf16")
        sub = run_scan_workload(args, "bptt_bf16", cfg2, pas2, max(3, min(steps, 10)), 3, env)
        if line is not None:
            line["bptt"] = {k: sub[k] for k in ("value", "unit", "steps", "warmup", "ms_per_step", "ms_fwd", "ms_bwd", "dtype",
                                                 "config", "roofline", "gpu_launches", "clocks", "e2e", "cpu_baseline") if k in sub}
    if line is not None:
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def run_scan_workload(args, workload, cfg, pas, steps, warmup, env):
    """Times one scan workload; returns the JSON line as a dict on rank 0, None elsewhere."""
    binding, world, rank, local, dev, dist = (env[k] for k in ("binding", "world", "rank", "local", "dev", "dist"))
    bwd = pas == "fwd+bwd"
    io = inputs.torch_dtype(cfg.dtype)
    B, T, N, K, V = cfg.B, cfg.T, cfg.N, cfg.K, cfg.V
    # seeded input sets per rank, resident in HBM; the same sets pinned on the host for e2e (decode: a
    # ring of 8 token sets, so that every step of a short ring still sees fresh per-token inputs)
    ROTATE = 8 if pas == "decode" else globals()["ROTATE"]
    # The decode workload rotates its per-token inputs; its state (2 x 1 GB per step) is far above L2.
    host_sets = []
    for r in range(ROTATE):
        d = inputs.make_inputs(cfg, backward=bwd, seed=rank_input_seed(cfg.seed, rank, r))
        if pas == "decode":
            d = {k: (v[:, 0].contiguous() if k in ("q", "k", "v", "gate") else v) for k, v in d.items()}
        host_sets.append({k: (v.pin_memory() if isinstance(v, torch.Tensor) else v) for k, v in d.items()})
    dev_sets = [{k: (v.to(dev) if isinstance(v, torch.Tensor) else v) for k, v in hs.items()} for hs in host_sets]
    W = dev_sets[0]["W"]
    stream = torch.cuda.current_stream()
    launches_per_step = 1

    if pas == "decode":
        state = dev_sets[0]["h0"].clone()
        y1 = torch.empty((B, N, V), dtype=io, device=dev)
        y_bufs = [y1, torch.empty_like(y1)]

        def step(i, s=None, ob=0):
            s = s or dev_sets[i % ROTATE]
            binding.m2rnn_decode_step(s["q"], s["k"], s["v"], s["gate"], W, state, gate_kind=cfg.gate_kind, y=y_bufs[ob],
                                      stream=stream)
        out_tensors = [y1]
        out_sets = [[y_bufs[0]], [y_bufs[1]]]
    else:
        p = binding._params(dev_sets[0]["q"], dev_sets[0]["k"], dev_sets[0]["v"], W, cfg.gate_kind)
        outs = dict(y=torch.empty((B, T, N, V), dtype=io, device=dev),
                    hT=torch.empty((B, N, K, V), dtype=torch.float32, device=dev))
        out_tensors = list(outs.values())
        fws_bytes = binding.m2rnn_fwd_workspace_bytes(p)
        fws = torch.empty(fws_bytes, dtype=torch.uint8, device=dev) if fws_bytes else None
        launches_per_step = 2 if fws_bytes else 1          # the scan (+ the add of the row slabs' shares of y)
        if bwd:
            C = binding.m2rnn_ckpt_interval(p)
            outs["ckpt"] = torch.empty((B, N, (T + C - 1) // C, K, V), dtype=torch.float32, device=dev)
            s0 = dev_sets[0]
            gouts = dict(dq=torch.empty_like(s0["q"]), dk=torch.empty_like(s0["k"]), dv=torch.empty_like(s0["v"]),
                         dgate=torch.empty_like(s0["gate"]), dW=torch.empty((N, V, V), dtype=torch.float32, device=dev),
                         dh0=torch.empty((B, N, K, V), dtype=torch.float32, device=dev))
            ws = torch.empty(max(1, binding.m2rnn_bwd_workspace_bytes(p, True)), dtype=torch.uint8, device=dev)
            out_tensors += list(gouts.values())
            # fwd, bwd, dW reduce (+ dv and dgate reduces when a state's rows are split over CTAs)
            launches_per_step += 2 + (2 if binding.m2rnn_bwd_row_slab(p) != K else 0)
        ev_mid = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        # a second set of result buffers for the end-to-end leg (results of step i leave the device
        # while step i+1 computes); the checkpoints never leave and are shared
        outs_b = [outs, {k: (v if k == "ckpt" else torch.empty_like(v)) for k, v in outs.items()}]
        gouts_b = [gouts, {k: torch.empty_like(v) for k, v in gouts.items()}] if bwd else [None, None]
        out_sets = [[t for k, t in outs_b[j].items() if k != "ckpt"] + (list(gouts_b[j].values()) if bwd else [])
                    for j in range(2)]

        def step(i, s=None, mark=False, ob=0):
            s = s or dev_sets[i % ROTATE]
            binding.m2rnn_fwd(s["q"], s["k"], s["v"], s["gate"], W, s["h0"], gate_kind=cfg.gate_kind,
                              save_ckpt=bwd, out=outs_b[ob], workspace=fws, stream=stream)
            if bwd:
                if mark:
                    ev_mid[0].record(stream)
                binding.m2rnn_bwd(s["q"], s["k"], s["v"], s["gate"], W, s["h0"], s["dy"], ckpt=outs["ckpt"],
                                  gate_kind=cfg.gate_kind, workspace=ws, out=gouts_b[ob], stream=stream)
                if mark:
                    ev_mid[1].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(warmup):
        step(i)
    barrier()
    binding.check_device_status()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    with ClockSampler(local) as clocks:
        barrier()
        ev[0].record(stream)
        for i in range(steps):
            step(i)
        ev[1].record(stream)
        barrier()
    ms_total = ev[0].elapsed_time(ev[1])
    binding.check_device_status()
    # the backward call alone (its kernels only), for the roofline of the dominant call
    ms_bwd = 0.0
    if bwd:
        reps = min(steps, 10)
        for i in range(reps):
            step(i, mark=True)
            torch.cuda.synchronize()
            ms_bwd += ev_mid[0].elapsed_time(ev_mid[1]) / reps

    # end to end: host buffers in, host buffers out, every step
    ms_e2e, e2e_steps, h2d, d2h = 0.0, 0, 0, 0
    if not args.no_e2e:
        host_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in out_sets[0]]
        # Two device-side input buffers: the copy of step i+1's inputs runs on a stream of its own
        # while step i computes and its results go back (as an input pipeline of a training or
        # serving loop would); every timed step still moves its own inputs in and its results out.
        stages = [{k: torch.empty_like(v) for k, v in dev_sets[0].items()
                   if isinstance(v, torch.Tensor) and k != "W" and not (pas == "decode" and k == "h0")} for _ in range(2)]
        h2d = sum(nbytes(t) for t in stages[0].values())
        d2h = sum(nbytes(t) for t in host_out)

        def copy_in(i, b):
            hs = host_sets[i % ROTATE]
            for k, t in stages[b].items():
                t.copy_(hs[k], non_blocking=True)

        def compute(i, b):
            step(i, s={**stages[b], "W": W, "h0": stages[b].get("h0", dev_sets[0].get("h0"))}, ob=b)

        def copy_out(b):
            for h, d_ in zip(host_out, out_sets[b]):
                h.copy_(d_, non_blocking=True)

        def e2e_run(n):
            return e2e_pipeline(stream, dev, n, copy_in, compute, copy_out)

        e2e_steps = max(3, min(steps, 50))
        e2e_run(3)
        barrier()
        ev2 = e2e_run(e2e_steps)
        barrier()
        ms_e2e = ev2[0].elapsed_time(ev2[1])

    ms_total, ms_e2e, ms_bwd = max_over_ranks([ms_total, ms_e2e, ms_bwd], dist, dev)
    if rank != 0:
        return None

    ms_step = ms_total / steps
    tokens = (B if pas == "decode" else cfg.tokens) * world
    value = whole_job_tokens_per_s(tokens // world, world, ms_step)
    peaks = measured_peaks()
    esz = 2 if cfg.dtype == "bf16" else 4
    Tn = 1 if pas == "decode" else T
    th = B * Tn * N                                              # token-heads per step
    in_bytes = B * Tn * (cfg.nq + cfg.nk) * K * esz + th * V * esz + th * 4          # q,k | v | gate
    state_bytes = 2 * B * N * K * V * 4                                                # h0 in, hT out
    traffic = None if (args.seq_len or args.multi_value) else profiled_traffic(workload, B * Tn * N)
    if pas == "decode":
        # HBM-bound: the fp32 state is read and written once per step
        alg_bytes = state_bytes + in_bytes + th * V * esz
        achieved = alg_bytes / (ms_step * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": traffic and traffic["bytes"],
                "traffic_source": traffic and traffic["source"], "call": "m2rnn_decode_step",
                "peak_source": f"{peaks['source']} HBM copy", "algorithmic_bytes_per_step": alg_bytes}
    else:
        # the contraction(s): forward 2KV^2 per token-head; backward 6KV^2 (recompute, dX W^T, H^T dX)
        call_ms = ms_bwd if bwd else ms_step
        flops = (6.0 if bwd else 2.0) * K * V * V * th
        alg_bytes = in_bytes + th * V * esz + state_bytes
        if bwd:  # + dy in, dq dk dv dgate out, dh0 out (checkpoints are not algorithmic)
            alg_bytes = 2 * in_bytes + th * V * esz + state_bytes
        t_tensor, t_hbm = flops / (peaks["tflops_burst"] * 1e12), alg_bytes / (peaks["hbm_gbs"] * 1e9)
        passes = 2 if bwd else 1                                 # tanh per state element: recompute counts once more
        mufu_s = th * K * V / (16 * SM_COUNT * SM_HZ)
        # the roofline that bounds the call: the slower of its contraction at the tensor peak and its
        # streamed bytes at the HBM bandwidth
        if cfg.dtype == "f32":   # the fp32 path is plain FMA: 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz
            bound, peak, psrc = "alu", SM_COUNT * 128 * 2 * SM_HZ / 1e12, "derived: 148 SMs x 128 fp32 FMA/clk x 1.965 GHz"
            achieved, unit = flops / (call_ms * 1e-3) / 1e12, "TFLOP/s"
        elif t_tensor >= t_hbm:
            bound, peak, psrc = "tensor", peaks["tflops_burst"], f"{peaks['source']} cuBLAS bf16 burst"
            achieved, unit = flops / (call_ms * 1e-3) / 1e12, "TFLOP/s"
        else:
            bound, peak, psrc = "hbm", peaks["hbm_gbs"], f"{peaks['source']} HBM copy"
            achieved, unit = alg_bytes / (call_ms * 1e-3) / 1e9, "GB/s"
        roof = {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "traffic": traffic and traffic["bytes"],
                "traffic_source": traffic and traffic["source"],
                "call": "m2rnn_bwd" if bwd else "m2rnn_fwd", "call_ms": call_ms,
                "peak_source": psrc, "algorithmic_bytes_per_call": alg_bytes, "flops_per_call": flops,
                "t_tensor_ms": t_tensor * 1e3, "t_hbm_ms": t_hbm * 1e3, "t_mufu_ms": mufu_s * 1e3,
                "frac_of_mufu_ceiling": mufu_s / (call_ms * 1e-3),
                "ns_per_scan_step": call_ms * 1e6 / T / passes}
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "pass": pas, "B": B, "T": Tn, "N": N, "K": K, "V": V,
                   "Nq": cfg.nq, "Nk": cfg.nk, "gate": "logit", "state": "fp32", "accumulate": "fp32",
                   "per_gpu_batch": B,
                   "l2": f"{ROTATE} input sets cycled; bytes touched per step {int((alg_bytes) / 1e6)} MB"
                         f" x {ROTATE} sets vs 126 MB L2"},
        "roofline": roof,
        "gpu_launches": steps * launches_per_step,
        "clocks": clocks.summary(),
    }
    if bwd:
        line["ms_fwd"], line["ms_bwd"] = ms_step - ms_bwd, ms_bwd
    if not args.no_e2e:
        line["e2e"] = {"value": tokens / (ms_e2e / e2e_steps * 1e-3), "unit": "tokens/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    if not args.no_cpu_baseline:
        rate, desc, dt = oracle_sample_rate(cfg, pas)
        line["cpu_baseline"] = {"value": rate, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": desc,
                                "seconds": dt}
        if pas != "decode":
            rate32, cores, desc32, dt32 = oracle_all_cores_rate(cfg, pas)
            line["cpu_baseline"]["fp32_all_cores"] = {"value": rate32, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                                      "sample": desc32, "seconds": dt32}
    return line


if __name__ == "__main__":
    main()
