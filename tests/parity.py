"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the
same seeded inputs and compare every output with ||gpu - ref||_inf / ||ref||_inf."""
from __future__ import annotations

import numpy as np
import torch

from paper_2603_14360_b200 import binding, inputs

# max relative error (infinity norms, per tensor) allowed for each I/O dtype
TOL = {"f32": 1e-4, "bf16": 2e-2}


def rel_err(gpu, ref) -> float:
    g = gpu.detach().to("cpu", torch.float64).numpy() if isinstance(gpu, torch.Tensor) else np.asarray(gpu)
    assert g.shape == ref.shape, (g.shape, ref.shape)
    assert np.isfinite(g).all()
    den = np.abs(ref).max()
    return float(np.abs(g - ref).max() / den) if den > 0 else float(np.abs(g).max())


def to_dev(d, dev="cuda"):
    return {k: (v.to(dev) if isinstance(v, torch.Tensor) else v) for k, v in d.items()}


def oracle_fwd(oracle, cfg, d, **kw):
    f = inputs.to_f64
    return oracle.fwd(f(d["q"]), f(d["k"]), f(d["v"]), f(d["gate"]), f(d["W"]), f(d["h0"]),
                      gate_kind=cfg.gate_kind, alpha=f(d["alpha"]), beta=f(d["beta"]), w_r=f(d["w_r"]), **kw)


def oracle_bwd(oracle, cfg, d, dh_clip=0.0):
    f = inputs.to_f64
    return oracle.bwd(f(d["q"]), f(d["k"]), f(d["v"]), f(d["gate"]), f(d["W"]), f(d["h0"]), f(d["dy"]),
                      f(d["d_hT"]), gate_kind=cfg.gate_kind, alpha=f(d["alpha"]), beta=f(d["beta"]),
                      w_r=f(d["w_r"]), dh_clip=dh_clip)


def gpu_fwd(cfg, g, **kw):
    return binding.m2rnn_fwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], gate_kind=cfg.gate_kind,
                             alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"], **kw)


def gpu_bwd(cfg, g, **kw):
    return binding.m2rnn_bwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], g["dy"], g["d_hT"],
                             gate_kind=cfg.gate_kind, alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"], **kw)


def check_fwd(oracle, cfg, *, tol=None, **mk):
    tol = tol or TOL[cfg.dtype]
    d = inputs.make_inputs(cfg, **mk)
    y_ref, hT_ref = oracle_fwd(oracle, cfg, d)
    y, hT, _ = gpu_fwd(cfg, to_dev(d))
    binding.check_device_status()
    errs = dict(y=rel_err(y, y_ref), hT=rel_err(hT, hT_ref))
    assert max(errs.values()) <= tol, (cfg.name, errs)
    return errs


def check_bwd(oracle, cfg, *, tol=None, use_fwd_ckpt=True, dh_clip=0.0, **mk):
    tol = tol or TOL[cfg.dtype]
    d = inputs.make_inputs(cfg, backward=True, **mk)
    ref = oracle_bwd(oracle, cfg, d, dh_clip=dh_clip)
    g = to_dev(d)
    ckpt = None
    if use_fwd_ckpt:
        _, _, ckpt = gpu_fwd(cfg, g, save_ckpt=True)
    out = gpu_bwd(cfg, g, ckpt=ckpt, dh_clip=dh_clip)
    binding.check_device_status()
    errs = {name: rel_err(out[name], ref[name]) for name in ref}
    assert max(errs.values()) <= tol, (cfg.name, errs)
    return errs
