"""Seeded synthetic inputs for the M2RNN scan: shapes and distributions only.

This module holds none of the method's arithmetic.  It is the one piece of code
the CUDA library's tests/bench and the CPU oracle's tests both use, so that the
two sides see bit-identical inputs.  Values are drawn in fp32 on the CPU from a
numpy PCG64 stream in the fixed order q, k, v, gate, W, h0, dy, d_hT, then the
q/k/v/W/dy tensors are rounded (nearest-even) to the I/O dtype; the oracle is fed
those rounded values widened to fp64.

Layouts (paper, Algorithm 1/2 I/O lists): q [B,T,Nq,K], k [B,T,Nk,K],
v [B,T,N,V], gate [B,T,N] (fp32), W [N,V,V], h0 [B,N,K,V] (fp32), dy [B,T,N,V].
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

GATE_VALUE, GATE_LOGIT, GATE_PSI = 0, 1, 2


@dataclass(frozen=True)
class ScanConfig:
    name: str
    B: int
    T: int
    N: int
    K: int
    V: int
    dtype: str = "bf16"          # I/O dtype of q,k,v,W,y,dy and the gradients: "bf16" | "f32"
    Nq: int = 0                  # 0 -> N (multi-head); 1 -> the paper's multi-value layout
    Nk: int = 0
    gate_kind: int = GATE_LOGIT
    gate_mean: float = 2.0       # gate pre-activations ~ N(gate_mean, 1)
    h0_std: float = 0.1          # 0 -> zero initial state (passed as NULL)
    dist: str = "baseline"       # "baseline" | "saturating" | "identity_w"
    w_scale: float = 1.0         # W ~ N(0, w_scale^2 / V): 1 puts the recurrence at the edge of stability
    seed: int = 0

    @property
    def nq(self) -> int:
        return self.Nq or self.N

    @property
    def nk(self) -> int:
        return self.Nk or self.N

    @property
    def tokens(self) -> int:
        return self.B * self.T

    def with_(self, **kw) -> "ScanConfig":
        return replace(self, **kw)


# The five benchmark configurations (state-size sweep and long-context/decode expanded).
CONFIGS = {
    "tiny_f32": ScanConfig("tiny_f32", B=1, T=64, N=2, K=16, V=16, dtype="f32",
                           gate_mean=0.0, h0_std=0.0, seed=0),
    "fwd_bf16": ScanConfig("fwd_bf16", B=8, T=2048, N=16, K=64, V=64, seed=1),
    "bptt_bf16": ScanConfig("bptt_bf16", B=8, T=4096, N=32, K=64, V=64, seed=2),
    "sweep16": ScanConfig("sweep16", B=4, T=8192, N=16, K=16, V=16, seed=3),
    "sweep32": ScanConfig("sweep32", B=4, T=8192, N=16, K=32, V=32, seed=3),
    "sweep64": ScanConfig("sweep64", B=4, T=8192, N=16, K=64, V=64, seed=3),
    "sweep128": ScanConfig("sweep128", B=4, T=8192, N=16, K=128, V=128, seed=3),
    "long_ctx": ScanConfig("long_ctx", B=1, T=65536, N=32, K=128, V=128, seed=4),
    "decode": ScanConfig("decode", B=512, T=1, N=32, K=128, V=128, seed=4),
    # the layer shape of the paper's own models: K=64, V=16, 84 value heads sharing one q/k head,
    # identity-initialised transition matrices, 4k training context
    "paper_layer": ScanConfig("paper_layer", B=4, T=4096, N=84, K=64, V=16, Nq=1, Nk=1,
                              dist="identity_w", seed=5),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]


def _normal(rng: np.random.Generator, shape, std=1.0, mean=0.0) -> torch.Tensor:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    if mean != 0.0:
        a += np.float32(mean)
    return torch.from_numpy(a)


def make_inputs(cfg: ScanConfig, *, backward: bool = False, seed: int | None = None,
                psi_params: bool = False, residual: bool = False, d_hT: bool = False) -> dict:
    """CPU tensors for one scan call.

    baseline:    q,k,v ~ N(0,1)/sqrt(K); W ~ N(0, 1/V) (std V^-1/2); gate ~ N(gate_mean,1);
                 h0 ~ N(0, h0_std^2) (None when h0_std == 0); dy ~ N(0,1).
    identity_w:  as baseline with W = I (the paper's initialisation of W).
    saturating:  q,k,v ~ N(0,1) (so k v^T has unit scale); W ~ N(0,1/V); h0 ~ U(-1,1): drives
                 tanh well into its non-linear range so a wrong non-linearity cannot pass, while
                 the map stays contracting (an expanding W would amplify rounding differences
                 between any two correct implementations).
    """
    rng = np.random.Generator(np.random.PCG64(cfg.seed if seed is None else seed))
    io = torch_dtype(cfg.dtype)
    B, T, N, K, V = cfg.B, cfg.T, cfg.N, cfg.K, cfg.V
    sat = cfg.dist == "saturating"
    s_in = 1.0 if sat else K ** -0.5
    out = {}
    out["q"] = _normal(rng, (B, T, cfg.nq, K), s_in).to(io)
    out["k"] = _normal(rng, (B, T, cfg.nk, K), s_in).to(io)
    out["v"] = _normal(rng, (B, T, N, V), s_in).to(io)
    gate = _normal(rng, (B, T, N), 1.0, cfg.gate_mean)
    if cfg.gate_kind == GATE_VALUE:
        gate = torch.sigmoid(gate)
    out["gate"] = gate
    W = _normal(rng, (N, V, V), cfg.w_scale * V ** -0.5)
    if cfg.dist == "identity_w":
        W = torch.eye(V).expand(N, V, V).clone()
    out["W"] = W.to(io)
    if sat:
        out["h0"] = torch.from_numpy(rng.uniform(-1.0, 1.0, size=(B, N, K, V)).astype(np.float32))
    elif cfg.h0_std > 0:
        out["h0"] = _normal(rng, (B, N, K, V), cfg.h0_std)
    else:
        out["h0"] = None
    if backward:
        out["dy"] = _normal(rng, (B, T, N, V)).to(io)
        out["d_hT"] = _normal(rng, (B, N, K, V), 0.1) if d_hT else None
    if psi_params or cfg.gate_kind == GATE_PSI:
        # alpha ~ U(0.5, 2), beta ~ LogU(0.1, 2): one pair per head
        out["alpha"] = torch.from_numpy(rng.uniform(0.5, 2.0, size=(N,)).astype(np.float32))
        out["beta"] = torch.from_numpy(np.exp(rng.uniform(np.log(0.1), np.log(2.0), size=(N,))).astype(np.float32))
    else:
        out["alpha"] = out["beta"] = None
    out["w_r"] = _normal(rng, (N, V), 1.0).to(io) if residual else None
    return out


def make_gated_norm_inputs(B: int, T: int, N: int, V: int, dtype: str = "bf16", seed: int = 0) -> dict:
    """CPU tensors for the output path after the scan: y, g_in, dout [B,T,N,V] ~ N(0,1) (the scan's
    readout is of unit scale), w [N*V] ~ U(0.5, 1.5); drawn in fp32 in that order from one PCG64
    stream, then rounded to the I/O dtype."""
    rng = np.random.Generator(np.random.PCG64(seed))
    io = torch_dtype(dtype)
    out = {"y": _normal(rng, (B, T, N, V)).to(io), "g_in": _normal(rng, (B, T, N, V)).to(io)}
    out["dout"] = _normal(rng, (B, T, N, V)).to(io)
    out["w"] = torch.from_numpy(rng.uniform(0.5, 1.5, size=(N * V,)).astype(np.float32)).to(io)
    return out


def to_f64(t):
    """Exact widening of a (possibly bf16) tensor to a numpy float64 array; None stays None."""
    return None if t is None else t.detach().to("cpu", torch.float64).numpy()


def make_conv_inputs(B: int, T: int, C: int, dtype: str, seed: int = 0, prev: bool = True) -> dict:
    """Inputs of the path before the scan (SiLU of a depthwise causal conv1d over the projections):
    x, dout ~ N(0,1), filter taps w ~ N(0, 1/4) (so that the pre-activation has unit scale), bias ~
    N(0, 0.1^2), the three carried rows ~ N(0,1); rounded to the I/O dtype."""
    rng = np.random.Generator(np.random.PCG64(seed))
    io = torch_dtype(dtype)
    out = dict(x=_normal(rng, (B, T, C)).to(io), w=_normal(rng, (C, 4), 0.5).to(io), bias=_normal(rng, (C,), 0.1).to(io),
               dout=_normal(rng, (B, T, C)).to(io))
    out["prev"] = _normal(rng, (B, 3, C)).to(io) if prev else None
    return out
