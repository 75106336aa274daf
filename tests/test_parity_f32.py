"""fp32 path of the CUDA library against the fp64 oracle (max relative error <= 1e-4)."""
import numpy as np
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import CONFIGS, GATE_LOGIT, GATE_PSI, GATE_VALUE, ScanConfig

pytestmark = pytest.mark.gpu


def test_tiny_config_forward(oracle):
    errs = parity.check_fwd(oracle, CONFIGS["tiny_f32"])
    assert max(errs.values()) < 1e-5


def test_tiny_config_backward(oracle):
    errs = parity.check_bwd(oracle, CONFIGS["tiny_f32"])
    assert max(errs.values()) < 1e-5
    parity.check_bwd(oracle, CONFIGS["tiny_f32"], use_fwd_ckpt=False)


SHAPES = [
    # B, T, N, K, V, Nq, Nk
    (2, 37, 3, 16, 16, 0, 0),
    (1, 19, 2, 32, 64, 0, 0),
    (2, 21, 4, 64, 16, 1, 1),     # the paper's K=64, V=16 multi-value layout
    (1, 9, 2, 128, 128, 0, 0),
    (2, 18, 4, 48, 32, 2, 4),
    (1, 5, 1, 16, 128, 0, 0),
    (1, 33, 2, 112, 64, 1, 2),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("gate_kind", [GATE_VALUE, GATE_LOGIT, GATE_PSI])
def test_shapes_forward_backward(oracle, shape, gate_kind):
    B, T, N, K, V, Nq, Nk = shape
    cfg = ScanConfig("case", B=B, T=T, N=N, K=K, V=V, Nq=Nq, Nk=Nk, dtype="f32", gate_kind=gate_kind,
                     gate_mean=1.0, seed=100 + T)
    parity.check_fwd(oracle, cfg, residual=True)
    parity.check_bwd(oracle, cfg, residual=True, d_hT=True)


@pytest.mark.parametrize("K,V", [(16, 16), (64, 64)])
def test_saturating_inputs(oracle, K, V):
    """tanh driven far from its linear range, so a wrong non-linearity cannot pass."""
    cfg = ScanConfig("sat", B=2, T=64, N=2, K=K, V=V, dtype="f32", dist="saturating", gate_mean=0.0, seed=7)
    parity.check_fwd(oracle, cfg)
    parity.check_bwd(oracle, cfg)


def test_no_initial_state_and_split_scan(oracle):
    cfg = ScanConfig("split", B=2, T=40, N=2, K=32, V=32, dtype="f32", h0_std=0.0, seed=3)
    d = inputs.make_inputs(cfg)
    assert d["h0"] is None
    g = parity.to_dev(d)
    y, hT, _ = parity.gpu_fwd(cfg, g)
    y_ref, hT_ref = parity.oracle_fwd(oracle, cfg, d)
    assert parity.rel_err(y, y_ref) < 1e-4 and parity.rel_err(hT, hT_ref) < 1e-4
    # the final state resumes the scan exactly (state is fp32 end to end)
    a = {x: g[x][:, :17].contiguous() for x in ("q", "k", "v", "gate")}
    b = {x: g[x][:, 17:].contiguous() for x in ("q", "k", "v", "gate")}
    ya, ha, _ = binding.m2rnn_fwd(a["q"], a["k"], a["v"], a["gate"], g["W"], None)
    yb, hb, _ = binding.m2rnn_fwd(b["q"], b["k"], b["v"], b["gate"], g["W"], ha)
    assert torch.equal(torch.cat([ya, yb], dim=1), y) and torch.equal(hb, hT)


def test_decode_chain_equals_scan(oracle):
    cfg = ScanConfig("dec", B=3, T=12, N=2, K=32, V=16, Nq=1, Nk=2, dtype="f32", gate_kind=GATE_PSI, seed=5)
    d = inputs.make_inputs(cfg, residual=True)
    g = parity.to_dev(d)
    y, hT, _ = parity.gpu_fwd(cfg, g)
    state = g["h0"].clone()
    for t in range(cfg.T):
        yt = binding.m2rnn_decode_step(g["q"][:, t].contiguous(), g["k"][:, t].contiguous(),
                                       g["v"][:, t].contiguous(), g["gate"][:, t].contiguous(), g["W"], state,
                                       gate_kind=cfg.gate_kind, alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"])
        assert torch.equal(yt, y[:, t])
    assert torch.equal(state, hT)
    # and one step against the oracle directly
    f = inputs.to_f64
    y1, s1 = oracle.decode_step(f(d["q"][:, 0]), f(d["k"][:, 0]), f(d["v"][:, 0]), f(d["gate"][:, 0]), f(d["W"]),
                                f(d["h0"]), gate_kind=cfg.gate_kind, alpha=f(d["alpha"]), beta=f(d["beta"]), w_r=f(d["w_r"]))
    st = g["h0"].clone()
    yg = binding.m2rnn_decode_step(g["q"][:, 0].contiguous(), g["k"][:, 0].contiguous(), g["v"][:, 0].contiguous(),
                                   g["gate"][:, 0].contiguous(), g["W"], st, gate_kind=cfg.gate_kind,
                                   alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"])
    assert parity.rel_err(yg, y1) < 1e-4 and parity.rel_err(st, s1) < 1e-4


def test_state_gradient_clipping(oracle):
    cfg = ScanConfig("clip", B=2, T=24, N=2, K=16, V=32, dtype="f32", dist="saturating", gate_mean=1.0, seed=9)
    parity.check_bwd(oracle, cfg, dh_clip=0.05)


def test_backward_repeats_bit_for_bit(oracle):
    cfg = ScanConfig("det", B=4, T=50, N=4, K=32, V=32, Nq=1, Nk=1, dtype="f32", seed=11)
    g = parity.to_dev(inputs.make_inputs(cfg, backward=True))
    a = parity.gpu_bwd(cfg, g)
    b = parity.gpu_bwd(cfg, g)
    for name in a:
        assert torch.equal(a[name], b[name]), name
