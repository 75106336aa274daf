"""bf16 decoding step against the fp64 oracle (max relative error <= 2e-2 on y and the new state)."""
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import GATE_LOGIT, GATE_PSI, GATE_VALUE, ScanConfig

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, N, K, V, Nq, Nk
    (37, 3, 16, 16, 0, 0),        # eight units per CTA pass, ragged batch
    (9, 2, 32, 32, 0, 0),
    (5, 4, 64, 64, 1, 2),
    (7, 2, 128, 128, 0, 0),
    (11, 4, 64, 16, 1, 1),        # the paper's K=64, V=16 multi-value layout
    (6, 4, 48, 32, 2, 4),         # three warps per unit, two idle warps per CTA
    (3, 1, 16, 128, 0, 0),
    (4, 2, 112, 64, 1, 2),
    (1, 1, 64, 64, 0, 0),
    (300, 5, 32, 64, 0, 0),       # more tasks than SMs: several per CTA, head changes inside a CTA
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("gate_kind", [GATE_VALUE, GATE_LOGIT, GATE_PSI])
def test_decode_shapes(oracle, shape, gate_kind):
    B, N, K, V, Nq, Nk = shape
    cfg = ScanConfig("dec", B=B, T=3, N=N, K=K, V=V, Nq=Nq, Nk=Nk, gate_kind=gate_kind, gate_mean=1.0, seed=400 + B)
    d = inputs.make_inputs(cfg, residual=True)
    g = parity.to_dev(d)
    f = inputs.to_f64
    state = g["h0"].clone()
    ref_state = f(d["h0"])
    for t in range(cfg.T):
        y_ref, ref_state = oracle.decode_step(f(d["q"][:, t]), f(d["k"][:, t]), f(d["v"][:, t]), f(d["gate"][:, t]),
                                              f(d["W"]), ref_state, gate_kind=cfg.gate_kind, alpha=f(d["alpha"]),
                                              beta=f(d["beta"]), w_r=f(d["w_r"]))
        yt = binding.m2rnn_decode_step(g["q"][:, t].clone(), g["k"][:, t].clone(), g["v"][:, t].clone(),
                                       g["gate"][:, t].clone(), g["W"], state, gate_kind=cfg.gate_kind,
                                       alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"])
        assert parity.rel_err(yt, y_ref) < 1e-2 and parity.rel_err(state, ref_state) < 1e-2, t
    binding.check_device_status()


def test_decode_chain_tracks_the_scan():
    """T decode steps and one forward scan follow the same recurrence with the same arithmetic
    (bf16 operands, fp32 state); they use different kernels, so they agree to rounding, not bitwise."""
    cfg = ScanConfig("chain", B=6, T=24, N=3, K=64, V=64, gate_mean=1.0, w_scale=0.5, seed=17)
    g = parity.to_dev(inputs.make_inputs(cfg))
    y, hT, _ = parity.gpu_fwd(cfg, g)
    state = g["h0"].clone()
    ys = [binding.m2rnn_decode_step(g["q"][:, t].clone(), g["k"][:, t].clone(), g["v"][:, t].clone(),
                                    g["gate"][:, t].clone(), g["W"], state) for t in range(cfg.T)]
    yd = torch.stack(ys, dim=1)
    assert parity.rel_err(yd, y.double().cpu().numpy()) < 1e-2
    assert parity.rel_err(state, hT.double().cpu().numpy()) < 1e-3
