"""The input path before the scan (SiLU of a depthwise causal conv1d of width 4 over the q, k, v
projections) against the fp64 oracle, forward and backward; and the chain conv -> strided views ->
scan that the library is meant to be used in."""
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import ScanConfig

pytestmark = pytest.mark.gpu
F = inputs.to_f64

SHAPES = [(2, 37, 64), (1, 1, 8), (3, 200, 328), (1, 64, 8), (2, 129, 1032), (4, 3, 16)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("with_prev", [False, True])
def test_forward_backward(oracle, dtype, shape, with_prev):
    B, T, C = shape
    d = inputs.make_conv_inputs(B, T, C, dtype, seed=500 + T, prev=with_prev)
    g = {k: (None if v is None else v.cuda()) for k, v in d.items()}
    tol = parity.TOL[dtype]
    out = binding.m2rnn_conv_silu_fwd(g["x"], g["w"], g["bias"], g["prev"])
    ref = oracle.conv_silu_fwd(F(d["x"]), F(d["w"]), F(d["bias"]), F(d["prev"]))
    assert parity.rel_err(out, ref) <= tol
    got = binding.m2rnn_conv_silu_bwd(g["x"], g["w"], g["dout"], g["bias"], g["prev"])
    want = oracle.conv_silu_bwd(F(d["x"]), F(d["w"]), F(d["dout"]), F(d["bias"]), F(d["prev"]))
    for name in ("dx", "dw", "dbias") + (("dprev",) if with_prev else ()):
        assert parity.rel_err(got[name], want[name]) <= tol, name
    again = binding.m2rnn_conv_silu_bwd(g["x"], g["w"], g["dout"], g["bias"], g["prev"])
    assert all(torch.equal(again[x], got[x]) for x in got if got[x] is not None)     # fixed-order sums


def test_no_bias_and_empty(oracle):
    d = inputs.make_conv_inputs(2, 19, 32, "f32", seed=9, prev=False)
    g = {k: (None if v is None else v.cuda()) for k, v in d.items()}
    out = binding.m2rnn_conv_silu_fwd(g["x"], g["w"])
    assert parity.rel_err(out, oracle.conv_silu_fwd(F(d["x"]), F(d["w"]))) <= 1e-4
    e = binding.m2rnn_conv_silu_fwd(g["x"][:, :0], g["w"])
    assert e.shape == (2, 0, 32)
    r = binding.m2rnn_conv_silu_bwd(g["x"][:, :0].contiguous(), g["w"], g["dout"][:, :0].contiguous())
    assert float(r["dw"].abs().max()) == 0.0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_projection_through_conv_into_the_scan(oracle, dtype):
    """One [B,T,Nq K + Nk K + N V] projection tensor -> one conv call in place of three -> column
    slices of its output as the scan's strided q, k, v; backward the same way round."""
    cfg = ScanConfig("chain", B=2, T=45, N=4, K=32, V=16, Nq=1, Nk=1, dtype=dtype, gate_mean=1.0, seed=91)
    wq, wv = cfg.nq * cfg.K, cfg.N * cfg.V
    C = 2 * wq + wv
    d = inputs.make_conv_inputs(cfg.B, cfg.T, C, dtype, seed=92, prev=False)
    s = inputs.make_inputs(cfg, backward=True)
    g = {k: (None if v is None else v.cuda()) for k, v in d.items()}
    gs = parity.to_dev(s)
    act = binding.m2rnn_conv_silu_fwd(g["x"], g["w"], g["bias"])
    q = act[..., :wq].unflatten(2, (cfg.nq, cfg.K))
    k = act[..., wq:2 * wq].unflatten(2, (cfg.nk, cfg.K))
    v = act[..., 2 * wq:].unflatten(2, (cfg.N, cfg.V))
    y, hT, ckpt = binding.m2rnn_fwd(q, k, v, gs["gate"], gs["W"], gs["h0"], save_ckpt=True)
    grads = binding.m2rnn_bwd(q, k, v, gs["gate"], gs["W"], gs["h0"], gs["dy"], ckpt=ckpt)
    dact = torch.cat([grads["dq"].flatten(2), grads["dk"].flatten(2), grads["dv"].flatten(2)], dim=2)
    back = binding.m2rnn_conv_silu_bwd(g["x"], g["w"], dact, g["bias"])
    binding.check_device_status()
    # the oracle, step by step in fp64 from the same inputs
    act_ref = oracle.conv_silu_fwd(F(d["x"]), F(d["w"]), F(d["bias"]))
    qr, kr = act_ref[..., :wq].reshape(cfg.B, cfg.T, cfg.nq, cfg.K), act_ref[..., wq:2 * wq].reshape(cfg.B, cfg.T, cfg.nk, cfg.K)
    vr = act_ref[..., 2 * wq:].reshape(cfg.B, cfg.T, cfg.N, cfg.V)
    y_ref, hT_ref = oracle.fwd(qr, kr, vr, F(s["gate"]), F(s["W"]), F(s["h0"]))
    r = oracle.bwd(qr, kr, vr, F(s["gate"]), F(s["W"]), F(s["h0"]), F(s["dy"]))
    import numpy as np
    dact_ref = np.concatenate([r["dq"].reshape(cfg.B, cfg.T, -1), r["dk"].reshape(cfg.B, cfg.T, -1), r["dv"].reshape(cfg.B, cfg.T, -1)], axis=2)
    back_ref = oracle.conv_silu_bwd(F(d["x"]), F(d["w"]), dact_ref, F(d["bias"]))
    tol = parity.TOL[dtype]
    assert parity.rel_err(y, y_ref) <= tol and parity.rel_err(hT, hT_ref) <= tol
    for name in ("dx", "dw", "dbias"):
        assert parity.rel_err(back[name], back_ref[name]) <= tol, name
