"""The tcgen05 backward kernel (V = 128: every product of a step on the 5th-generation tensor
cores, W and W^T in tensor memory) against the fp64 oracle; and the register kernel on the same
shapes, forced through M2RNN_BWD_VARIANT=mma, so that both paths stay covered."""
import numpy as np
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import GATE_LOGIT, GATE_PSI, GATE_VALUE, ScanConfig

pytestmark = pytest.mark.gpu
F = inputs.to_f64

SHAPES = [
    # B, T, N, K, Nq, Nk        (V = 128)
    (1, 21, 2, 128, 0, 0),
    (2, 37, 2, 32, 0, 0),       # one 32-row CTA per unit: dv and dgate written directly
    (1, 26, 4, 96, 2, 4),       # three CTAs per unit, shared query heads
    (1, 13, 2, 48, 0, 0),       # K not a multiple of 32: the register kernel takes it either way
    (2, 9, 3, 32, 1, 1),        # the multi-value layout
    (3, 1, 2, 64, 0, 0),        # a single step
    (1, 4, 1, 64, 0, 0),        # exactly one chunk
    (1, 5, 1, 32, 0, 0),        # a chunk and one step
    (20, 7, 4, 32, 0, 0),       # more CTAs than SMs
]


@pytest.mark.parametrize("variant", ["tc", "mma"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("gate_kind", [GATE_VALUE, GATE_LOGIT, GATE_PSI])
def test_shapes_backward(oracle, monkeypatch, shape, gate_kind, variant):
    monkeypatch.setenv("M2RNN_BWD_VARIANT", variant)
    B, T, N, K, Nq, Nk = shape
    cfg = ScanConfig("case", B=B, T=T, N=N, K=K, V=128, Nq=Nq, Nk=Nk, gate_kind=gate_kind, gate_mean=1.0,
                     w_scale=0.5 if gate_kind == GATE_PSI else 1.0, seed=600 + T)
    errs = parity.check_bwd(oracle, cfg, residual=True, d_hT=True)
    assert max(errs.values()) < 1.5e-2, errs


def test_checkpoints_recomputed_when_not_passed(oracle):
    cfg = ScanConfig("nock", B=2, T=29, N=2, K=32, V=128, gate_mean=1.0, seed=21)
    parity.check_bwd(oracle, cfg, use_fwd_ckpt=False)


def test_saturating_inputs_and_clipping(oracle):
    cfg = ScanConfig("sat", B=2, T=48, N=2, K=128, V=128, dist="saturating", gate_mean=0.0, seed=7)
    parity.check_bwd(oracle, cfg)
    cfg = ScanConfig("clip", B=2, T=24, N=2, K=32, V=128, dist="saturating", gate_mean=1.0, seed=9)
    parity.check_bwd(oracle, cfg, dh_clip=0.5)


def test_shorter_chunks(oracle):
    cfg = ScanConfig("ck2", B=1, T=23, N=2, K=32, V=128, gate_mean=1.0, seed=13)
    d = inputs.make_inputs(cfg, backward=True)
    ref = parity.oracle_bwd(oracle, cfg, d)
    g = parity.to_dev(d)
    _, _, ckpt = parity.gpu_fwd(cfg, g, save_ckpt=True, ckpt_interval=2)
    out = parity.gpu_bwd(cfg, g, ckpt=ckpt, ckpt_interval=2)
    binding.check_device_status()
    for name in ref:
        assert parity.rel_err(out[name], ref[name]) < 1.5e-2, name


def test_repeats_bit_for_bit_and_matches_the_register_kernel(monkeypatch):
    cfg = ScanConfig("det", B=3, T=50, N=4, K=64, V=128, Nq=1, Nk=1, seed=11)
    g = parity.to_dev(inputs.make_inputs(cfg, backward=True))
    a = parity.gpu_bwd(cfg, g)
    b = parity.gpu_bwd(cfg, g)
    for name in a:
        assert torch.equal(a[name], b[name]), name
    monkeypatch.setenv("M2RNN_BWD_VARIANT", "mma")
    c = parity.gpu_bwd(cfg, g)
    for name in a:      # two correct bf16 implementations: equal to rounding
        assert parity.rel_err(a[name], c[name].double().cpu().numpy()) < 2e-2, name
    binding.check_device_status()


def test_packed_batch_with_an_empty_sequence(oracle):
    lengths = [19, 0, 8, 1]
    cfg = ScanConfig("vl", B=len(lengths), T=max(lengths), N=2, K=32, V=128, gate_mean=1.0, seed=427)
    dense = inputs.make_inputs(cfg, backward=True, d_hT=True)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    d = {x: (torch.cat([t[b, :L] for b, L in enumerate(lengths)], dim=0).contiguous()
             if x in ("q", "k", "v", "gate", "dy") and t is not None else t) for x, t in dense.items()}
    ref = oracle.bwd_varlen(F(d["q"]), F(d["k"]), F(d["v"]), F(d["gate"]), F(d["W"]), cu, F(d["h0"]), F(d["dy"]), F(d["d_hT"]))
    g = parity.to_dev(d)
    kw = dict(cu_seqlens=torch.from_numpy(cu).cuda(), max_seqlen=max(lengths))
    _, _, ckpt = binding.m2rnn_fwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], save_ckpt=True, **kw)
    out = binding.m2rnn_bwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], g["dy"], g["d_hT"], ckpt=ckpt, **kw)
    binding.check_device_status()
    for x in ref:
        assert parity.rel_err(out[x], ref[x]) <= 2e-2, x
    assert torch.equal(out["dh0"][1], g["d_hT"][1])
