"""bf16 tensor-core backward through time against the fp64 oracle
(max relative error <= 2e-2 on every gradient; inputs are the bf16-rounded values)."""
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import CONFIGS, GATE_LOGIT, GATE_PSI, GATE_VALUE, ScanConfig

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, T, N, K, V, Nq, Nk       T spans several chunks and a ragged tail
    (2, 50, 3, 16, 16, 0, 0),
    (1, 37, 2, 32, 32, 0, 0),
    (2, 45, 2, 64, 64, 0, 0),
    (1, 21, 2, 128, 128, 0, 0),
    (2, 33, 4, 64, 16, 1, 1),     # the paper's K=64, V=16 multi-value layout
    (1, 26, 4, 48, 32, 2, 4),     # K = 3 row slabs of 16
    (1, 11, 1, 16, 128, 0, 0),
    (1, 19, 2, 112, 64, 1, 2),    # K = 7 row slabs of 16
    (3, 1, 2, 64, 64, 0, 0),      # a single step
    (1, 4, 1, 64, 64, 0, 0),      # exactly one chunk
    (40, 9, 4, 64, 64, 0, 0),     # enough units that a CTA takes all 64 rows
    (40, 7, 4, 32, 128, 0, 0),    # ... and the 32-row CTAs of V = 128 (W in shared memory)
    (40, 7, 4, 32, 64, 0, 0),     # two slabs per CTA
    (40, 15, 4, 64, 16, 1, 1),    # V = 16 with more units than SMs: shorter chunks, two CTAs per SM
    (4, 13, 84, 64, 16, 1, 1),    # the paper's layer shape (336 units): 32-row CTAs, three per SM
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("gate_kind", [GATE_VALUE, GATE_LOGIT, GATE_PSI])
def test_shapes_backward(oracle, shape, gate_kind):
    B, T, N, K, V, Nq, Nk = shape
    # W ~ N(0, 1/V) as in the benchmark configurations for the value and logit gates, half that
    # scale for the psi gate (short memory: chaotic at full scale, see test_parity_bf16_fwd.W_SCALE)
    cfg = ScanConfig("case", B=B, T=T, N=N, K=K, V=V, Nq=Nq, Nk=Nk, gate_kind=gate_kind, gate_mean=1.0,
                     w_scale=0.5 if gate_kind == GATE_PSI else 1.0, seed=300 + T)
    errs = parity.check_bwd(oracle, cfg, residual=True, d_hT=True)
    assert max(errs.values()) < 1.5e-2, errs


def test_checkpoints_recomputed_when_not_passed(oracle):
    cfg = ScanConfig("nock", B=2, T=29, N=2, K=32, V=64, gate_mean=1.0, seed=21)
    parity.check_bwd(oracle, cfg, use_fwd_ckpt=False)


@pytest.mark.parametrize("K,V", [(16, 16), (64, 64), (128, 128)])
def test_saturating_inputs(oracle, K, V):
    """tanh far from its linear range: dX = dZ (1 - Z^2) is taken where |Z| is close to 1."""
    cfg = ScanConfig("sat", B=2, T=48, N=2, K=K, V=V, dist="saturating", gate_mean=0.0, seed=7)
    parity.check_bwd(oracle, cfg)


def test_identity_transition_and_zero_state(oracle):
    cfg = ScanConfig("eye", B=2, T=70, N=3, K=64, V=16, Nq=1, Nk=1, dist="identity_w", h0_std=0.0, seed=8)
    parity.check_bwd(oracle, cfg)


def test_state_gradient_clipping(oracle):
    # The carried gradient has unit scale here, so 0.5 clamps a good part of it at every step.  (A
    # threshold far below that scale would make the clamped outputs' own magnitude, by which the
    # error is normalised, much smaller than the rounding error of the values it did not clamp.)
    cfg = ScanConfig("clip", B=2, T=24, N=2, K=16, V=32, dist="saturating", gate_mean=1.0, seed=9)
    parity.check_bwd(oracle, cfg, dh_clip=0.5)


def test_explicit_checkpoint_interval(oracle):
    cfg = ScanConfig("ck2", B=1, T=23, N=2, K=32, V=32, gate_mean=1.0, seed=13)
    d = inputs.make_inputs(cfg, backward=True)
    ref = parity.oracle_bwd(oracle, cfg, d)
    g = parity.to_dev(d)
    for C in (2, 6):
        _, _, ckpt = parity.gpu_fwd(cfg, g, save_ckpt=True, ckpt_interval=C)
        assert ckpt.shape[2] == (cfg.T + C - 1) // C
        out = parity.gpu_bwd(cfg, g, ckpt=ckpt, ckpt_interval=C)
        binding.check_device_status()
        for name in ref:
            assert parity.rel_err(out[name], ref[name]) < 1e-2, (C, name)


def test_backward_repeats_bit_for_bit():
    cfg = ScanConfig("det", B=4, T=50, N=4, K=64, V=32, Nq=1, Nk=1, seed=11)
    g = parity.to_dev(inputs.make_inputs(cfg, backward=True))
    a = parity.gpu_bwd(cfg, g)
    b = parity.gpu_bwd(cfg, g)
    for name in a:
        assert torch.equal(a[name], b[name]), name
    binding.check_device_status()
