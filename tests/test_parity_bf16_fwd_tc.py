"""The tcgen05 forward scan kernel (tensor-memory accumulator, transposed product with the
transition matrix stationary) against the fp64 oracle, forced through M2RNN_FWD_VARIANT=tc so that
every shape below runs in that kernel whatever the library's default choice is."""
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import GATE_LOGIT, GATE_PSI, GATE_VALUE, ScanConfig

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["32", "64"], ids=["rows32", "rows64"])
def _force_tc(monkeypatch, request):
    """Both tilings of the kernel: two chain groups of 16 or of 32 state rows per CTA (the library
    falls back to 16-row groups where K is not a multiple of 32)."""
    monkeypatch.setenv("M2RNN_FWD_VARIANT", "tc")
    monkeypatch.setenv("M2RNN_TC_ROWS", request.param)


SHAPES = [
    # B, T, N, K, V, Nq, Nk
    (2, 100, 3, 16, 16, 0, 0),    # 8 heads per tile, 3 live; one 16-row group
    (1, 77, 2, 32, 32, 0, 0),     # 4 heads per tile, 2 live
    (2, 131, 2, 64, 64, 0, 0),    # two heads per tile, two CTAs per unit pair
    (1, 45, 2, 128, 128, 0, 0),   # one head per tile, four CTAs per unit
    (2, 61, 12, 64, 16, 1, 1),    # the paper's multi-value layout, a full and a half tile of heads
    (1, 50, 4, 48, 32, 2, 4),     # K = 48: the second CTA has one live group
    (1, 23, 1, 16, 128, 0, 0),
    (1, 39, 3, 112, 64, 1, 3),    # odd head count at two heads per tile
    (3, 1, 2, 64, 64, 0, 0),      # a single step
    (1, 16, 1, 64, 64, 0, 0),     # exactly one stage
    (1, 48, 5, 32, 64, 5, 1),
]
W_SCALE = {GATE_VALUE: 1.0, GATE_LOGIT: 1.0, GATE_PSI: 0.5}   # see test_parity_bf16_fwd.W_SCALE


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("gate_kind", [GATE_VALUE, GATE_LOGIT, GATE_PSI])
def test_shapes_forward(oracle, shape, gate_kind):
    B, T, N, K, V, Nq, Nk = shape
    cfg = ScanConfig("case", B=B, T=T, N=N, K=K, V=V, Nq=Nq, Nk=Nk, gate_kind=gate_kind, gate_mean=1.0,
                     w_scale=W_SCALE[gate_kind], seed=200 + T)
    errs = parity.check_fwd(oracle, cfg, residual=True)
    assert max(errs.values()) < 1.5e-2


@pytest.mark.parametrize("K,V", [(16, 16), (64, 64), (128, 128)])
def test_saturating_inputs(oracle, K, V):
    cfg = ScanConfig("sat", B=2, T=96, N=2, K=K, V=V, dist="saturating", gate_mean=0.0, seed=7)
    parity.check_fwd(oracle, cfg)


def test_zero_state_and_identity_transition(oracle):
    cfg = ScanConfig("eye", B=2, T=200, N=3, K=64, V=16, Nq=1, Nk=1, dist="identity_w", h0_std=0.0, seed=8)
    parity.check_fwd(oracle, cfg)


@pytest.mark.parametrize("K,V", [(64, 64), (128, 128), (48, 32)])
def test_split_scan_and_checkpoints_are_exact(K, V):
    cfg = ScanConfig("split", B=2, T=150, N=3, K=K, V=V, seed=3)
    g = parity.to_dev(inputs.make_inputs(cfg))
    y, hT, ckpt = parity.gpu_fwd(cfg, g, save_ckpt=True)
    C = binding.m2rnn_ckpt_interval(binding._params(g["q"], g["k"], g["v"], g["W"], cfg.gate_kind))
    assert ckpt.shape[2] == (cfg.T + C - 1) // C
    assert torch.equal(ckpt[:, :, 0], g["h0"])
    cut = 3 * C
    a = {x: g[x][:, :cut].contiguous() for x in ("q", "k", "v", "gate")}
    b = {x: g[x][:, cut:].contiguous() for x in ("q", "k", "v", "gate")}
    ya, ha, _ = binding.m2rnn_fwd(a["q"], a["k"], a["v"], a["gate"], g["W"], g["h0"])
    assert torch.equal(ha, ckpt[:, :, 3])
    yb, hb, _ = binding.m2rnn_fwd(b["q"], b["k"], b["v"], b["gate"], g["W"], ha)
    assert torch.equal(torch.cat([ya, yb], dim=1), y) and torch.equal(hb, hT)
    binding.check_device_status()


def test_backward_from_this_kernels_checkpoints(oracle):
    """The checkpoints this kernel writes feed the backward pass (whose own recompute repeats the
    forward arithmetic in another kernel: equal to rounding, within the bf16 tolerance)."""
    cfg = ScanConfig("bw", B=2, T=45, N=2, K=64, V=64, gate_mean=1.0, seed=345)
    parity.check_bwd(oracle, cfg, residual=True, d_hT=True)


def test_many_units(oracle):
    cfg = ScanConfig("many", B=20, T=37, N=8, K=64, V=64, gate_mean=1.0, seed=428)   # 160 CTAs
    parity.check_fwd(oracle, cfg)
