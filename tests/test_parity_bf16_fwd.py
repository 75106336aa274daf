"""bf16 tensor-core forward scan and decode step against the fp64 oracle
(max relative error <= 2e-2 on y and the final state; inputs are the bf16-rounded values)."""
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import CONFIGS, GATE_LOGIT, GATE_PSI, GATE_VALUE, ScanConfig

pytestmark = pytest.mark.gpu

# W ~ N(0, w_scale^2 / V).  The gate tensor and the logits keep the benchmark configurations' scale
# (w_scale 1: f ~ 0.7, a long memory).  With the psi gate at the same gate mean f ~ 0.2: the state
# is nearly Z_t alone, and Eq. 1 with W ~ N(0, 1/V) is then a chaotic map for some seeds (the
# oracle's own amplification of a 1e-6 nudge of h0 reaches 136 within 33 steps on the K = 64, V = 16
# case, against 1-5 with the other two gates), so that no two implementations agree element by
# element; w_scale 0.5 keeps those cases about the kernel's arithmetic.
W_SCALE = {GATE_VALUE: 1.0, GATE_LOGIT: 1.0, GATE_PSI: 0.5}

SHAPES = [
    # B, T, N, K, V, Nq, Nk       T spans several pipeline stages and a ragged tail
    (2, 100, 3, 16, 16, 0, 0),
    (1, 77, 2, 32, 32, 0, 0),
    (2, 131, 2, 64, 64, 0, 0),
    (1, 45, 2, 128, 128, 0, 0),
    (2, 61, 4, 64, 16, 1, 1),     # the paper's K=64, V=16 multi-value layout
    (1, 50, 4, 48, 32, 2, 4),
    (1, 23, 1, 16, 128, 0, 0),
    (1, 39, 2, 112, 64, 1, 2),
    (3, 1, 2, 64, 64, 0, 0),      # a single step
    (1, 16, 1, 64, 64, 0, 0),     # exactly one stage
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("gate_kind", [GATE_VALUE, GATE_LOGIT, GATE_PSI])
def test_shapes_forward(oracle, shape, gate_kind):
    B, T, N, K, V, Nq, Nk = shape
    cfg = ScanConfig("case", B=B, T=T, N=N, K=K, V=V, Nq=Nq, Nk=Nk, gate_kind=gate_kind, gate_mean=1.0,
                     w_scale=W_SCALE[gate_kind], seed=200 + T)
    errs = parity.check_fwd(oracle, cfg, residual=True)
    assert max(errs.values()) < 1.5e-2        # typical error is a few 1e-3: bf16 rounding of H, tanh.approx


@pytest.mark.parametrize("K,V", [(32, 32), (48, 32), (64, 32), (32, 64), (48, 64), (64, 64), (32, 128), (96, 64), (64, 16)])
def test_more_units_than_sms(oracle, K, V):
    """152 (b, n) units: every CTA keeps a whole state (two to four 16-row slabs per CTA in the
    column-split kernel, six in the one-warp-per-slab kernel), the launch takes two waves."""
    B = 80 if V == 16 else 38          # V = 16: more than 296 units, three CTAs per SM
    cfg = ScanConfig("many", B=B, T=37, N=4, K=K, V=V, gate_mean=1.0, seed=300 + K + V)
    errs = parity.check_fwd(oracle, cfg)
    assert max(errs.values()) < 1.5e-2


@pytest.mark.parametrize("K,V", [(16, 16), (64, 64), (128, 128)])
def test_saturating_inputs(oracle, K, V):
    cfg = ScanConfig("sat", B=2, T=96, N=2, K=K, V=V, dist="saturating", gate_mean=0.0, seed=7)
    parity.check_fwd(oracle, cfg)


def test_identity_transition_and_zero_state(oracle):
    cfg = ScanConfig("eye", B=2, T=200, N=3, K=64, V=16, Nq=1, Nk=1, dist="identity_w", h0_std=0.0, seed=8)
    parity.check_fwd(oracle, cfg)


def test_split_scan_and_checkpoints_are_exact():
    """The state is fp32 end to end, so resuming from hT (or from a checkpoint) repeats the
    one-shot scan bit for bit; checkpoints hold the state before steps 0, C, 2C, ..."""
    cfg = ScanConfig("split", B=2, T=150, N=2, K=64, V=64, seed=3)
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


def test_decode_step(oracle):
    cfg = ScanConfig("dec", B=5, T=6, N=4, K=128, V=128, Nq=1, Nk=2, gate_kind=GATE_PSI, seed=5)
    d = inputs.make_inputs(cfg, residual=True)
    g = parity.to_dev(d)
    f = inputs.to_f64
    state = g["h0"].clone()
    ref_state = f(d["h0"])
    for t in range(cfg.T):
        y_ref, ref_state = oracle.decode_step(f(d["q"][:, t]), f(d["k"][:, t]), f(d["v"][:, t]), f(d["gate"][:, t]),
                                              f(d["W"]), ref_state, gate_kind=cfg.gate_kind, alpha=f(d["alpha"]),
                                              beta=f(d["beta"]), w_r=f(d["w_r"]))
        yt = binding.m2rnn_decode_step(g["q"][:, t].contiguous(), g["k"][:, t].contiguous(), g["v"][:, t].contiguous(),
                                       g["gate"][:, t].contiguous(), g["W"], state, gate_kind=cfg.gate_kind,
                                       alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"])
        assert parity.rel_err(yt, y_ref) < 2e-2 and parity.rel_err(state, ref_state) < 2e-2
    binding.check_device_status()


def test_units_are_independent():
    """(b,n) units never interact: permuting the batch permutes the outputs bit for bit."""
    cfg = ScanConfig("perm", B=4, T=40, N=2, K=32, V=64, seed=12)
    g = parity.to_dev(inputs.make_inputs(cfg))
    y, hT, _ = parity.gpu_fwd(cfg, g)
    perm = torch.tensor([2, 0, 3, 1], device="cuda")
    gp = {x: (g[x][perm].contiguous() if x in ("q", "k", "v", "gate", "h0") else g[x]) for x in g}
    yp, hTp, _ = parity.gpu_fwd(cfg, gp)
    assert torch.equal(yp, y[perm]) and torch.equal(hTp, hT[perm])


def _windows(T, width):
    starts = sorted({0, (T // 2 // width) * width, max(0, T - width - 37)})
    return [(s, min(T, s + width)) for s in starts]


@pytest.mark.parametrize("name", ["fwd_bf16"])
def test_full_size_forward(oracle, name):
    """The benchmark configuration at full size, in the launch configuration the bench times, cut
    into windows (the free-running comparison over all 2048 steps is in test_full_size.py):
    (1) windows of 256 steps restarted from the ORACLE's state must match the oracle within 2e-2 on
    every sampled unit, also on the heads that amplify a difference over a long scan; (2) the
    one-shot full scan must equal, bit for bit, the same windows chained through their own final
    states.
    """
    cfg = CONFIGS[name]
    d = inputs.make_inputs(cfg)
    g = parity.to_dev(d)
    y, hT, _ = parity.gpu_fwd(cfg, g)
    torch.cuda.synchronize()
    binding.check_device_status()
    # (2) chained windows == one shot
    W = 512
    state = g["h0"]
    for s in range(0, cfg.T, W):
        part = {x: g[x][:, s:s + W].contiguous() for x in ("q", "k", "v", "gate")}
        yw, state, _ = binding.m2rnn_fwd(part["q"], part["k"], part["v"], part["gate"], g["W"], state)
        assert torch.equal(yw, y[:, s:s + W])
    assert torch.equal(state, hT)
    # (1) oracle-restarted windows on a seeded subset of (b,n) units (all units are independent)
    f = inputs.to_f64
    units = [(0, 0), (cfg.B - 1, cfg.N - 1), (3, 5)]
    for (b, n) in units:
        sel = lambda t, head=True: f(t[b:b + 1, :, n:n + 1] if head else t[b:b + 1])
        q, k, v, gate = sel(d["q"]), sel(d["k"]), sel(d["v"]), sel(d["gate"])
        Wn, h0 = f(d["W"][n:n + 1]), f(d["h0"][b:b + 1, n:n + 1])
        y_ref, hT_ref, Hs = oracle.fwd(q, k, v, gate, Wn, h0, return_states=True)
        # free-running error over the first 256 steps
        assert parity.rel_err(y[b:b + 1, :256, n:n + 1], y_ref[:, :256]) < 2e-2
        for (s, e) in _windows(cfg.T, 256):
            start = torch.from_numpy(Hs[:, :, s]).float().cuda()
            yw, hw, _ = binding.m2rnn_fwd(*(torch.from_numpy(x[:, s:e]).to(torch.bfloat16).cuda().contiguous() for x in (q, k, v)),
                                          torch.from_numpy(gate[:, s:e]).float().cuda().contiguous(),
                                          g["W"][n:n + 1].contiguous(), start)
            assert parity.rel_err(yw, y_ref[:, s:e]) < 2e-2, (b, n, s)
            assert parity.rel_err(hw, Hs[:, :, e]) < 2e-2, (b, n, s)
