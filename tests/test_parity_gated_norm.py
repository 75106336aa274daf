"""Output path after the scan, out = RMSNorm(y (.) SiLU(g)) over the head-concatenated features, forward
and backward on the GPU against the fp64 oracle (max relative error per tensor <= 1e-4 in fp32,
<= 2e-2 in bf16; inputs are the rounded values)."""
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, T, N, V          tokens not a multiple of the 4 warps of a CTA; d = N V from 48 to 4096
    (1, 1, 3, 16),
    (2, 37, 16, 64),
    (3, 50, 84, 16),      # the paper's layer: d = 1344
    (1, 131, 32, 128),    # d = 4096: several chunks per lane
    (5, 7, 2, 32),
    (2, 700, 4, 16),      # more tokens than one pass of the grid
    (3, 41, 4, 64),       # d = 256: eight rows in flight per pass of the staged kernel
    (1, 67, 8, 64),       # d = 512
    (2, 29, 16, 128),     # d = 2048: one row per pass
    (1, 1300, 16, 64),    # d = 1024, more blocks of rows than CTAs (the ring of stages wraps)
]


def _run(oracle, shape, dtype, silu, eps):
    B, T, N, V = shape
    d = inputs.make_gated_norm_inputs(B, T, N, V, dtype, seed=500 + T)
    f = inputs.to_f64
    ref_out, ref_rstd = oracle.gated_norm_fwd(f(d["y"]), f(d["g_in"]), f(d["w"]), eps=eps, silu=silu)
    ref = oracle.gated_norm_bwd(f(d["y"]), f(d["g_in"]), f(d["w"]), f(d["dout"]), eps=eps, silu=silu)
    g = parity.to_dev(d)
    out, rstd = binding.m2rnn_gated_norm_fwd(g["y"], g["g_in"], g["w"], eps=eps, silu=silu)
    got = binding.m2rnn_gated_norm_bwd(g["y"], g["g_in"], g["w"], rstd, g["dout"], silu=silu)
    torch.cuda.synchronize()
    errs = {"out": parity.rel_err(out, ref_out), "rstd": parity.rel_err(rstd, ref_rstd),
            "dy": parity.rel_err(got["dy"], ref["dy"]), "dg": parity.rel_err(got["dg"], ref["dg"]),
            "dw": parity.rel_err(got["dw"], ref["dw"])}
    return errs


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("silu", [False, True])
def test_gated_norm_bf16(oracle, shape, silu):
    errs = _run(oracle, shape, "bf16", silu, 1e-6)
    assert max(errs.values()) < 2e-2, errs
    assert errs["rstd"] < 1e-5, errs          # fp32 statistics of exactly representable inputs


@pytest.mark.parametrize("shape", SHAPES[:4] + SHAPES[6:9], ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("silu", [False, True])
def test_gated_norm_f32(oracle, shape, silu):
    errs = _run(oracle, shape, "f32", silu, 0.0)
    assert max(errs.values()) < 1e-4, errs


def test_gated_norm_at_the_bench_size(oracle):
    """The token count and row length bench.py times (fwd_bf16's y: 16 384 tokens of 1 024 features),
    every element against the oracle."""
    errs = _run(oracle, (8, 2048, 16, 64), "bf16", True, 1e-6)
    assert max(errs.values()) < 2e-2, errs


def test_gated_norm_repeatable_and_empty():
    d = parity.to_dev(inputs.make_gated_norm_inputs(2, 300, 16, 64, "bf16", seed=9))
    out, rstd = binding.m2rnn_gated_norm_fwd(d["y"], d["g_in"], d["w"], eps=1e-6)
    a = binding.m2rnn_gated_norm_bwd(d["y"], d["g_in"], d["w"], rstd, d["dout"])
    b = binding.m2rnn_gated_norm_bwd(d["y"], d["g_in"], d["w"], rstd, d["dout"])
    assert torch.equal(a["dw"], b["dw"]) and torch.equal(a["dy"], b["dy"])      # fixed summation order
    e = {k: (v[:, :0].contiguous() if v.dim() == 4 else v) for k, v in d.items()}
    out0, rstd0 = binding.m2rnn_gated_norm_fwd(e["y"], e["g_in"], e["w"])
    got0 = binding.m2rnn_gated_norm_bwd(e["y"], e["g_in"], e["w"], rstd0, e["dout"])
    assert out0.numel() == 0 and float(got0["dw"].abs().max()) == 0.0


def test_gated_norm_rejects_bad_arguments():
    d = parity.to_dev(inputs.make_gated_norm_inputs(1, 4, 3, 4, "bf16", seed=1))     # d = 12: not a multiple of 8
    with pytest.raises(binding.M2RNNError):
        binding.m2rnn_gated_norm_fwd(d["y"], d["g_in"], d["w"])
