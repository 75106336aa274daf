"""Packed variable-length batches (cu_seqlens) and strided q, k, v (views into one fused projection
output), forward and backward, fp32 and bf16, against the fp64 oracle."""
import numpy as np
import pytest
import torch

import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import GATE_LOGIT, GATE_PSI, ScanConfig

F = inputs.to_f64


# ------------------------------------------------------------------ CPU: the oracle's packed form
def test_oracle_packed_batch_of_equal_lengths_is_the_dense_batch(oracle):
    """The packed wrapper against the C loops' own handling of a batch: equal lengths, so the two
    layouts hold the same numbers."""
    cfg = ScanConfig("eq", B=3, T=7, N=2, K=4, V=3, Nq=1, Nk=2, dtype="f32", seed=51)
    d = inputs.make_inputs(cfg, backward=True, d_hT=True)
    a = {x: F(d[x]) for x in ("q", "k", "v", "gate", "W", "h0", "dy", "d_hT")}
    pk = lambda t: t.reshape((-1,) + t.shape[2:])
    cu = [0, 7, 14, 21]
    y, hT = oracle.fwd(a["q"], a["k"], a["v"], a["gate"], a["W"], a["h0"])
    yp, hTp = oracle.fwd_varlen(pk(a["q"]), pk(a["k"]), pk(a["v"]), pk(a["gate"]), a["W"], cu, a["h0"])
    assert np.array_equal(pk(y), yp) and np.array_equal(hT, hTp)
    r = oracle.bwd(a["q"], a["k"], a["v"], a["gate"], a["W"], a["h0"], a["dy"], a["d_hT"])
    rp = oracle.bwd_varlen(pk(a["q"]), pk(a["k"]), pk(a["v"]), pk(a["gate"]), a["W"], cu, a["h0"], pk(a["dy"]), a["d_hT"])
    for x in ("dq", "dk", "dv", "dgate"):
        assert np.array_equal(pk(r[x]), rp[x]), x
    assert np.allclose(r["dW"], rp["dW"], rtol=1e-13, atol=1e-15) and np.array_equal(r["dh0"], rp["dh0"])


def test_oracle_empty_sequence_passes_state_and_gradient_through(oracle):
    cfg = ScanConfig("e", B=1, T=5, N=1, K=2, V=2, dtype="f32", seed=52)
    d = inputs.make_inputs(cfg, backward=True, d_hT=True)
    a = {x: F(d[x]) for x in ("q", "k", "v", "gate", "W", "h0", "dy", "d_hT")}
    pk = lambda t: t.reshape((-1,) + t.shape[2:])
    h2, g2 = np.concatenate([a["h0"], 2 * a["h0"]]), np.concatenate([a["d_hT"], -a["d_hT"]])
    cu = [0, 5, 5]
    y, hT = oracle.fwd_varlen(pk(a["q"]), pk(a["k"]), pk(a["v"]), pk(a["gate"]), a["W"], cu, h2)
    assert np.array_equal(hT[1], h2[1])
    r = oracle.bwd_varlen(pk(a["q"]), pk(a["k"]), pk(a["v"]), pk(a["gate"]), a["W"], cu, h2, pk(a["dy"]), g2)
    assert np.array_equal(r["dh0"][1], g2[1])


def test_strides_are_checked_on_the_host():
    import ctypes
    from paper_2603_14360_b200 import build
    build.build()
    lib = binding._lib()
    fake = ctypes.c_void_p(0x10000)
    base = dict(B=2, T=8, N=4, Nq=4, Nk=4, K=32, V=32, io_dtype=1, gate_kind=1, ckpt_interval=0, dh_clip=0.0)
    call = lambda **kw: lib.m2rnn_fwd(ctypes.byref(binding.Params(**{**base, **kw})), *([fake] * 5), None, None, None, None,
                                      fake, None, None, None, 0, None, None)
    assert call(q_stride=64) == -2             # shorter than a token's 4 x 32 elements
    assert call(v_stride=128 + 4) == -2        # not a multiple of 16 bytes
    assert call(total_tokens=5) == -2          # only with cu_seqlens
    assert call(total_tokens=100, cu_seqlens=0x10000) == -2    # more tokens than B T


# ------------------------------------------------------------------ GPU
def _pack(d, lengths):
    """Cut a dense [B, Tmax, ...] input set down to the given lengths and pack it."""
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    out = {}
    for x, t in d.items():
        if x in ("q", "k", "v", "gate", "dy") and t is not None:
            out[x] = torch.cat([t[b, :L] for b, L in enumerate(lengths)], dim=0).contiguous()
        else:
            out[x] = t
    return out, cu


CASES = [
    # dtype, B, lengths, N, K, V, Nq, Nk, gate
    ("f32", [9, 0, 17, 1], 2, 16, 16, 0, 0, GATE_LOGIT),
    ("f32", [5, 33], 4, 32, 64, 1, 2, GATE_PSI),
    ("bf16", [37, 0, 64, 1, 16, 50], 2, 64, 64, 0, 0, GATE_LOGIT),      # column-split forward, 64-row backward
    ("bf16", [21, 40, 3], 4, 64, 16, 1, 1, GATE_LOGIT),                  # the paper's layout: one-warp-per-slab forward
    ("bf16", [19, 8], 2, 128, 128, 0, 0, GATE_LOGIT),
    ("bf16", [45, 2, 31], 3, 48, 32, 3, 1, GATE_PSI),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES, ids=lambda c: f"{c[0]}-{'_'.join(map(str, c[1]))}-K{c[3]}V{c[4]}")
@pytest.mark.parametrize("variant", ["default", "tc"])
def test_packed_batches(oracle, monkeypatch, case, variant):
    dtype, lengths, N, K, V, Nq, Nk, gate_kind = case
    if variant == "tc":
        if dtype != "bf16":
            pytest.skip("the tcgen05 kernel is a bf16 kernel")
        monkeypatch.setenv("M2RNN_FWD_VARIANT", "tc")
    tol = parity.TOL[dtype]
    cfg = ScanConfig("vl", B=len(lengths), T=max(lengths), N=N, K=K, V=V, Nq=Nq, Nk=Nk, dtype=dtype, gate_kind=gate_kind,
                     gate_mean=1.0, w_scale=0.5 if gate_kind == GATE_PSI else 1.0, seed=400 + sum(lengths))
    d, cu = _pack(inputs.make_inputs(cfg, backward=True, residual=True, d_hT=True), lengths)
    kw = dict(gate_kind=gate_kind, alpha=F(d["alpha"]), beta=F(d["beta"]), w_r=F(d["w_r"]))
    y_ref, hT_ref = oracle.fwd_varlen(F(d["q"]), F(d["k"]), F(d["v"]), F(d["gate"]), F(d["W"]), cu, F(d["h0"]), **kw)
    ref = oracle.bwd_varlen(F(d["q"]), F(d["k"]), F(d["v"]), F(d["gate"]), F(d["W"]), cu, F(d["h0"]), F(d["dy"]), F(d["d_hT"]), **kw)
    g = parity.to_dev(d)
    cu_dev = torch.from_numpy(cu).cuda()
    gk = dict(gate_kind=gate_kind, alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"], cu_seqlens=cu_dev, max_seqlen=max(lengths))
    y, hT, ckpt = binding.m2rnn_fwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], save_ckpt=True, **gk)
    assert parity.rel_err(y, y_ref) <= tol and parity.rel_err(hT, hT_ref) <= tol
    for use_ckpt in (True, False):
        out = binding.m2rnn_bwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], g["dy"], g["d_hT"],
                                ckpt=ckpt if use_ckpt else None, **gk)
        binding.check_device_status()
        for x in ref:
            assert parity.rel_err(out[x], ref[x]) <= tol, (x, use_ckpt)
    # the empty sequences' states and state gradients pass through bit for bit
    for b, L in enumerate(lengths):
        if L == 0:
            assert torch.equal(hT[b], g["h0"][b]) and torch.equal(out["dh0"][b], g["d_hT"][b])


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,K,V,N,Nq", [("f32", 32, 32, 2, 2), ("bf16", 64, 64, 2, 2), ("bf16", 64, 16, 8, 1), ("bf16", 128, 128, 1, 1)])
def test_views_into_a_fused_projection(oracle, dtype, K, V, N, Nq):
    """q, k, v as column slices of one [B, T, Nq K + Nq K + N V + pad] tensor: token stride larger
    than any of the three rows.  Same results, bit for bit, as from contiguous copies."""
    cfg = ScanConfig("st", B=2, T=29, N=N, K=K, V=V, Nq=Nq, Nk=Nq, dtype=dtype, gate_mean=1.0, seed=77)
    d = inputs.make_inputs(cfg, backward=True)
    g = parity.to_dev(d)
    wq, wv, pad = Nq * K, N * V, 24
    fused = torch.empty((cfg.B, cfg.T, 2 * wq + wv + pad), dtype=g["q"].dtype, device="cuda").normal_()
    fused[..., :wq] = g["q"].flatten(2)
    fused[..., wq:2 * wq] = g["k"].flatten(2)
    fused[..., 2 * wq:2 * wq + wv] = g["v"].flatten(2)
    qv = fused[..., :wq].unflatten(2, (Nq, K))
    kv = fused[..., wq:2 * wq].unflatten(2, (Nq, K))
    vv = fused[..., 2 * wq:2 * wq + wv].unflatten(2, (N, V))
    assert not qv.is_contiguous()
    y0, h0_, ck0 = binding.m2rnn_fwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], save_ckpt=True)
    y1, h1_, ck1 = binding.m2rnn_fwd(qv, kv, vv, g["gate"], g["W"], g["h0"], save_ckpt=True)
    assert torch.equal(y0, y1) and torch.equal(h0_, h1_) and torch.equal(ck0, ck1)
    r0 = binding.m2rnn_bwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], g["dy"], ckpt=ck0)
    r1 = binding.m2rnn_bwd(qv, kv, vv, g["gate"], g["W"], g["h0"], g["dy"], ckpt=ck1)
    binding.check_device_status()
    for x in r0:
        assert r1[x].is_contiguous() and torch.equal(r0[x], r1[x]), x
    y_ref, hT_ref = parity.oracle_fwd(oracle, cfg, d)
    assert parity.rel_err(y1, y_ref) <= parity.TOL[dtype] and parity.rel_err(h1_, hT_ref) <= parity.TOL[dtype]
