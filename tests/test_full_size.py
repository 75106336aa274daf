"""The benchmark configurations at full size, in the launch configuration the bench times.

Three kinds of check that together cover every step of the full-size launches:
  (0) free-running: the full-size launch against the fp64 oracle, element by element over the whole
      sequence (a long prefix where the oracle's T does not fit the time budget), on sampled (b, n)
      units -- units are independent, so sampling units loses nothing but time.  With W ~ N(0, 1/V)
      some heads amplify any small difference over hundreds of steps (free_running.py measures that
      with the oracle alone); the bound is asserted on every unit whose amplification stays below
      free_running.A_BOUND, and error and amplification are printed for the others;
  (1) the one-shot launch equals, bit for bit (but for dq at a window's last step), the same scan
      cut into windows that are chained through their final states (forward) and through
      dh0 -> d_hT (backward); dW, a sum over the windows, agrees to fp32 rounding;
  (2) windows of the same inputs, launched with the full batch and head count, restarted from
      states the oracle (or a seeded generator) supplies, match the oracle on sampled units.
"""
import numpy as np
import pytest
import torch

import free_running as fr
import parity
from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import CONFIGS

pytestmark = pytest.mark.gpu
TOL = 2e-2
SEQ = ("q", "k", "v", "gate", "dy")


def _window(g, s, e):
    return {x: (g[x][:, s:e].contiguous() if x in SEQ and g.get(x) is not None else g[x]) for x in g}


def _unit_f64(d, b, n, s, e):
    f = inputs.to_f64
    out = {x: f(d[x][b:b + 1, s:e, n:n + 1]) for x in SEQ if d.get(x) is not None}
    out["W"] = f(d["W"][n:n + 1])
    return out


def _bptt_full_size(oracle, name, window, oracle_len, heads_sampled):
    cfg = CONFIGS[name]
    d = inputs.make_inputs(cfg, backward=True)
    g = parity.to_dev(d)
    B, T, N = cfg.B, cfg.T, cfg.N
    y, hT, ckpt = parity.gpu_fwd(cfg, g, save_ckpt=True)
    full = parity.gpu_bwd(cfg, g, ckpt=ckpt)
    torch.cuda.synchronize()
    binding.check_device_status()
    C = binding.m2rnn_ckpt_interval(binding._params(g["q"], g["k"], g["v"], g["W"], cfg.gate_kind))
    assert window % C == 0 and T % window == 0

    # (1) chained windows == one shot
    carry, dW_sum = None, torch.zeros_like(full["dW"], dtype=torch.float64)
    state_at = lambda s: ckpt[:, :, s // C].contiguous()
    for s in range(T - window, -1, -window):
        gw = _window(g, s, s + window)
        gw["h0"], gw["d_hT"] = state_at(s), carry
        yw, hw, ck = parity.gpu_fwd(cfg, gw, save_ckpt=True)
        assert torch.equal(yw, y[:, s:s + window])
        out = parity.gpu_bwd(cfg, gw, ckpt=ck)
        for x in ("dk", "dv", "dgate"):
            assert torch.equal(out[x], full[x][:, s:s + window]), (x, s)
        # dq_t = H_t dy_t reads H_t as the bf16 tile of the step handled before; at a window's last
        # step that is the window's own recomputed final state instead of the next chunk's
        # checkpoint, which the forward kernel accumulated in another order: equal to rounding there,
        # bit for bit everywhere else
        assert torch.equal(out["dq"][:, :-1], full["dq"][:, s:s + window - 1]), ("dq", s)
        last, ref_last = out["dq"][:, -1].float(), full["dq"][:, s + window - 1].float()
        assert (last - ref_last).abs().max() <= 2e-2 * ref_last.abs().max(), ("dq last", s)
        dW_sum += out["dW"].double()
        carry = out["dh0"]
    assert torch.equal(carry, full["dh0"])
    assert parity.rel_err(full["dW"], dW_sum.cpu().numpy()) < 1e-3   # fp32 accumulation over T steps in a different order (measured: 2e-4)
    del full, y
    binding.check_device_status()

    # (2) oracle-restarted windows at the full batch and head count
    rng = np.random.default_rng(cfg.seed + 99)
    f = inputs.to_f64
    for n in heads_sampled:
        for s in sorted({0, (T // 2 // oracle_len) * oracle_len, T - oracle_len}):
            e = s + oracle_len
            gw = _window(g, s, e)
            # restart states: seeded, one per unit (any state is a valid starting point)
            h0 = torch.from_numpy(rng.normal(0, 0.3, size=(B, N, cfg.K, cfg.V)).astype(np.float32))
            dhT = torch.from_numpy(rng.normal(0, 0.1, size=(B, N, cfg.K, cfg.V)).astype(np.float32))
            gw["h0"], gw["d_hT"] = h0.cuda(), dhT.cuda()
            yw, hw, ck = parity.gpu_fwd(cfg, gw, save_ckpt=True)
            out = parity.gpu_bwd(cfg, gw, ckpt=ck)
            binding.check_device_status()
            dW_ref = 0.0
            for b in range(B):
                u = _unit_f64(d, b, n, s, e)
                h0u, dhTu = f(h0[b:b + 1, n:n + 1]), f(dhT[b:b + 1, n:n + 1])
                y_ref, hT_ref = oracle.fwd(u["q"], u["k"], u["v"], u["gate"], u["W"], h0u)
                ref = oracle.bwd(u["q"], u["k"], u["v"], u["gate"], u["W"], h0u, u["dy"], dhTu)
                assert parity.rel_err(yw[b:b + 1, :, n:n + 1], y_ref) < TOL, (n, s, b)
                assert parity.rel_err(hw[b:b + 1, n:n + 1], hT_ref) < TOL, (n, s, b)
                for x in ("dq", "dk", "dv"):
                    assert parity.rel_err(out[x][b:b + 1, :, n:n + 1], ref[x]) < TOL, (x, n, s, b)
                assert parity.rel_err(out["dgate"][b:b + 1, :, n:n + 1], ref["dgate"]) < TOL, (n, s, b)
                assert parity.rel_err(out["dh0"][b:b + 1, n:n + 1], ref["dh0"]) < TOL, (n, s, b)
                dW_ref = dW_ref + ref["dW"]
            assert parity.rel_err(out["dW"][n:n + 1], dW_ref) < TOL, (n, s)


def test_bptt_config(oracle):
    _bptt_full_size(oracle, "bptt_bf16", window=1024, oracle_len=128, heads_sampled=[5])


@pytest.mark.parametrize("name", ["sweep16", "sweep32", "sweep64", "sweep128"])
def test_state_size_sweep(oracle, name):
    _bptt_full_size(oracle, name, window=2048, oracle_len=64 if name == "sweep128" else 128, heads_sampled=[3])


def test_long_context_forward(oracle):
    cfg = CONFIGS["long_ctx"]
    d = inputs.make_inputs(cfg)
    g = parity.to_dev(d)
    y, hT, _ = parity.gpu_fwd(cfg, g)
    torch.cuda.synchronize()
    binding.check_device_status()
    # (1) chained windows == one shot
    Wn, state = 16384, g["h0"]
    for s in range(0, cfg.T, Wn):
        gw = _window(g, s, s + Wn)
        gw["h0"] = state
        yw, state, _ = parity.gpu_fwd(cfg, gw)
        assert torch.equal(yw, y[:, s:s + Wn])
    assert torch.equal(state, hT)
    # (2) oracle on windows restarted from seeded states, all 32 heads launched, 3 sampled
    rng = np.random.default_rng(cfg.seed + 99)
    f = inputs.to_f64
    L = 64
    for s in (0, 32768, cfg.T - L):
        gw = _window(g, s, s + L)
        h0 = torch.from_numpy(rng.normal(0, 0.3, size=(cfg.B, cfg.N, cfg.K, cfg.V)).astype(np.float32))
        gw["h0"] = h0.cuda()
        yw, hw, _ = parity.gpu_fwd(cfg, gw)
        binding.check_device_status()
        for n in (0, 17, 31):
            u = {x: f(d[x][:, s:s + L, n:n + 1]) for x in ("q", "k", "v", "gate")}
            y_ref, hT_ref = oracle.fwd(u["q"], u["k"], u["v"], u["gate"], f(d["W"][n:n + 1]), f(h0[:, n:n + 1]))
            assert parity.rel_err(yw[:, :, n:n + 1], y_ref) < TOL, (n, s)
            assert parity.rel_err(hw[:, n:n + 1], hT_ref) < TOL, (n, s)


def test_decode_config(oracle):
    cfg = CONFIGS["decode"]
    d = inputs.make_inputs(cfg)
    g = parity.to_dev(d)
    tok = {x: g[x][:, 0].contiguous() for x in ("q", "k", "v", "gate")}
    state = g["h0"].clone()
    y = binding.m2rnn_decode_step(tok["q"], tok["k"], tok["v"], tok["gate"], g["W"], state)
    torch.cuda.synchronize()
    binding.check_device_status()
    f = inputs.to_f64
    for (b, n) in [(0, 0), (511, 31), (100, 7), (257, 16), (3, 30)]:
        y_ref, s_ref = oracle.decode_step(f(d["q"][b:b + 1, 0, n:n + 1]), f(d["k"][b:b + 1, 0, n:n + 1]),
                                          f(d["v"][b:b + 1, 0, n:n + 1]), f(d["gate"][b:b + 1, 0, n:n + 1]),
                                          f(d["W"][n:n + 1]), f(d["h0"][b:b + 1, n:n + 1]))
        assert parity.rel_err(y[b:b + 1, n:n + 1], y_ref) < TOL, (b, n)
        assert parity.rel_err(state[b:b + 1, n:n + 1], s_ref) < TOL, (b, n)
    # units the step must not have touched differently: a second step from the same state repeats bit for bit
    state2 = g["h0"].clone()
    y2 = binding.m2rnn_decode_step(tok["q"], tok["k"], tok["v"], tok["gate"], g["W"], state2)
    assert torch.equal(y2, y) and torch.equal(state2, state)


# ------------------------------------------------------------------------------ (0) free-running
def _free_running(oracle, name, heads, batches, T_cmp, bwd):
    """Full-size launch of workload `name` (the calls and arguments of the bench) against the oracle
    on the units heads x batches over the first T_cmp steps.  Gradients are compared when bwd is set
    (then T_cmp must be the whole sequence: a gradient depends on every later step)."""
    cfg = CONFIGS[name]
    T = cfg.T
    assert not bwd or T_cmp == T
    d = inputs.make_inputs(cfg, backward=bwd)
    g = parity.to_dev(d)
    y, hT, ckpt = parity.gpu_fwd(cfg, g, save_ckpt=bwd)
    grads = parity.gpu_bwd(cfg, g, ckpt=ckpt) if bwd else {}
    torch.cuda.synchronize()
    binding.check_device_status()
    y, hT = y.cpu(), hT.cpu()
    grads = {x: t.cpu() for x, t in grads.items()}
    units = [(b, n) for n in heads for b in batches]

    def reference(bn):
        b, n = bn
        u = fr.unit_inputs(cfg, d, b, n, T_cmp)
        y_ref, states = fr.oracle_unit_forward(oracle, u)
        A = fr.amplification(oracle, u, states, seed=1000 * b + n)
        ref = dict(y=y_ref, hT=states[T_cmp] if T_cmp == T else None)
        if bwd:
            ref.update(oracle.bwd(u["q"], u["k"], u["v"], u["gate"], u["W"], u["h0"], u["dy"]))
        return A, ref

    results = fr.run_units(reference, units)
    rows, failures = [], []
    dW_ref = {n: 0.0 for n in heads}
    A_head = {n: 0.0 for n in heads}
    A_all = {n: max(A for (b_, n_), (A, _) in zip(units, results) if n_ == n) for n in heads}
    for (b, n), (A, ref) in zip(units, results):
        A_head[n] = max(A_head[n], A)
        got = dict(y=y[b, :T_cmp, n].double().numpy())
        if ref["hT"] is not None:
            got["hT"] = hT[b, n].double().numpy()
        if bwd:
            dW_ref[n] = dW_ref[n] + ref["dW"][0]
            for x in ("dq", "dk", "dv"):
                got[x] = grads[x][b, :, n].double().numpy()
                ref[x] = ref[x][0, :, 0]
            got["dgate"], ref["dgate"] = grads["dgate"][b, :, n].double().numpy(), ref["dgate"][0, :, 0]
            got["dh0"], ref["dh0"] = grads["dh0"][b, n].double().numpy(), ref["dh0"][0, 0]
        errs = {x: parity.rel_err(got[x], ref[x]) for x in got}
        viol = {x: fr.violations(got[x], ref[x], TOL) for x in got}
        rows.append(f"  unit {(b, n)}: A = {A:.3g}; " + ", ".join(f"{x} {e:.1e}/{viol[x]}" for x, e in errs.items()))
        if A <= fr.A_BOUND:
            # the forward amplification of one unit says little about its gradients when the same head
            # amplifies on other units (instability is a property of W_n): gradients go by the head
            failures += [((b, n), x, e) for x, e in errs.items() if not e <= TOL and (x in ("y", "hT") or A_all[n] <= fr.A_BOUND)]
    if bwd and len(batches) == cfg.B:      # dW[n] sums over the whole batch
        for n in heads:
            e = parity.rel_err(grads["dW"][n].double().numpy(), dW_ref[n])
            rows.append(f"  head {n}: max A = {A_head[n]:.3g}; dW {e:.1e}/{fr.violations(grads['dW'][n].double().numpy(), dW_ref[n], TOL)}")
            if A_head[n] <= fr.A_BOUND and not e <= TOL:
                failures.append((n, "dW", e))
    asserted = sum(1 for (A, _) in results if A <= fr.A_BOUND)
    print(f"\n{name}: free-running scan vs the fp64 oracle over {T_cmp} of {T} steps "
          f"(relative error in the infinity norm / elements outside atol + rtol); "
          f"{asserted} of {len(units)} units below A = {fr.A_BOUND:g} are asserted on\n" + "\n".join(rows))
    assert asserted >= (len(units) + 1) // 2, "too few units below the amplification bound to call this a parity test"
    assert not failures, failures


def test_free_running_forward_config(oracle):
    """fwd_bf16: every head once, all 2048 steps."""
    _free_running(oracle, "fwd_bf16", heads=range(16), batches=[0], T_cmp=2048, bwd=False)
    _free_running(oracle, "fwd_bf16", heads=[2, 9], batches=range(8), T_cmp=2048, bwd=False)


def test_free_running_bptt_config(oracle):
    """bptt_bf16: all 4096 steps forward and backward, the whole batch of two heads (so that dW,
    a sum over the batch, is compared too) and one unit of six more heads."""
    _free_running(oracle, "bptt_bf16", heads=[5, 17], batches=range(8), T_cmp=4096, bwd=True)
    _free_running(oracle, "bptt_bf16", heads=[0, 9, 14, 22, 27, 31], batches=[3], T_cmp=4096, bwd=True)


@pytest.mark.parametrize("name", ["sweep16", "sweep32", "sweep64", "sweep128"])
def test_free_running_state_size_sweep(oracle, name):
    """All 8192 steps forward and backward; the whole batch of one head (two below K = V = 128)."""
    _free_running(oracle, name, heads=[3] if name == "sweep128" else [3, 9], batches=range(4), T_cmp=8192, bwd=True)


def test_free_running_long_context(oracle):
    """long_ctx: the first 16384 of 65536 steps of the full-size launch on four heads (the oracle
    needs 3 ms per step of a K = V = 128 unit)."""
    _free_running(oracle, "long_ctx", heads=[0, 11, 17, 31], batches=[0], T_cmp=16384, bwd=False)
