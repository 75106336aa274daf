"""Helpers of the free-running parity tests: the fp64 oracle on single (b, n) units of a
benchmark configuration over thousands of steps, and the oracle's own sensitivity on that unit.

Why sensitivity is measured.  Eq. 1-2 with W ~ N(0, 1/V) put some heads past the edge of stability:
there a small difference in the state (the bf16 rounding of the MMA operand, say) is amplified over
hundreds of steps, by an amount that is a property of the inputs and not of the implementation.
The oracle can measure that by itself: run the unit twice, the second time from h0 + 1e-6 * noise,
and take

    A = max over sampled t of  ||H'_t - H_t||_inf / ||H'_0 - H_0||_inf.

A <= 1 means the map forgets the difference; a unit with a large A cannot be compared element by
element over a long free-running scan, whatever computes it.  Nothing here comes from the GPU.
"""
from __future__ import annotations

import concurrent.futures
import os

import numpy as np

from paper_2603_14360_b200 import inputs

SEQ = ("q", "k", "v", "gate", "dy")
EPS = 1e-6        # size of the perturbation of the initial state
A_BOUND = 2.0     # units above this amplification are reported, not asserted


def unit_inputs(cfg, d, b, n, T=None):
    """fp64 inputs of unit (b, n) over the first T steps, as one-unit tensors (B = N = 1)."""
    f = inputs.to_f64
    T = cfg.T if T is None else T
    hq, hk = n // (cfg.N // cfg.nq), n // (cfg.N // cfg.nk)
    u = dict(q=f(d["q"][b:b + 1, :T, hq:hq + 1]), k=f(d["k"][b:b + 1, :T, hk:hk + 1]),
             v=f(d["v"][b:b + 1, :T, n:n + 1]), gate=f(d["gate"][b:b + 1, :T, n:n + 1]),
             W=f(d["W"][n:n + 1]),
             h0=f(d["h0"][b:b + 1, n:n + 1]) if d.get("h0") is not None else np.zeros((1, 1, cfg.K, cfg.V)))
    if d.get("dy") is not None:
        u["dy"] = f(d["dy"][b:b + 1, :T, n:n + 1])
    return u


def oracle_unit_forward(oracle, u, h0=None, seg=256, gate_kind=1):
    """The oracle's forward scan of a unit, cut into segments chained through the final state (for
    the oracle that is exact: its split scan is pinned bit for bit), so that states along the way
    come back without storing all of them.  -> (y [T,V], {t: H_t [K,V] for t = 0, seg, 2 seg, .., T})"""
    T = u["q"].shape[1]
    state = u["h0"] if h0 is None else h0
    states = {0: state[0, 0].copy()}
    ys = []
    for s in range(0, T, seg):
        e = min(T, s + seg)
        y, state = oracle.fwd(u["q"][:, s:e], u["k"][:, s:e], u["v"][:, s:e], u["gate"][:, s:e], u["W"], state,
                              gate_kind=gate_kind)
        ys.append(y[0, :, 0])
        states[e] = state[0, 0].copy()
    return np.concatenate(ys, axis=0), states


def amplification(oracle, u, base_states, seg=256, seed=0, gate_kind=1):
    """A of the module docstring for one unit, given the unperturbed states at the segment ends."""
    rng = np.random.default_rng(seed)
    h0p = u["h0"] + EPS * rng.standard_normal(u["h0"].shape)
    _, st = oracle_unit_forward(oracle, u, h0=h0p, seg=seg, gate_kind=gate_kind)
    d0 = np.abs(st[0] - base_states[0]).max()
    return max(np.abs(st[t] - base_states[t]).max() for t in st) / d0


def run_units(fn, units, workers=None):
    """fn(unit) for every unit on a thread pool (the oracle's C loops run outside the GIL)."""
    workers = workers or max(1, min(len(units), (os.cpu_count() or 2) - 1))
    with concurrent.futures.ThreadPoolExecutor(max_workers=workers) as ex:
        return list(ex.map(fn, units))


def violations(gpu, ref, tol):
    """Count of elements with |gpu - ref| > atol + tol |ref|, atol = tol ||ref||_inf / 16: the
    element-wise companion of the infinity-norm ratio (an element is not excused by a large
    neighbour, nor condemned for being near zero)."""
    g = np.asarray(gpu, dtype=np.float64)
    atol = tol * np.abs(ref).max() / 16.0
    return int((np.abs(g - ref) > atol + tol * np.abs(ref)).sum())
