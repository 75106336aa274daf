"""Pins for the fp64 CPU oracle: each test checks it against something the paper
or the mathematics fixes, not against itself.  No GPU needed."""
import json
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
VALUE, LOGIT, PSI = 0, 1, 2


def _rand(rng, B=2, T=6, N=2, K=3, V=4, Nq=None, Nk=None, scale=0.7):
    Nq, Nk = Nq or N, Nk or N
    return dict(q=rng.standard_normal((B, T, Nq, K)) * scale, k=rng.standard_normal((B, T, Nk, K)) * scale,
                v=rng.standard_normal((B, T, N, V)) * scale, gate=rng.standard_normal((B, T, N)),
                W=rng.standard_normal((N, V, V)) * 0.6, h0=rng.standard_normal((B, N, K, V)) * 0.5)


def _sigmoid(x):
    from scipy.special import expit
    return expit(x)


# ---------------------------------------------------------------- T = 1 by hand (Eq. 1-3)
def test_t1_by_hand(oracle):
    g = json.load(open(os.path.join(GOLDEN, "t1_by_hand.json")))
    H0 = np.array(g["H0"]); k = np.array(g["k"]); v = np.array(g["v"]); q = np.array(g["q"])
    X = 0.5 * np.array(g["X_sign"]) * np.log(np.array(g["X_log_ratio"]))
    W = np.linalg.solve(H0, X - np.outer(k, v))
    args = (q.reshape(1, 1, 1, 2), k.reshape(1, 1, 1, 2), v.reshape(1, 1, 1, 2),
            np.full((1, 1, 1), g["f"]), W.reshape(1, 2, 2), H0.reshape(1, 1, 2, 2))
    y, hT, Hs = oracle.fwd(*args, gate_kind=VALUE, return_states=True)
    np.testing.assert_allclose(hT[0, 0], np.array(g["H1"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(y[0, 0, 0], np.array(g["y"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(Hs[0, 0, 0], H0, rtol=0, atol=0)
    y2, _ = oracle.fwd(*args, gate_kind=VALUE, w_r=np.array(g["w_r"]).reshape(1, 2))
    np.testing.assert_allclose(y2[0, 0, 0], np.array(g["y_with_residual"]), rtol=0, atol=1e-14)
    # the decode entry point is the same single step
    yd, sd = oracle.decode_step(args[0][:, 0], args[1][:, 0], args[2][:, 0], args[3][:, 0], args[4],
                                args[5], gate_kind=VALUE)
    np.testing.assert_allclose(sd[0, 0], np.array(g["H1"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(yd[0, 0], np.array(g["y"]), rtol=0, atol=1e-14)


# ---------------------------------------------------------------- closed form when W = 0
def test_closed_form_w_zero(oracle):
    """With W = 0 the state is a gated running sum:
    H_t = P_t H_0 + sum_s (prod_{r>s} f_r) (1-f_s) tanh(k_s v_s^T),  P_t = prod_{r<=t} f_r."""
    rng = np.random.default_rng(1)
    d = _rand(rng, B=2, T=9, N=3, K=4, V=5)
    d["W"][:] = 0.0
    y, hT, Hs = oracle.fwd(**d, gate_kind=LOGIT, return_states=True)
    f = _sigmoid(d["gate"])                                   # [B,T,N]
    B, T, N = f.shape
    U = np.tanh(np.einsum("btni,btnj->btnij", d["k"], d["v"]))  # tanh(k v^T)
    for t in range(1, T + 1):
        # weights via cumulative products taken from the right
        tail = np.concatenate([np.cumprod(f[:, :t][:, ::-1], axis=1)[:, ::-1][:, 1:], np.ones((B, 1, N))], axis=1)
        Ht = (np.prod(f[:, :t], axis=1)[..., None, None] * d["h0"]
              + np.einsum("bsn,bsnij->bnij", tail * (1 - f[:, :t]), U[:, :t]))
        np.testing.assert_allclose(Hs[:, :, t], Ht, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(y[:, t - 1], np.einsum("bnij,bni->bnj", Ht, d["q"][:, t - 1]),
                                   rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(hT, Hs[:, :, T])


def test_trivial_gates(oracle):
    rng = np.random.default_rng(2)
    d = _rand(rng, T=5)
    # f == 1 keeps the state: y_t = H_0^T q_t, a plain matrix product
    g1 = np.ones_like(d["gate"])
    y, hT = oracle.fwd(d["q"], d["k"], d["v"], g1, d["W"], d["h0"], gate_kind=VALUE)
    np.testing.assert_allclose(hT, d["h0"], rtol=0, atol=0)
    np.testing.assert_allclose(y, np.einsum("bnij,btni->btnj", d["h0"], d["q"]), rtol=1e-13, atol=1e-14)
    # f == 0 and W == 0: y_t[j] = sum_i q_t[i] tanh(k_t[i] v_t[j]), no memory at all
    y, _ = oracle.fwd(d["q"], d["k"], d["v"], np.zeros_like(g1), np.zeros_like(d["W"]), d["h0"], gate_kind=VALUE)
    ref = np.einsum("btni,btnij->btnj", d["q"], np.tanh(np.einsum("btni,btnj->btnij", d["k"], d["v"])))
    np.testing.assert_allclose(y, ref, rtol=1e-13, atol=1e-14)


# ---------------------------------------------------------------- Theorem 1: an Elman RNN inside
def test_elman_reduction_matches_torch_rnn(oracle):
    """f=0, q=k=e_1, H_0=0  =>  y_t = tanh(y_{t-1} W + v_t): torch.nn.RNN with W_ih=I, W_hh=W^T."""
    rng = np.random.default_rng(3)
    B, T, N, K, V = 2, 12, 1, 4, 6
    v = rng.standard_normal((B, T, N, V))
    W = rng.standard_normal((N, V, V)) * 0.8
    e1 = np.zeros((B, T, N, K)); e1[..., 0] = 1.0
    y, hT, Hs = oracle.fwd(e1, e1, v, np.zeros((B, T, N)), W, None, gate_kind=VALUE, return_states=True)
    rnn = torch.nn.RNN(V, V, bias=False, batch_first=True, nonlinearity="tanh").double()
    with torch.no_grad():
        rnn.weight_ih_l0.copy_(torch.eye(V, dtype=torch.float64))
        rnn.weight_hh_l0.copy_(torch.from_numpy(W[0].T.copy()))
        ref, _ = rnn(torch.from_numpy(v[:, :, 0]))
    np.testing.assert_allclose(y[:, :, 0], ref.numpy(), rtol=1e-12, atol=1e-13)
    # rows 2..K see k_i = 0 and H_0 = 0: they stay exactly zero
    assert np.all(Hs[:, :, :, 1:, :] == 0.0)


def test_scalar_chain(oracle):
    """K=V=1 reduces to the scalar map h <- f h + (1-f) tanh(w h + k v), y = q h."""
    rng = np.random.default_rng(4)
    T = 20
    d = _rand(rng, B=1, T=T, N=1, K=1, V=1)
    y, hT = oracle.fwd(**d, gate_kind=LOGIT)
    import math
    h = float(d["h0"].ravel()[0]); w = float(d["W"].ravel()[0])
    for t in range(T):
        f = 1.0 / (1.0 + math.exp(-float(d["gate"][0, t, 0])))
        h = f * h + (1 - f) * math.tanh(w * h + float(d["k"][0, t, 0, 0]) * float(d["v"][0, t, 0, 0]))
        assert abs(y[0, t, 0, 0] - float(d["q"][0, t, 0, 0]) * h) < 1e-14
    assert abs(hT.ravel()[0] - h) < 1e-14


# ---------------------------------------------------------------- invariants
def test_state_bound(oracle):
    """|tanh| < 1 and f in [0,1]:  ||H_t||_inf <= P_t ||H_0||_inf + (1 - P_t)."""
    rng = np.random.default_rng(5)
    d = _rand(rng, B=2, T=40, N=2, K=4, V=4, scale=3.0)
    d["W"] *= 5.0
    d["h0"] *= 4.0
    y, hT, Hs = oracle.fwd(**d, gate_kind=LOGIT, return_states=True)
    P = np.cumprod(_sigmoid(d["gate"]), axis=1)               # [B,T,N]
    h0max = np.abs(d["h0"]).max(axis=(2, 3))                  # [B,N]
    for t in range(1, 41):
        bound = P[:, t - 1] * h0max + (1 - P[:, t - 1])
        assert np.all(np.abs(Hs[:, :, t]).max(axis=(2, 3)) <= bound + 1e-12)
        qn = np.abs(d["q"][:, t - 1]).sum(axis=-1)            # ||q||_1
        assert np.all(np.abs(y[:, t - 1]).max(axis=-1) <= qn * bound + 1e-12)


def test_symmetries(oracle):
    rng = np.random.default_rng(6)
    d = _rand(rng, B=3, T=7, N=2, K=3, V=4)
    y, hT = oracle.fwd(**d)
    # odd symmetry: (H0, v) -> (-H0, -v) flips H and y exactly
    y2, hT2 = oracle.fwd(d["q"], d["k"], -d["v"], d["gate"], d["W"], -d["h0"])
    assert np.array_equal(y2, -y) and np.array_equal(hT2, -hT)
    # y is linear in q, the state does not see q
    y3, hT3 = oracle.fwd(2.5 * d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"])
    np.testing.assert_allclose(y3, 2.5 * y, rtol=1e-14)
    assert np.array_equal(hT3, hT)
    # (b,n) units are independent: permuting batch permutes outputs bit for bit
    perm = np.array([2, 0, 1])
    y4, hT4 = oracle.fwd(*(d[x][perm] for x in ("q", "k", "v", "gate")), d["W"], d["h0"][perm])
    assert np.array_equal(y4, y[perm]) and np.array_equal(hT4, hT[perm])
    # heads too (W, v, gate, h0 permute together; q,k are per head here)
    hp = np.array([1, 0])
    y5, hT5 = oracle.fwd(d["q"][:, :, hp], d["k"][:, :, hp], d["v"][:, :, hp], d["gate"][:, :, hp],
                         d["W"][hp], d["h0"][:, hp])
    assert np.array_equal(y5, y[:, :, hp]) and np.array_equal(hT5, hT[:, hp])
    # rows of H are independent chains: changing row 0 of H0 and k[...,0] leaves rows 1.. alone
    d2 = {x: d[x].copy() for x in d}
    d2["h0"][:, :, 0] += 1.0
    d2["k"][..., 0] -= 0.3
    _, hT6 = oracle.fwd(**d2)
    assert np.array_equal(hT6[:, :, 1:], hT[:, :, 1:]) and not np.array_equal(hT6[:, :, 0], hT[:, :, 0])


def test_multi_value_equals_broadcast(oracle):
    """Nq=Nk=1 (multi-value) is the multi-head layout with q,k repeated; grouped layouts in between."""
    rng = np.random.default_rng(7)
    N = 4
    d = _rand(rng, B=2, T=5, N=N, K=3, V=2, Nq=1, Nk=2)
    y, hT = oracle.fwd(**d)
    qb = np.repeat(d["q"], N, axis=2)
    kb = np.repeat(d["k"], 2, axis=2)                          # head n uses k-head n // 2
    yb, hTb = oracle.fwd(qb, kb, d["v"], d["gate"], d["W"], d["h0"])
    assert np.array_equal(y, yb) and np.array_equal(hT, hTb)
    dy = rng.standard_normal(y.shape)
    g = oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], dy)
    gb = oracle.bwd(qb, kb, d["v"], d["gate"], d["W"], d["h0"], dy)
    # shared q/k gradients are the sums over the heads of the group (Algorithm 2's atomic adds)
    np.testing.assert_allclose(g["dq"][:, :, 0], gb["dq"].sum(axis=2), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(g["dk"], gb["dk"].reshape(2, 5, 2, 2, 3).sum(axis=3), rtol=1e-12, atol=1e-14)
    for name in ("dv", "dgate", "dW", "dh0"):
        np.testing.assert_allclose(g[name], gb[name], rtol=1e-12, atol=1e-14)


def test_chaining(oracle):
    rng = np.random.default_rng(8)
    d = _rand(rng, B=2, T=10, N=2, K=3, V=4)
    y, hT = oracle.fwd(**d)
    # split scan: hT of the first part seeds the second
    a = {x: d[x][:, :4] for x in ("q", "k", "v", "gate")}
    b = {x: d[x][:, 4:] for x in ("q", "k", "v", "gate")}
    ya, ha = oracle.fwd(**a, W=d["W"], h0=d["h0"])
    yb, hb = oracle.fwd(**b, W=d["W"], h0=ha)
    assert np.array_equal(np.concatenate([ya, yb], axis=1), y) and np.array_equal(hb, hT)
    # T decode steps == one scan
    s = d["h0"].copy()
    for t in range(10):
        yt, s = oracle.decode_step(d["q"][:, t], d["k"][:, t], d["v"][:, t], d["gate"][:, t], d["W"], s)
        assert np.array_equal(yt, y[:, t])
    assert np.array_equal(s, hT)
    # absent initial state means zeros
    y0, h0T = oracle.fwd(d["q"], d["k"], d["v"], d["gate"], d["W"], None)
    y0b, h0Tb = oracle.fwd(d["q"], d["k"], d["v"], d["gate"], d["W"], np.zeros_like(d["h0"]))
    assert np.array_equal(y0, y0b) and np.array_equal(h0T, h0Tb)


# ---------------------------------------------------------------- forget gate
def test_gate_modes(oracle):
    xs = np.linspace(-30, 30, 41)
    for x in xs:
        f, d = oracle.gate_fn(x, VALUE)
        assert f == x and d == 1.0
        f, d = oracle.gate_fn(x, LOGIT)
        assert abs(f - _sigmoid(x)) < 1e-15 and abs(d - _sigmoid(x) * (1 - _sigmoid(x))) < 1e-15
        # alpha = 1: the reflected, shifted sigmoid the paper points out
        f, d = oracle.gate_fn(x, PSI, 1.0, 0.7)
        assert abs(f - _sigmoid(-x - 0.7)) < 1e-15
    # general alpha against the printed formula where it is well-conditioned, derivative by differences
    for a, b in ((0.3, 0.1), (1.7, 1.2), (2.0, 0.01)):
        for x in np.linspace(-8, 8, 33):
            f, d = oracle.gate_fn(x, PSI, a, b)
            assert abs(f - (1.0 + np.exp(x + b)) ** (-a)) <= 1e-13 * max(f, 1e-300) + 1e-300
            h = 1e-5
            fd = (oracle.gate_fn(x + h, PSI, a, b)[0] - oracle.gate_fn(x - h, PSI, a, b)[0]) / (2 * h)
            assert abs(d - fd) < 1e-9
            assert 0.0 <= f <= 1.0 and d <= 0.0          # psi decreases in x
    # no overflow at the extremes
    assert oracle.gate_fn(800.0, PSI, 1.5, 0.0)[0] == 0.0
    assert oracle.gate_fn(-800.0, PSI, 1.5, 0.0)[0] == 1.0


# ---------------------------------------------------------------- gradients
def _loss(oracle, d, dy, d_hT, kw):
    y, hT = oracle.fwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], **kw)
    return float((y * dy).sum() + ((hT * d_hT).sum() if d_hT is not None else 0.0))


@pytest.mark.parametrize("gate_kind", [VALUE, LOGIT, PSI])
@pytest.mark.parametrize("shared", [False, True])
def test_bwd_matches_finite_differences(oracle, gate_kind, shared):
    rng = np.random.default_rng(10 + gate_kind + 3 * shared)
    B, T, N, K, V = 2, 5, 2, 3, 2
    d = _rand(rng, B, T, N, K, V, Nq=1 if shared else N, Nk=1 if shared else N)
    if gate_kind == VALUE:
        d["gate"] = _sigmoid(d["gate"])
    kw = dict(gate_kind=gate_kind)
    if gate_kind == PSI:
        kw.update(alpha=rng.uniform(0.5, 2, N), beta=rng.uniform(0.1, 2, N))
    kw["w_r"] = rng.standard_normal((N, V))
    dy = rng.standard_normal((B, T, N, V))
    d_hT = rng.standard_normal((B, N, K, V))
    g = oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], dy, d_hT, **kw)
    names = dict(q="dq", k="dk", v="dv", gate="dgate", W="dW", h0="dh0")
    h = 1e-6
    for x, gname in names.items():
        fd = np.zeros_like(d[x])
        it = np.nditer(d[x], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = d[x][idx]
            d[x][idx] = keep + h; lp = _loss(oracle, d, dy, d_hT, kw)
            d[x][idx] = keep - h; lm = _loss(oracle, d, dy, d_hT, kw)
            d[x][idx] = keep
            fd[idx] = (lp - lm) / (2 * h)
        err = np.abs(g[gname] - fd).max() / max(np.abs(fd).max(), 1e-12)
        assert err < 1e-7, (gname, err)


def test_bwd_matches_autograd(oracle):
    """Reverse sweep against automatic differentiation of Eq. 1-3 written in torch (fp64, CPU)."""
    rng = np.random.default_rng(20)
    B, T, N, K, V = 2, 24, 4, 16, 16
    d = _rand(rng, B, T, N, K, V, Nq=2, Nk=1, scale=0.5)
    alpha, beta = rng.uniform(0.5, 2, N), rng.uniform(0.1, 2, N)
    w_r = rng.standard_normal((N, V))
    dy = rng.standard_normal((B, T, N, V)); d_hT = rng.standard_normal((B, N, K, V))
    g = oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], dy, d_hT, gate_kind=PSI,
                   alpha=alpha, beta=beta, w_r=w_r)
    t = {x: torch.tensor(d[x], dtype=torch.float64, requires_grad=True) for x in d}
    al, be, wr = (torch.from_numpy(a) for a in (alpha, beta, w_r))
    H = t["h0"]
    qh = t["q"].repeat_interleave(N // 2, dim=2); kh = t["k"].repeat_interleave(N, dim=2)
    loss = 0.0
    for s in range(T):
        f = (1 + torch.exp(t["gate"][:, s] + be)) ** (-al)                 # forget-gate equation as printed
        Z = torch.tanh(H @ t["W"] + kh[:, s, :, :, None] * t["v"][:, s, :, None, :])
        H = f[..., None, None] * H + (1 - f[..., None, None]) * Z
        y = (H * qh[:, s, :, :, None]).sum(dim=2) + wr * t["v"][:, s]
        loss = loss + (y * torch.from_numpy(dy[:, s])).sum()
    loss = loss + (H * torch.from_numpy(d_hT)).sum()
    loss.backward()
    for x, gname in dict(q="dq", k="dk", v="dv", gate="dgate", W="dW", h0="dh0").items():
        ref = t[x].grad.numpy()
        err = np.abs(g[gname] - ref).max() / np.abs(ref).max()
        assert err < 1e-11, (gname, err)


def test_bwd_last_step_matches_algorithm2(oracle):
    """At T=1 with no incoming state gradient the printed lines of Algorithm 2 are exact:
    r = q dy^T; dq = H dy; df = sum r.(Hprev - Z); dZ = r(1-f); dX = dZ.(1 - Z.Z);
    dW = Hprev^T dX; dk = dX v; dv = dX^T k; and dH_prev = r f + dX W^T."""
    rng = np.random.default_rng(21)
    K, V = 4, 3
    d = _rand(rng, 1, 1, 1, K, V)
    f = 0.3
    dy = rng.standard_normal((1, 1, 1, V))
    g = oracle.bwd(d["q"], d["k"], d["v"], np.full((1, 1, 1), f), d["W"], d["h0"], dy, gate_kind=VALUE)
    Hp, W, q, k, v, dyv = d["h0"][0, 0], d["W"][0], d["q"][0, 0, 0], d["k"][0, 0, 0], d["v"][0, 0, 0], dy[0, 0, 0]
    Z = np.tanh(Hp @ W + np.outer(k, v)); H = f * Hp + (1 - f) * Z
    r = np.outer(q, dyv)
    dX = r * (1 - f) * (1 - Z * Z)
    np.testing.assert_allclose(g["dq"][0, 0, 0], H @ dyv, rtol=1e-13)
    np.testing.assert_allclose(g["dgate"][0, 0, 0], (r * (Hp - Z)).sum(), rtol=1e-13)
    np.testing.assert_allclose(g["dW"][0], Hp.T @ dX, rtol=1e-13)
    np.testing.assert_allclose(g["dk"][0, 0, 0], dX @ v, rtol=1e-13)
    np.testing.assert_allclose(g["dv"][0, 0, 0], dX.T @ k, rtol=1e-13)
    np.testing.assert_allclose(g["dh0"][0, 0], r * f + dX @ W.T, rtol=1e-13)


def test_bwd_state_gradient_clipping(oracle):
    rng = np.random.default_rng(22)
    d = _rand(rng, 2, 6, 2, 3, 4)
    d["W"] *= 3.0
    dy = rng.standard_normal((2, 6, 2, 4)) * 5
    base = oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], dy)
    loose = oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], dy, dh_clip=1e9)
    for n in base:
        assert np.array_equal(base[n], loose[n])
    c = 0.05
    tight = oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["W"], d["h0"], dy, dh_clip=c)
    assert np.abs(tight["dh0"]).max() <= c and np.abs(base["dh0"]).max() > c
    # the last time step sees no clipped quantity yet
    np.testing.assert_array_equal(tight["dv"][:, -1], base["dv"][:, -1])
    assert not np.array_equal(tight["dv"][:, 0], base["dv"][:, 0])


# ---------------------------------------------------------------- output path: RMSNorm(y (.) g)
def test_gated_norm_by_hand(oracle):
    """x = (3, 4, 0, 0): mean square 25/4, s = 2/5, out = w (.) x (.) s; SiLU(1) from its definition."""
    y = np.array([[[1.5, 2.0], [0.0, 7.0]]])          # one token, N = 2 heads, V = 2
    g = np.array([[[2.0, 2.0], [5.0, 0.0]]])
    w = np.array([1.0, 0.5, 3.0, 3.0])
    out, rstd = oracle.gated_norm_fwd(y, g, w, eps=0.0, silu=False)
    np.testing.assert_allclose(rstd, [0.4], rtol=0, atol=1e-15)
    np.testing.assert_allclose(out.reshape(-1), [1.2, 0.8, 0.0, 0.0], rtol=0, atol=1e-15)
    out2, rstd2 = oracle.gated_norm_fwd(y, g, w, eps=0.75, silu=False)     # 25/4 + 3/4 = 7
    np.testing.assert_allclose(rstd2, [7.0 ** -0.5], rtol=1e-15)
    # SiLU: the gate value is g / (1 + e^-g); with y = 1 the normalised vector is SiLU(g) / rms
    gin = np.array([[[1.0, -2.0]]])
    sl = np.array([1.0 / (1.0 + np.e ** -1.0), -2.0 / (1.0 + np.e ** 2.0)])
    out3, _ = oracle.gated_norm_fwd(np.ones((1, 1, 2)), gin, np.ones(2), eps=0.0, silu=True)
    np.testing.assert_allclose(out3.reshape(-1), sl / np.sqrt(np.mean(sl ** 2)), rtol=1e-14)


def test_gated_norm_invariants(oracle):
    rng = np.random.default_rng(31)
    y, g = rng.standard_normal((3, 5, 4, 6)), rng.standard_normal((3, 5, 4, 6))
    w = rng.uniform(0.5, 2.0, size=24)
    out, rstd = oracle.gated_norm_fwd(y, g, w, eps=0.0, silu=True)
    # unit root-mean-square before the weight; scale invariance in y; rstd is what it says
    np.testing.assert_allclose(np.mean((out.reshape(3, 5, 24) / w) ** 2, axis=-1), 1.0, rtol=1e-13)
    out_s, rstd_s = oracle.gated_norm_fwd(-3.0 * y, g, w, eps=0.0, silu=True)
    np.testing.assert_allclose(out_s, -out, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(rstd_s, rstd / 3.0, rtol=1e-13)
    # against torch's RMSNorm and SiLU (library routines, fp64)
    x = torch.from_numpy(y) * torch.nn.functional.silu(torch.from_numpy(g))
    ref = torch.nn.functional.rms_norm(x.reshape(3, 5, 24), (24,), torch.from_numpy(w), eps=1e-3)
    out_e, _ = oracle.gated_norm_fwd(y, g, w, eps=1e-3, silu=True)
    np.testing.assert_allclose(out_e.reshape(3, 5, 24), ref.numpy(), rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("silu", [False, True])
def test_gated_norm_bwd_matches_finite_differences(oracle, silu):
    rng = np.random.default_rng(32)
    y, g = rng.standard_normal((2, 3, 2, 4)), rng.standard_normal((2, 3, 2, 4))
    w, dout = rng.uniform(0.5, 2.0, size=8), rng.standard_normal((2, 3, 2, 4))
    eps = 0.05
    got = oracle.gated_norm_bwd(y, g, w, dout, eps=eps, silu=silu)

    def loss(y_, g_, w_):
        return float(np.sum(oracle.gated_norm_fwd(y_, g_, w_, eps=eps, silu=silu)[0] * dout))

    h = 1e-6
    for name, arr, grad in (("dy", y, got["dy"]), ("dg", g, got["dg"]), ("dw", w, got["dw"])):
        num = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            a, b = arr.copy(), arr.copy()
            a[i] += h; b[i] -= h
            args = {"dy": (a, g, w), "dg": (y, a, w), "dw": (y, g, a)}[name], {"dy": (b, g, w), "dg": (y, b, w), "dw": (y, g, b)}[name]
            num[i] = (loss(*args[0]) - loss(*args[1])) / (2 * h)
        np.testing.assert_allclose(grad, num, rtol=2e-6, atol=2e-8, err_msg=name)


def test_gated_norm_bwd_matches_autograd(oracle):
    rng = np.random.default_rng(33)
    y, g = rng.standard_normal((4, 2, 3, 8)), rng.standard_normal((4, 2, 3, 8))
    w, dout = rng.uniform(0.5, 2.0, size=24), rng.standard_normal((4, 2, 3, 8))
    ty, tg, tw = (torch.tensor(a, requires_grad=True) for a in (y, g, w))
    x = (ty * torch.nn.functional.silu(tg)).reshape(4, 2, 24)
    out = torch.nn.functional.rms_norm(x, (24,), tw, eps=1e-2)
    (out * torch.from_numpy(dout).reshape(4, 2, 24)).sum().backward()
    got = oracle.gated_norm_bwd(y, g, w, dout, eps=1e-2, silu=True)
    np.testing.assert_allclose(got["dy"], ty.grad.numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(got["dg"], tg.grad.numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(got["dw"], tw.grad.numpy(), rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- input path: SiLU(conv1d(.))
def test_conv_silu_by_hand(oracle):
    """One channel, taps (w0..w3) = (1, 10, 100, 1000) on x = (1, 2, 3, 4, 5): the current token is
    weighed by w3 and the window is causal, so pre = (1000, 2100, 3210, 4321, 5432); a bias adds
    to every step.  SiLU is checked at values where e^-x is a rational number."""
    x = np.arange(1.0, 6.0).reshape(1, 5, 1)
    w = np.array([[1.0, 10.0, 100.0, 1000.0]])
    big = oracle.conv_silu_fwd(x, w)                       # pre >= 1000: SiLU(pre) = pre to fp64
    np.testing.assert_allclose(big.reshape(-1), [1000.0, 2100.0, 3210.0, 4321.0, 5432.0], rtol=1e-15)
    prev = np.array([[[7.0], [8.0], [9.0]]])               # inputs at t = -3, -2, -1
    withprev = oracle.conv_silu_fwd(x, w, prev=prev)
    np.testing.assert_allclose(withprev.reshape(-1)[:3], [1000 + 900 + 80 + 7, 2100 + 90 + 8, 3210 + 9], rtol=1e-15)
    np.testing.assert_allclose(withprev.reshape(-1)[3:], big.reshape(-1)[3:], rtol=0)
    # SiLU(ln 3) = ln 3 / (1 + 1/3);  SiLU(-ln 3) = -ln 3 / (1 + 3)
    ln3 = np.log(3.0)
    small = oracle.conv_silu_fwd(np.array([[[1.0], [-1.0]]]), np.array([[0.0, 0.0, 0.0, ln3]]))
    np.testing.assert_allclose(small.reshape(-1), [0.75 * ln3, -0.25 * ln3], rtol=1e-15)
    withbias = oracle.conv_silu_fwd(np.zeros((1, 2, 1)), np.array([[0.0, 0.0, 0.0, 1.0]]), bias=np.array([ln3]))
    np.testing.assert_allclose(withbias.reshape(-1), [0.75 * ln3] * 2, rtol=1e-15)


def test_conv_silu_matches_torch_and_is_causal(oracle):
    rng = np.random.default_rng(61)
    B, T, C = 3, 11, 5
    x, w, bias = rng.standard_normal((B, T, C)), rng.standard_normal((C, 4)), rng.standard_normal(C)
    out = oracle.conv_silu_fwd(x, w, bias)
    # library routine: depthwise cross-correlation over time with three zeros on the left, then SiLU
    xt = torch.nn.functional.pad(torch.from_numpy(x).transpose(1, 2), (3, 0))
    ref = torch.nn.functional.silu(torch.nn.functional.conv1d(xt, torch.from_numpy(w)[:, None, :], torch.from_numpy(bias), groups=C))
    np.testing.assert_allclose(out, ref.transpose(1, 2).numpy(), rtol=1e-13, atol=1e-15)
    # causal: changing inputs after step 6 changes no output up to step 6
    x2 = x.copy()
    x2[:, 7:] += 1.0
    np.testing.assert_array_equal(oracle.conv_silu_fwd(x2, w, bias)[:, :7], out[:, :7])
    # a segment continued through `prev` equals the one-shot result
    tail = oracle.conv_silu_fwd(x[:, 6:], w, bias, prev=x[:, 3:6])
    np.testing.assert_allclose(tail, out[:, 6:], rtol=1e-14, atol=1e-16)
    # channels are independent: permuting them permutes the output
    perm = np.array([3, 0, 4, 1, 2])
    np.testing.assert_array_equal(oracle.conv_silu_fwd(x[..., perm], w[perm], bias[perm]), out[..., perm])


def test_conv_silu_bwd_matches_autograd(oracle):
    rng = np.random.default_rng(62)
    B, T, C = 2, 9, 4
    x, w, bias = rng.standard_normal((B, T, C)), rng.standard_normal((C, 4)), rng.standard_normal(C)
    prev, dout = rng.standard_normal((B, 3, C)), rng.standard_normal((B, T, C))
    got = oracle.conv_silu_bwd(x, w, dout, bias, prev)
    tx, tw, tb, tp = (torch.tensor(a, requires_grad=True) for a in (x, w, bias, prev))
    full = torch.cat([tp, tx], dim=1).transpose(1, 2)
    y = torch.nn.functional.silu(torch.nn.functional.conv1d(full, tw[:, None, :], tb, groups=C)).transpose(1, 2)
    y.backward(torch.from_numpy(dout))
    for name, t in (("dx", tx), ("dw", tw), ("dbias", tb), ("dprev", tp)):
        np.testing.assert_allclose(got[name], t.grad.numpy(), rtol=1e-12, atol=1e-14, err_msg=name)


def test_conv_silu_bwd_matches_finite_differences(oracle):
    rng = np.random.default_rng(63)
    B, T, C = 1, 6, 2
    x, w, bias = rng.standard_normal((B, T, C)), rng.standard_normal((C, 4)), rng.standard_normal(C)
    prev, dout = rng.standard_normal((B, 3, C)), rng.standard_normal((B, T, C))
    got = oracle.conv_silu_bwd(x, w, dout, bias, prev)
    loss = lambda **kw: float((oracle.conv_silu_fwd(kw.get("x", x), kw.get("w", w), kw.get("bias", bias), kw.get("prev", prev)) * dout).sum())
    eps = 1e-6
    for name, arr, key in (("dx", x, "x"), ("dw", w, "w"), ("dbias", bias, "bias"), ("dprev", prev, "prev")):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            p, m = arr.copy(), arr.copy()
            p[idx] += eps
            m[idx] -= eps
            num[idx] = (loss(**{key: p}) - loss(**{key: m})) / (2 * eps)
        np.testing.assert_allclose(got[name], num, rtol=1e-6, atol=1e-8, err_msg=name)
