"""ctypes front end of the fp64 CPU oracle (``m2rnn_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
bench's CPU-baseline leg, never by the CUDA library's package.  Takes and
returns numpy float64 arrays in the paper's layouts (Algorithm 1/2 I/O lists):
q [B,T,Nq,K], k [B,T,Nk,K], v [B,T,N,V], gate [B,T,N], W [N,V,V],
h0 [B,N,K,V], y [B,T,N,V].
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "m2rnn_ref.c")
_LIB = os.path.join(_HERE, "libm2rnn_ref.so")

GATE_VALUE, GATE_LOGIT, GATE_PSI = 0, 1, 2


def build(force: bool = False, src: str = _SRC, out: str = _LIB) -> str:
    """Compile the oracle with gcc (IEEE semantics: no -ffast-math)."""
    hdr = os.path.join(_HERE, "m2rnn_ref.h")
    stale = (not os.path.exists(out)
             or os.path.getmtime(out) < max(os.path.getmtime(src), os.path.getmtime(hdr)))
    if force or stale:
        tmp = f"{out}.{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-I", _HERE,
                               "-o", tmp, src, "-lm"])
        os.replace(tmp, out)
    return out


def build_f32(force: bool = False) -> str:
    """Compile the fp32 build of the same loops (m2rnn_ref_f32.c) for the bench's all-cores leg."""
    src, out = os.path.join(_HERE, "m2rnn_ref_f32.c"), os.path.join(_HERE, "libm2rnn_ref_f32.so")
    deps = [src, _SRC, os.path.join(_HERE, "m2rnn_ref.h")]
    if force or not os.path.exists(out) or os.path.getmtime(out) < max(os.path.getmtime(d) for d in deps):
        tmp = f"{out}.{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-I", _HERE, "-o", tmp, src, "-lm"])
        os.replace(tmp, out)
    return out


class _Params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int), ("T", ctypes.c_int), ("N", ctypes.c_int),
                ("Nq", ctypes.c_int), ("Nk", ctypes.c_int), ("K", ctypes.c_int),
                ("V", ctypes.c_int), ("gate_kind", ctypes.c_int), ("dh_clip", ctypes.c_double)]


_dp = ctypes.POINTER(ctypes.c_double)


def load(path: str | None = None) -> ctypes.CDLL:
    lib = ctypes.CDLL(path or build())
    lib.m2rnn_ref_gate.restype = ctypes.c_double
    lib.m2rnn_ref_gate.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                   ctypes.c_double, _dp]
    lib.m2rnn_ref_fwd.restype = ctypes.c_int
    lib.m2rnn_ref_fwd.argtypes = [ctypes.POINTER(_Params)] + [_dp] * 12
    lib.m2rnn_ref_bwd.restype = ctypes.c_int
    lib.m2rnn_ref_bwd.argtypes = [ctypes.POINTER(_Params)] + [_dp] * 17
    lib.m2rnn_ref_decode_step.restype = ctypes.c_int
    lib.m2rnn_ref_decode_step.argtypes = [ctypes.POINTER(_Params)] + [_dp] * 10
    lib.m2rnn_ref_gated_norm_fwd.restype = ctypes.c_int
    lib.m2rnn_ref_gated_norm_fwd.argtypes = [ctypes.c_long, ctypes.c_int] + [_dp] * 3 + [ctypes.c_double, ctypes.c_int] + [_dp] * 2
    lib.m2rnn_ref_gated_norm_bwd.restype = ctypes.c_int
    lib.m2rnn_ref_gated_norm_bwd.argtypes = [ctypes.c_long, ctypes.c_int] + [_dp] * 3 + [ctypes.c_double, ctypes.c_int] + [_dp] * 4
    lib.m2rnn_ref_conv_silu_fwd.restype = ctypes.c_int
    lib.m2rnn_ref_conv_silu_fwd.argtypes = [ctypes.c_int] * 3 + [_dp] * 5
    lib.m2rnn_ref_conv_silu_bwd.restype = ctypes.c_int
    lib.m2rnn_ref_conv_silu_bwd.argtypes = [ctypes.c_int] * 3 + [_dp] * 9
    return lib


_lib = None


def _get():
    global _lib
    if _lib is None:
        _lib = load()
    return _lib


def _c(a, shape=None):
    """float64, C-contiguous copy-if-needed; None stays None."""
    if a is None:
        return None
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _shapes(q, k, v, W):
    B, T, Nq, K = q.shape
    Nk = k.shape[2]
    N, V = v.shape[2], v.shape[3]
    assert k.shape == (B, T, Nk, K) and v.shape == (B, T, N, V) and W.shape == (N, V, V)
    return B, T, N, Nq, Nk, K, V


def gate_fn(x, kind=GATE_LOGIT, alpha=1.0, beta=0.0, lib=None):
    """f and df/dx of one gate entry (scalar)."""
    d = ctypes.c_double(0.0)
    f = (lib or _get()).m2rnn_ref_gate(kind, float(x), float(alpha), float(beta), ctypes.byref(d))
    return f, d.value


def fwd(q, k, v, gate, W, h0=None, *, gate_kind=GATE_LOGIT, alpha=None, beta=None, w_r=None,
        return_states=False, lib=None):
    """Forward scan -> (y [B,T,N,V], hT [B,N,K,V]) (+ all states [B,N,T+1,K,V])."""
    lib = lib or _get()
    q, k, v, W = _c(q), _c(k), _c(v), _c(W)
    B, T, N, Nq, Nk, K, V = _shapes(q, k, v, W)
    gate = _c(gate, (B, T, N))
    h0 = _c(h0, (B, N, K, V)) if h0 is not None else None
    alpha, beta = _c(alpha, (N,)) if alpha is not None else None, _c(beta, (N,)) if beta is not None else None
    w_r = _c(w_r, (N, V)) if w_r is not None else None
    y = np.empty((B, T, N, V), np.float64)
    hT = np.empty((B, N, K, V), np.float64)
    H_all = np.empty((B, N, T + 1, K, V), np.float64) if return_states else None
    p = _Params(B, T, N, Nq, Nk, K, V, gate_kind, 0.0)
    rc = lib.m2rnn_ref_fwd(ctypes.byref(p), _p(q), _p(k), _p(v), _p(gate), _p(W), _p(h0),
                           _p(alpha), _p(beta), _p(w_r), _p(y), _p(hT), _p(H_all))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_fwd failed: {rc}")
    return (y, hT, H_all) if return_states else (y, hT)


def bwd(q, k, v, gate, W, h0, dy, d_hT=None, *, gate_kind=GATE_LOGIT, alpha=None, beta=None,
        w_r=None, dh_clip=0.0, lib=None):
    """Backward through time -> dict(dq, dk, dv, dgate, dW, dh0)."""
    lib = lib or _get()
    q, k, v, W = _c(q), _c(k), _c(v), _c(W)
    B, T, N, Nq, Nk, K, V = _shapes(q, k, v, W)
    gate, dy = _c(gate, (B, T, N)), _c(dy, (B, T, N, V))
    h0 = _c(h0, (B, N, K, V)) if h0 is not None else None
    d_hT = _c(d_hT, (B, N, K, V)) if d_hT is not None else None
    alpha, beta = _c(alpha, (N,)) if alpha is not None else None, _c(beta, (N,)) if beta is not None else None
    w_r = _c(w_r, (N, V)) if w_r is not None else None
    out = dict(dq=np.empty((B, T, Nq, K)), dk=np.empty((B, T, Nk, K)), dv=np.empty((B, T, N, V)),
               dgate=np.empty((B, T, N)), dW=np.empty((N, V, V)), dh0=np.empty((B, N, K, V)))
    p = _Params(B, T, N, Nq, Nk, K, V, gate_kind, float(dh_clip))
    rc = lib.m2rnn_ref_bwd(ctypes.byref(p), _p(q), _p(k), _p(v), _p(gate), _p(W), _p(h0),
                           _p(alpha), _p(beta), _p(w_r), _p(dy), _p(d_hT), _p(out["dq"]),
                           _p(out["dk"]), _p(out["dv"]), _p(out["dgate"]), _p(out["dW"]),
                           _p(out["dh0"]))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_bwd failed: {rc}")
    return out


def decode_step(q, k, v, gate, W, state, *, gate_kind=GATE_LOGIT, alpha=None, beta=None,
                w_r=None, lib=None):
    """One step on a cached state -> (y [B,N,V], new state [B,N,K,V]); inputs untouched."""
    lib = lib or _get()
    q, k, v, W = _c(q), _c(k), _c(v), _c(W)
    B, Nq, K = q.shape
    Nk, (N, V) = k.shape[1], v.shape[1:]
    gate = _c(gate, (B, N))
    state = np.array(state, dtype=np.float64, order="C", copy=True)
    assert state.shape == (B, N, K, V)
    alpha, beta = _c(alpha, (N,)) if alpha is not None else None, _c(beta, (N,)) if beta is not None else None
    w_r = _c(w_r, (N, V)) if w_r is not None else None
    y = np.empty((B, N, V), np.float64)
    p = _Params(B, 1, N, Nq, Nk, K, V, gate_kind, 0.0)
    rc = lib.m2rnn_ref_decode_step(ctypes.byref(p), _p(q), _p(k), _p(v), _p(gate), _p(W),
                                   _p(alpha), _p(beta), _p(w_r), _p(state), _p(y))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_decode_step failed: {rc}")
    return y, state


def gated_norm_fwd(y, g_in, w, *, eps=0.0, silu=True, lib=None):
    """out = RMSNorm(y * g) over the last axis flattened with the head axis: y, g_in [..., N, V],
    w [N*V] -> (out like y, rstd [...])."""
    lib = lib or _get()
    y, g_in = _c(y), _c(g_in, y.shape)
    d = y.shape[-2] * y.shape[-1]
    w = _c(np.asarray(w).reshape(-1), (d,))
    tokens = int(np.prod(y.shape[:-2]))
    out = np.empty(y.shape, np.float64)
    rstd = np.empty(y.shape[:-2], np.float64)
    rc = lib.m2rnn_ref_gated_norm_fwd(tokens, d, _p(y), _p(g_in), _p(w), float(eps), int(bool(silu)), _p(out), _p(rstd))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_gated_norm_fwd failed: {rc}")
    return out, rstd


def gated_norm_bwd(y, g_in, w, dout, *, eps=0.0, silu=True, lib=None):
    """Backward of gated_norm_fwd -> dict(dy, dg, dw [N*V])."""
    lib = lib or _get()
    y, g_in, dout = _c(y), _c(g_in, y.shape), _c(dout, y.shape)
    d = y.shape[-2] * y.shape[-1]
    w = _c(np.asarray(w).reshape(-1), (d,))
    tokens = int(np.prod(y.shape[:-2]))
    out = dict(dy=np.empty(y.shape), dg=np.empty(y.shape), dw=np.empty((d,)))
    rc = lib.m2rnn_ref_gated_norm_bwd(tokens, d, _p(y), _p(g_in), _p(w), float(eps), int(bool(silu)), _p(dout),
                                      _p(out["dy"]), _p(out["dg"]), _p(out["dw"]))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_gated_norm_bwd failed: {rc}")
    return out


def conv_silu_fwd(x, w, bias=None, prev=None, *, lib=None):
    """SiLU(depthwise causal conv1d of width 4 along time): x [B,T,C], w [C,4] (w[:,3] weighs the
    current token), bias [C], prev [B,3,C] (the three inputs before t = 0; None = zeros) -> out [B,T,C]."""
    lib = lib or _get()
    x = _c(x)
    B, T, C = x.shape
    w, bias, prev = _c(w, (C, 4)), (None if bias is None else _c(bias, (C,))), (None if prev is None else _c(prev, (B, 3, C)))
    out = np.empty((B, T, C))
    rc = lib.m2rnn_ref_conv_silu_fwd(B, T, C, _p(x), _p(w), _p(bias), _p(prev), _p(out))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_conv_silu_fwd failed: {rc}")
    return out


def conv_silu_bwd(x, w, dout, bias=None, prev=None, *, lib=None):
    """Backward of conv_silu_fwd -> dict(dx [B,T,C], dw [C,4], dbias [C], dprev [B,3,C])."""
    lib = lib or _get()
    x = _c(x)
    B, T, C = x.shape
    w, dout = _c(w, (C, 4)), _c(dout, (B, T, C))
    bias, prev = (None if bias is None else _c(bias, (C,))), (None if prev is None else _c(prev, (B, 3, C)))
    out = dict(dx=np.empty((B, T, C)), dw=np.empty((C, 4)), dbias=np.empty((C,)), dprev=np.empty((B, 3, C)))
    rc = lib.m2rnn_ref_conv_silu_bwd(B, T, C, _p(x), _p(w), _p(bias), _p(prev), _p(dout), _p(out["dx"]), _p(out["dw"]),
                                     _p(out["dbias"]), _p(out["dprev"]))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_conv_silu_bwd failed: {rc}")
    return out


# ------------------------------------------------------------------ fp32 build (bench leg only)
class _Params32(ctypes.Structure):
    _fields_ = _Params._fields_[:-1] + [("dh_clip", ctypes.c_float)]


_fp = ctypes.POINTER(ctypes.c_float)
_lib32 = None


def _get32():
    global _lib32
    if _lib32 is None:
        _lib32 = ctypes.CDLL(build_f32())
        _lib32.m2rnn_ref_fwd.restype = ctypes.c_int
        _lib32.m2rnn_ref_fwd.argtypes = [ctypes.POINTER(_Params32)] + [_fp] * 12
        _lib32.m2rnn_ref_bwd.restype = ctypes.c_int
        _lib32.m2rnn_ref_bwd.argtypes = [ctypes.POINTER(_Params32)] + [_fp] * 17
    return _lib32


def _c32(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _p32(a):
    return None if a is None else a.ctypes.data_as(_fp)


def fwd_f32(q, k, v, gate, W, h0=None, *, gate_kind=GATE_LOGIT):
    """The forward loop in its fp32 build -> (y, hT) as float32."""
    q, k, v, gate, W, h0 = (_c32(a) for a in (q, k, v, gate, W, h0))
    B, T, N, Nq, Nk, K, V = _shapes(q, k, v, W)
    y, hT = np.empty((B, T, N, V), np.float32), np.empty((B, N, K, V), np.float32)
    p = _Params32(B, T, N, Nq, Nk, K, V, gate_kind, 0.0)
    rc = _get32().m2rnn_ref_fwd(ctypes.byref(p), _p32(q), _p32(k), _p32(v), _p32(gate), _p32(W), _p32(h0),
                                None, None, None, _p32(y), _p32(hT), None)
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_fwd (fp32 build) failed: {rc}")
    return y, hT


def bwd_f32(q, k, v, gate, W, h0, dy, *, gate_kind=GATE_LOGIT):
    """The backward loop in its fp32 build -> dict(dq, dk, dv, dgate, dW, dh0) as float32."""
    q, k, v, gate, W, h0, dy = (_c32(a) for a in (q, k, v, gate, W, h0, dy))
    B, T, N, Nq, Nk, K, V = _shapes(q, k, v, W)
    out = dict(dq=np.empty((B, T, Nq, K), np.float32), dk=np.empty((B, T, Nk, K), np.float32),
               dv=np.empty((B, T, N, V), np.float32), dgate=np.empty((B, T, N), np.float32),
               dW=np.empty((N, V, V), np.float32), dh0=np.empty((B, N, K, V), np.float32))
    p = _Params32(B, T, N, Nq, Nk, K, V, gate_kind, 0.0)
    rc = _get32().m2rnn_ref_bwd(ctypes.byref(p), _p32(q), _p32(k), _p32(v), _p32(gate), _p32(W), _p32(h0),
                                None, None, None, _p32(dy), None, _p32(out["dq"]), _p32(out["dk"]),
                                _p32(out["dv"]), _p32(out["dgate"]), _p32(out["dW"]), _p32(out["dh0"]))
    if rc != 0:
        raise RuntimeError(f"m2rnn_ref_bwd (fp32 build) failed: {rc}")
    return out


# ------------------------------------------------------------------ packed variable-length batches
# A packed batch is B independent sequences laid one after the other along the token axis
# (sequence b = tokens cu_seqlens[b] .. cu_seqlens[b+1]-1).  The recurrence never couples
# sequences, so the definition is the dense scan applied to every sequence by itself; dW adds over
# sequences as it adds over batch entries.
def fwd_varlen(q, k, v, gate, W, cu_seqlens, h0=None, **kw):
    """q [tokens,Nq,K], k, v [tokens,N,V], gate [tokens,N], h0 [B,N,K,V] -> (y [tokens,N,V], hT [B,N,K,V])."""
    q, k, v, gate = (np.asarray(a, dtype=np.float64) for a in (q, k, v, gate))
    cu = [int(x) for x in cu_seqlens]
    B, N, K, V = len(cu) - 1, v.shape[1], q.shape[2], v.shape[2]
    y = np.zeros((q.shape[0], N, V))
    hT = np.zeros((B, N, K, V))
    for b in range(B):
        s, e = cu[b], cu[b + 1]
        hb = None if h0 is None else np.asarray(h0, dtype=np.float64)[b:b + 1]
        if e == s:      # an empty sequence leaves its state as it is
            hT[b] = 0.0 if hb is None else hb[0]
            continue
        yb, hTb = fwd(q[None, s:e], k[None, s:e], v[None, s:e], gate[None, s:e], W, hb, **kw)
        y[s:e], hT[b] = yb[0], hTb[0]
    return y, hT


def bwd_varlen(q, k, v, gate, W, cu_seqlens, h0, dy, d_hT=None, **kw):
    """Gradients of a packed batch: dq, dk, dv, dgate packed like their tensors, dW summed over the
    sequences, dh0 [B,N,K,V]."""
    q, k, v, gate, dy = (np.asarray(a, dtype=np.float64) for a in (q, k, v, gate, dy))
    cu = [int(x) for x in cu_seqlens]
    B, N, K, V = len(cu) - 1, v.shape[1], q.shape[2], v.shape[2]
    out = dict(dq=np.zeros(q.shape), dk=np.zeros(k.shape), dv=np.zeros(v.shape), dgate=np.zeros(gate.shape),
               dW=np.zeros((N, V, V)), dh0=np.zeros((B, N, K, V)))
    for b in range(B):
        s, e = cu[b], cu[b + 1]
        hb = None if h0 is None else np.asarray(h0, dtype=np.float64)[b:b + 1]
        db = None if d_hT is None else np.asarray(d_hT, dtype=np.float64)[b:b + 1]
        if e == s:      # no step: the state gradient passes through unchanged
            out["dh0"][b] = 0.0 if db is None else db[0]
            continue
        r = bwd(q[None, s:e], k[None, s:e], v[None, s:e], gate[None, s:e], W, hb, dy[None, s:e], db, **kw)
        for x in ("dq", "dk", "dv", "dgate"):
            out[x][s:e] = r[x][0]
        out["dW"] += r["dW"]
        out["dh0"][b] = r["dh0"][0]
    return out
