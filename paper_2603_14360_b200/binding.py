"""Thin ctypes binding of ``libm2rnn.so`` (declared in ``include/m2rnn.h``).

Argument marshalling only: every step of the scan runs in the library's CUDA kernels.
torch supplies device memory and the current stream; there is no CPU or eager fallback --
a missing or stale library raises.

    y, hT, ckpt = m2rnn_fwd(q, k, v, gate, W, h0, save_ckpt=True)
    grads       = m2rnn_bwd(q, k, v, gate, W, h0, dy, ckpt=ckpt)
    y1          = m2rnn_decode_step(q1, k1, v1, gate1, W, state)      # state updated in place
    out, rstd   = m2rnn_gated_norm_fwd(y, g_in, w)                    # RMSNorm(y * SiLU(g)) over N*V
    grads       = m2rnn_gated_norm_bwd(y, g_in, w, rstd, dout)        # dy, dg, dw

Tensor layouts are the paper's (Algorithm 1/2): q [B,T,Nq,K], k [B,T,Nk,K], v [B,T,N,V],
gate [B,T,N] fp32, W [N,V,V], h0 [B,N,K,V] fp32.
"""
from __future__ import annotations

import ctypes
import os

import torch

GATE_VALUE, GATE_LOGIT, GATE_PSI = 0, 1, 2
F32, BF16 = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libm2rnn.so")

STATUS = {0: "M2RNN_OK", -1: "M2RNN_ERR_NULL", -2: "M2RNN_ERR_SHAPE", -3: "M2RNN_ERR_UNSUPPORTED",
          -4: "M2RNN_ERR_ALIGN", -5: "M2RNN_ERR_WORKSPACE", -6: "M2RNN_ERR_CUDA", -7: "M2RNN_ERR_TIMEOUT"}


class M2RNNError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().m2rnn_status_string(status).decode() if _LIB is not None else ""
        super().__init__(f"{where}: {STATUS.get(status, status)} ({msg})")


class Params(ctypes.Structure):
    """Mirror of ``m2rnn_params``."""
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("N", ctypes.c_int32),
                ("Nq", ctypes.c_int32), ("Nk", ctypes.c_int32), ("K", ctypes.c_int32),
                ("V", ctypes.c_int32), ("io_dtype", ctypes.c_int32), ("gate_kind", ctypes.c_int32),
                ("ckpt_interval", ctypes.c_int32), ("dh_clip", ctypes.c_float),
                ("q_stride", ctypes.c_int64), ("k_stride", ctypes.c_int64), ("v_stride", ctypes.c_int64),
                ("total_tokens", ctypes.c_int64), ("cu_seqlens", ctypes.c_void_p)]


_LIB = None
_vp = ctypes.c_void_p
_pp = ctypes.POINTER(Params)

EXPORTS = {
    "m2rnn_version": (ctypes.c_int, []),
    "m2rnn_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "m2rnn_ckpt_interval": (ctypes.c_int, [_pp]),
    "m2rnn_bwd_row_slab": (ctypes.c_int, [_pp]),
    "m2rnn_ckpt_bytes": (ctypes.c_size_t, [_pp]),
    "m2rnn_fwd_workspace_bytes": (ctypes.c_size_t, [_pp]),
    "m2rnn_fwd": (ctypes.c_int, [_pp] + [_vp] * 13 + [ctypes.c_size_t, _vp, _vp]),
    "m2rnn_bwd_workspace_bytes": (ctypes.c_size_t, [_pp, ctypes.c_int]),
    "m2rnn_bwd": (ctypes.c_int, [_pp] + [_vp] * 19 + [ctypes.c_size_t, _vp, _vp]),
    "m2rnn_bwd_static_scratch": (ctypes.c_int, [_pp] + [_vp] * 20),
    "m2rnn_decode_step": (ctypes.c_int, [_pp] + [_vp] * 12),
    "m2rnn_conv_silu_fwd": (ctypes.c_int, [ctypes.c_int32] * 4 + [_vp, ctypes.c_int64, _vp, _vp, _vp, _vp, ctypes.c_int64, _vp]),
    "m2rnn_conv_silu_bwd_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int32] * 3),
    "m2rnn_conv_silu_bwd": (ctypes.c_int, [ctypes.c_int32] * 4 + [_vp, ctypes.c_int64, _vp, _vp, _vp, _vp, ctypes.c_int64, _vp,
                                             ctypes.c_int64, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]),
    "m2rnn_wait_selftest": (ctypes.c_int, [ctypes.c_int64, _vp, _vp, _vp]),
    "m2rnn_gated_norm_fwd": (ctypes.c_int, [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, _vp, _vp, _vp, ctypes.c_float,
                                            ctypes.c_int32, _vp, _vp, _vp]),
    "m2rnn_gated_norm_bwd_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int64, ctypes.c_int32]),
    "m2rnn_gated_norm_bwd": (ctypes.c_int, [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, _vp, _vp, _vp, _vp, ctypes.c_int32,
                                            _vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]),
}

STATIC_SCRATCH_BYTES = 8 << 20   # M2RNN_STATIC_SCRATCH_BYTES


def _lib() -> ctypes.CDLL:
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is not built: run `python -m paper_2603_14360_b200.build` "
                              "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)          # AttributeError if the library is stale
            fn.restype, fn.argtypes = res, args
        _LIB = lib
    return _LIB


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _io_code(dtype: torch.dtype) -> int:
    if dtype == torch.float32:
        return F32
    if dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported I/O dtype {dtype}")


def _chk(t, name, shape, dtype, strided_tokens=False):
    if t is None:
        return
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous() and not strided_tokens:     # (q, k, v: _token_stride checks the layout)
        raise ValueError(f"{name} must be contiguous")


_status_words: dict[int, torch.Tensor] = {}


def device_status_word(device=None) -> torch.Tensor:
    """The int32 word kernels raise when a bounded wait runs out (one per device, zero = fine)."""
    idx = torch.cuda.current_device() if device is None else torch.device(device).index
    if idx not in _status_words:
        _status_words[idx] = torch.zeros(1, dtype=torch.int32, device=f"cuda:{idx}")
    return _status_words[idx]


def check_device_status(device=None) -> None:
    """Synchronises and raises if any kernel since the last check reported a timeout."""
    w = device_status_word(device)
    v = int(w.item())
    if v != 0:
        w.zero_()
        raise M2RNNError(v, "device status")


def m2rnn_wait_selftest(limit_cycles: int, device=None, stream=None):
    """Launches the library's wait self-test: one warp waits, with a limit of ``limit_cycles`` SM
    clocks, on a barrier nothing completes.  Returns (status word as the kernel left it, SM clocks
    the wait took); the status must be M2RNN_ERR_TIMEOUT (-7).  Uses words of its own, not the
    device status word of the scan calls."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    waited = torch.zeros(1, dtype=torch.int64, device=dev)
    rc = _lib().m2rnn_wait_selftest(int(limit_cycles), _ptr(status), _ptr(waited), _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_wait_selftest")
    return int(status.item()), int(waited.item())


def _token_stride(t, name) -> int:
    """Elements between consecutive tokens of q, k or v ([B,T,heads,dim] or packed [tokens,heads,dim]).
    A token's heads must be contiguous and the token axis regular, so that the tensor may be a view
    into a fused projection output; 0 stands for the dense layout."""
    if t.numel() == 0:
        return 0
    if t.stride(-1) != 1 or t.stride(-2) != t.shape[-1]:
        raise ValueError(f"{name}: the heads of a token must be contiguous")
    tok = t.stride(-3)
    if t.dim() == 4 and t.shape[0] > 1 and t.stride(0) != t.shape[1] * tok:
        raise ValueError(f"{name}: batch entries must follow one another along the token axis")
    return 0 if tok == t.shape[-2] * t.shape[-1] else tok


def _params(q, k, v, W, gate_kind, ckpt_interval=0, dh_clip=0.0, decode=False, cu_seqlens=None,
            max_seqlen=None) -> Params:
    if decode:
        B, Nq, K = q.shape
        T, Nk, (N, V) = 1, k.shape[1], v.shape[1:]
        return Params(B, T, N, Nq, Nk, K, V, _io_code(q.dtype), gate_kind, ckpt_interval, dh_clip, 0, 0, 0, 0, None)
    if cu_seqlens is not None:   # packed variable-length batch: q [tokens, Nq, K]
        if cu_seqlens.dtype != torch.int32 or not cu_seqlens.is_cuda or not cu_seqlens.is_contiguous():
            raise TypeError("cu_seqlens must be a contiguous int32 CUDA tensor of B + 1 offsets")
        if max_seqlen is None:
            raise ValueError("max_seqlen (the longest sequence) is required with cu_seqlens")
        total, Nq, K = q.shape
        B, T, Nk, (N, V) = cu_seqlens.numel() - 1, int(max_seqlen), k.shape[1], v.shape[1:]
    else:
        B, T, Nq, K = q.shape
        total, Nk, (N, V) = 0, k.shape[2], v.shape[2:]
    return Params(B, T, N, Nq, Nk, K, V, _io_code(q.dtype), gate_kind, ckpt_interval, dh_clip,
                  _token_stride(q, "q"), _token_stride(k, "k"), _token_stride(v, "v"), total,
                  None if cu_seqlens is None else cu_seqlens.data_ptr())


def m2rnn_version() -> int:
    return _lib().m2rnn_version()


def m2rnn_ckpt_interval(p: Params) -> int:
    c = _lib().m2rnn_ckpt_interval(ctypes.byref(p))
    if c <= 0:
        raise M2RNNError(c, "m2rnn_ckpt_interval")
    return c


def m2rnn_bwd_row_slab(p: Params) -> int:
    r = _lib().m2rnn_bwd_row_slab(ctypes.byref(p))
    if r <= 0:
        raise M2RNNError(r, "m2rnn_bwd_row_slab")
    return r


def m2rnn_bwd_workspace_bytes(p: Params, have_ckpt: bool) -> int:
    return _lib().m2rnn_bwd_workspace_bytes(ctypes.byref(p), int(have_ckpt))


def m2rnn_fwd_workspace_bytes(p: Params) -> int:
    return _lib().m2rnn_fwd_workspace_bytes(ctypes.byref(p))


def m2rnn_fwd(q, k, v, gate, W, h0=None, *, gate_kind=GATE_LOGIT, alpha=None, beta=None, w_r=None,
              save_ckpt=False, ckpt_interval=0, want_hT=True, out=None, workspace=None, stream=None,
              cu_seqlens=None, max_seqlen=None):
    """Forward scan.  Returns (y, hT, ckpt); hT / ckpt are None when not requested.
    ``out`` may hold preallocated ``y`` / ``hT`` / ``ckpt`` tensors to write into; ``workspace``
    a preallocated uint8 tensor of at least ``m2rnn_fwd_workspace_bytes`` bytes.
    q, k, v may be strided views along the token axis (e.g. slices of one fused projection output).
    With ``cu_seqlens`` (int32 [B+1], CUDA) and ``max_seqlen`` the batch is packed: q [tokens,Nq,K],
    k, v, gate [tokens,N], y [tokens,N,V]; states stay [B,N,K,V]."""
    p = _params(q, k, v, W, gate_kind, ckpt_interval, cu_seqlens=cu_seqlens, max_seqlen=max_seqlen)
    B, T, N, K, V, io = p.B, p.T, p.N, p.K, p.V, q.dtype
    lead = (B, T) if cu_seqlens is None else (q.shape[0],)
    _chk(q, "q", (*lead, p.Nq, K), io, True); _chk(k, "k", (*lead, p.Nk, K), io, True); _chk(v, "v", (*lead, N, V), io, True)
    _chk(gate, "gate", (*lead, N), torch.float32); _chk(W, "W", (N, V, V), io)
    _chk(h0, "h0", (B, N, K, V), torch.float32); _chk(w_r, "w_r", (N, V), io)
    _chk(alpha, "alpha", (N,), torch.float32); _chk(beta, "beta", (N,), torch.float32)
    out = out or {}
    y = out.get("y")
    if y is None:
        y = torch.empty((*lead, N, V), dtype=io, device=q.device)
    hT = out.get("hT")
    if hT is None and want_hT:
        hT = torch.empty((B, N, K, V), dtype=torch.float32, device=q.device)
    ckpt = out.get("ckpt")
    if ckpt is None and save_ckpt:
        C = m2rnn_ckpt_interval(p)
        ckpt = torch.empty((B, N, (T + C - 1) // C, K, V), dtype=torch.float32, device=q.device)
    _chk(y, "y", (*lead, N, V), io); _chk(hT, "hT", (B, N, K, V), torch.float32)
    need = m2rnn_fwd_workspace_bytes(p)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    rc = _lib().m2rnn_fwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(W), _ptr(h0),
                          _ptr(alpha), _ptr(beta), _ptr(w_r), _ptr(y), _ptr(hT), _ptr(ckpt),
                          _ptr(workspace), 0 if workspace is None else workspace.numel(),
                          _ptr(device_status_word(q.device)), _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_fwd")
    return y, hT, ckpt


def m2rnn_bwd(q, k, v, gate, W, h0, dy, d_hT=None, *, ckpt=None, gate_kind=GATE_LOGIT, alpha=None,
              beta=None, w_r=None, ckpt_interval=0, dh_clip=0.0, want_dh0=True, workspace=None,
              out=None, stream=None, cu_seqlens=None, max_seqlen=None):
    """Backward through time.  Returns dict(dq, dk, dv, dgate, dW, dh0) (dense, whatever the strides
    of q, k, v).  ``cu_seqlens`` / ``max_seqlen``: packed batch, as in ``m2rnn_fwd``."""
    p = _params(q, k, v, W, gate_kind, ckpt_interval, dh_clip, cu_seqlens=cu_seqlens, max_seqlen=max_seqlen)
    B, T, N, K, V, io = p.B, p.T, p.N, p.K, p.V, q.dtype
    lead = (B, T) if cu_seqlens is None else (q.shape[0],)
    _chk(q, "q", (*lead, p.Nq, K), io, True); _chk(k, "k", (*lead, p.Nk, K), io, True); _chk(v, "v", (*lead, N, V), io, True)
    _chk(gate, "gate", (*lead, N), torch.float32); _chk(W, "W", (N, V, V), io)
    _chk(h0, "h0", (B, N, K, V), torch.float32); _chk(w_r, "w_r", (N, V), io)
    _chk(alpha, "alpha", (N,), torch.float32); _chk(beta, "beta", (N,), torch.float32)
    _chk(dy, "dy", (*lead, N, V), io); _chk(d_hT, "d_hT", (B, N, K, V), torch.float32)
    if ckpt is not None and T > 0:
        C = m2rnn_ckpt_interval(p)
        _chk(ckpt, "ckpt", (B, N, (T + C - 1) // C, K, V), torch.float32)
    dev = q.device
    out = out or {}
    g = dict(dq=out.get("dq"), dk=out.get("dk"), dv=out.get("dv"), dgate=out.get("dgate"),
             dW=out.get("dW"), dh0=out.get("dh0"))
    if g["dq"] is None: g["dq"] = torch.empty(q.shape, dtype=io, device=dev)
    if g["dk"] is None: g["dk"] = torch.empty(k.shape, dtype=io, device=dev)
    if g["dv"] is None: g["dv"] = torch.empty(v.shape, dtype=io, device=dev)
    if g["dgate"] is None: g["dgate"] = torch.empty_like(gate)
    if g["dW"] is None: g["dW"] = torch.empty((N, V, V), dtype=torch.float32, device=dev)
    if g["dh0"] is None and want_dh0: g["dh0"] = torch.empty((B, N, K, V), dtype=torch.float32, device=dev)
    for x in ("dq", "dk", "dv"):
        _chk(g[x], x, {"dq": q, "dk": k, "dv": v}[x].shape, io)
    need = m2rnn_bwd_workspace_bytes(p, ckpt is not None)
    if workspace is None:
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=dev)
    rc = _lib().m2rnn_bwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(W), _ptr(h0),
                          _ptr(alpha), _ptr(beta), _ptr(w_r), _ptr(ckpt), _ptr(dy), _ptr(d_hT),
                          _ptr(g["dq"]), _ptr(g["dk"]), _ptr(g["dv"]), _ptr(g["dgate"]), _ptr(g["dW"]),
                          _ptr(g["dh0"]), _ptr(workspace), workspace.numel(),
                          _ptr(device_status_word(dev)), _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_bwd")
    return g


def m2rnn_bwd_static_scratch(q, k, v, gate, W, h0, dy, d_hT=None, *, out, ckpt=None, gate_kind=GATE_LOGIT,
                             alpha=None, beta=None, w_r=None, ckpt_interval=0, dh_clip=0.0, stream=None):
    """Backward through time on the library's built-in scratch array, for callers that must not
    allocate device memory (an embedding application that owns the allocator, a service that
    forbids allocation after start-up).  Nothing is allocated here either: ``out`` must already
    hold ``dq, dk, dv, dgate, dW`` (and ``dh0`` if wanted), which are written in place and
    returned.  Problems that need more than ``STATIC_SCRATCH_BYTES`` of scratch raise
    ``M2RNNError`` with ``M2RNN_ERR_WORKSPACE``; calls must not overlap on the GPU, because they
    all share the one array."""
    p = _params(q, k, v, W, gate_kind, ckpt_interval, dh_clip)
    B, T, N, K, V, io = p.B, p.T, p.N, p.K, p.V, q.dtype
    _chk(q, "q", (B, T, p.Nq, K), io); _chk(k, "k", (B, T, p.Nk, K), io); _chk(v, "v", (B, T, N, V), io)
    _chk(gate, "gate", (B, T, N), torch.float32); _chk(W, "W", (N, V, V), io)
    _chk(h0, "h0", (B, N, K, V), torch.float32); _chk(w_r, "w_r", (N, V), io)
    _chk(alpha, "alpha", (N,), torch.float32); _chk(beta, "beta", (N,), torch.float32)
    _chk(dy, "dy", (B, T, N, V), io); _chk(d_hT, "d_hT", (B, N, K, V), torch.float32)
    _chk(out["dq"], "dq", q.shape, io); _chk(out["dk"], "dk", k.shape, io); _chk(out["dv"], "dv", v.shape, io)
    _chk(out["dgate"], "dgate", gate.shape, torch.float32); _chk(out["dW"], "dW", (N, V, V), torch.float32)
    _chk(out.get("dh0"), "dh0", (B, N, K, V), torch.float32)
    rc = _lib().m2rnn_bwd_static_scratch(
        ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(W), _ptr(h0), _ptr(alpha), _ptr(beta),
        _ptr(w_r), _ptr(ckpt), _ptr(dy), _ptr(d_hT), _ptr(out["dq"]), _ptr(out["dk"]), _ptr(out["dv"]),
        _ptr(out["dgate"]), _ptr(out["dW"]), _ptr(out.get("dh0")), _ptr(device_status_word(q.device)),
        _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_bwd_static_scratch")
    return out


def m2rnn_decode_step(q, k, v, gate, W, state, *, gate_kind=GATE_LOGIT, alpha=None, beta=None,
                      w_r=None, y=None, stream=None):
    """One decoding step; ``state`` [B,N,K,V] fp32 is updated in place.  Returns y [B,N,V]."""
    p = _params(q, k, v, W, gate_kind, decode=True)
    B, N, K, V, io = p.B, p.N, p.K, p.V, q.dtype
    _chk(q, "q", (B, p.Nq, K), io); _chk(k, "k", (B, p.Nk, K), io); _chk(v, "v", (B, N, V), io)
    _chk(gate, "gate", (B, N), torch.float32); _chk(W, "W", (N, V, V), io)
    _chk(state, "state", (B, N, K, V), torch.float32); _chk(w_r, "w_r", (N, V), io)
    _chk(alpha, "alpha", (N,), torch.float32); _chk(beta, "beta", (N,), torch.float32)
    if y is None:
        y = torch.empty((B, N, V), dtype=io, device=q.device)
    _chk(y, "y", (B, N, V), io)
    rc = _lib().m2rnn_decode_step(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(W),
                                  _ptr(alpha), _ptr(beta), _ptr(w_r), _ptr(state), _ptr(y),
                                  _ptr(device_status_word(q.device)), _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_decode_step")
    return y


def _norm_dims(y):
    if y.dim() < 2:
        raise ValueError("y needs at least the two trailing axes [N, V]")
    d = y.shape[-2] * y.shape[-1]
    tokens = y.numel() // d if d else 0
    return tokens, d


def m2rnn_gated_norm_fwd(y, g_in, w, *, eps=0.0, silu=True, out=None, rstd=None, stream=None):
    """out = RMSNorm(y * SiLU(g_in)) over the head-concatenated features: y, g_in [..., N, V],
    w [N*V] (or [N, V]).  Returns (out like y, rstd [...] fp32)."""
    tokens, d = _norm_dims(y)
    io = y.dtype
    _chk(g_in, "g_in", tuple(y.shape), io); _chk(w, "w", tuple(w.shape), io)
    if w.numel() != d:
        raise ValueError(f"w has {w.numel()} entries, the rows have {d}")
    if out is None:
        out = torch.empty_like(y)
    if rstd is None:
        rstd = torch.empty(tuple(y.shape[:-2]), dtype=torch.float32, device=y.device)
    _chk(out, "out", tuple(y.shape), io); _chk(rstd, "rstd", tuple(y.shape[:-2]), torch.float32)
    rc = _lib().m2rnn_gated_norm_fwd(tokens, d, _io_code(io), _ptr(y), _ptr(g_in), _ptr(w), float(eps), int(bool(silu)),
                                     _ptr(out), _ptr(rstd), _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_gated_norm_fwd")
    return out, rstd


def m2rnn_gated_norm_bwd_workspace_bytes(tokens: int, d: int) -> int:
    return int(_lib().m2rnn_gated_norm_bwd_workspace_bytes(tokens, d))


def m2rnn_gated_norm_bwd(y, g_in, w, rstd, dout, *, silu=True, workspace=None, out=None, stream=None):
    """Backward of m2rnn_gated_norm_fwd -> dict(dy, dg, dw [N*V] fp32)."""
    tokens, d = _norm_dims(y)
    io = y.dtype
    _chk(g_in, "g_in", tuple(y.shape), io); _chk(dout, "dout", tuple(y.shape), io); _chk(w, "w", tuple(w.shape), io)
    _chk(rstd, "rstd", tuple(y.shape[:-2]), torch.float32)
    out = out or {}
    dy = out.get("dy", None); dg = out.get("dg", None); dw = out.get("dw", None)
    dy = torch.empty_like(y) if dy is None else dy
    dg = torch.empty_like(y) if dg is None else dg
    dw = torch.empty((d,), dtype=torch.float32, device=y.device) if dw is None else dw
    _chk(dy, "dy", tuple(y.shape), io); _chk(dg, "dg", tuple(y.shape), io); _chk(dw, "dw", (d,), torch.float32)
    need = m2rnn_gated_norm_bwd_workspace_bytes(tokens, d)
    if workspace is None:
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=y.device)
    rc = _lib().m2rnn_gated_norm_bwd(tokens, d, _io_code(io), _ptr(y), _ptr(g_in), _ptr(w), _ptr(rstd), int(bool(silu)),
                                     _ptr(dout), _ptr(dy), _ptr(dg), _ptr(dw), _ptr(workspace), workspace.numel(),
                                     _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_gated_norm_bwd")
    return dict(dy=dy, dg=dg, dw=dw)


def _rows(t, name):
    """[B,T,C] with contiguous channels and a regular token axis -> token stride in elements."""
    if t.dim() == 3 and t.numel() == 0:
        return t.shape[2]
    if t.dim() != 3 or t.stride(2) != 1 or (t.shape[0] > 1 and t.stride(0) != t.shape[1] * t.stride(1)):
        raise ValueError(f"{name}: expected [B,T,C] with contiguous channels and batch entries one after the other")
    return t.stride(1)


def m2rnn_conv_silu_fwd(x, w, bias=None, prev=None, *, out=None, stream=None):
    """SiLU(depthwise causal conv1d of width 4 along time) of x [B,T,C] (a view into a wider tensor is
    fine); w [C,4], bias [C], prev [B,3,C] (the three inputs before t = 0).  Returns out [B,T,C]."""
    B, T, C = x.shape
    io = x.dtype
    _chk(w, "w", (C, 4), io); _chk(bias, "bias", (C,), io); _chk(prev, "prev", (B, 3, C), io)
    if out is None:
        out = torch.empty((B, T, C), dtype=io, device=x.device)
    _chk(out, "out", (B, T, C), io, True)
    rc = _lib().m2rnn_conv_silu_fwd(B, T, C, _io_code(io), _ptr(x), _rows(x, "x"), _ptr(w), _ptr(bias), _ptr(prev),
                                    _ptr(out), _rows(out, "out"), _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_conv_silu_fwd")
    return out


def m2rnn_conv_silu_bwd(x, w, dout, bias=None, prev=None, *, out=None, workspace=None, stream=None):
    """Backward of ``m2rnn_conv_silu_fwd`` -> dict(dx [B,T,C], dw [C,4] fp32, dbias [C] fp32, dprev [B,3,C])."""
    B, T, C = x.shape
    io, dev = x.dtype, x.device
    _chk(w, "w", (C, 4), io); _chk(bias, "bias", (C,), io); _chk(prev, "prev", (B, 3, C), io)
    _chk(dout, "dout", (B, T, C), io, True)
    out = dict(out or {})
    if out.get("dx") is None: out["dx"] = torch.empty((B, T, C), dtype=io, device=dev)
    if out.get("dw") is None: out["dw"] = torch.empty((C, 4), dtype=torch.float32, device=dev)
    if out.get("dbias") is None: out["dbias"] = torch.empty((C,), dtype=torch.float32, device=dev)
    if out.get("dprev") is None and prev is not None: out["dprev"] = torch.empty((B, 3, C), dtype=io, device=dev)
    _chk(out["dx"], "dx", (B, T, C), io, True); _chk(out["dw"], "dw", (C, 4), torch.float32)
    need = _lib().m2rnn_conv_silu_bwd_workspace_bytes(B, T, C)
    if workspace is None:
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=dev)
    rc = _lib().m2rnn_conv_silu_bwd(B, T, C, _io_code(io), _ptr(x), _rows(x, "x"), _ptr(w), _ptr(bias), _ptr(prev), _ptr(dout),
                                    _rows(dout, "dout"), _ptr(out["dx"]), _rows(out["dx"], "dx"), _ptr(out["dw"]),
                                    _ptr(out.get("dbias")), _ptr(out.get("dprev")), _ptr(workspace), workspace.numel(),
                                    _stream(stream))
    if rc != 0:
        raise M2RNNError(rc, "m2rnn_conv_silu_bwd")
    return out
