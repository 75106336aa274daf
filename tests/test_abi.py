"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

from paper_2603_14360_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2603_14360_b200 import build
    build.build()
    return binding._lib()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "m2rnn.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(m2rnn_[a-z0-9_]+)\s*\(", hdr))
    assert {"m2rnn_fwd", "m2rnn_bwd", "m2rnn_decode_step"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(binding.EXPORTS), "binding and header disagree"
    assert lib.m2rnn_version() >= 100
    assert b"NULL" in lib.m2rnn_status_string(-1)


def _p(**kw):
    base = dict(B=2, T=8, N=4, Nq=4, Nk=4, K=32, V=32, io_dtype=1, gate_kind=1, ckpt_interval=0, dh_clip=0.0)
    base.update(kw)
    return binding.Params(**base)


FAKE = ctypes.c_void_p(0x10000)      # aligned, never dereferenced: every call below must fail first
ODD = ctypes.c_void_p(0x10004)


def _fwd(lib, p, **over):
    a = dict(q=FAKE, k=FAKE, v=FAKE, gate=FAKE, W=FAKE, h0=None, alpha=None, beta=None, w_r=None,
             y=FAKE, hT=None, ckpt=None, ws=None, ws_bytes=0, st=None, stream=None)
    a.update(over)
    return lib.m2rnn_fwd(ctypes.byref(p), *a.values())


def test_fwd_rejects_bad_arguments(lib):
    assert lib.m2rnn_fwd(None, *([FAKE] * 13), 0, FAKE, FAKE) == -1
    assert _fwd(lib, _p(N=0)) == -2
    assert _fwd(lib, _p(Nq=3)) == -2                  # does not divide N
    assert _fwd(lib, _p(Nk=8)) == -2                  # more key heads than heads
    assert _fwd(lib, _p(T=-1)) == -2
    assert _fwd(lib, _p(K=24)) == -3                  # not a multiple of 16
    assert _fwd(lib, _p(K=144)) == -3
    assert _fwd(lib, _p(V=48)) == -3
    assert _fwd(lib, _p(io_dtype=7)) == -3
    assert _fwd(lib, _p(gate_kind=3)) == -3
    assert _fwd(lib, _p(ckpt_interval=100000)) == -3
    assert _fwd(lib, _p(), q=None) == -1
    assert _fwd(lib, _p(), y=None) == -1
    assert _fwd(lib, _p(gate_kind=2)) == -1           # psi needs alpha and beta
    assert _fwd(lib, _p(), v=ODD) == -4
    assert _fwd(lib, _p(), hT=ODD) == -4
    # few units: the rows of a state are split over CTAs and y passes through a workspace
    small = _p(B=1, N=2, Nq=2, Nk=2, K=64, V=64)
    need = lib.m2rnn_fwd_workspace_bytes(ctypes.byref(small))
    assert need >= 2 * 1 * 8 * 2 * 64 * 4
    assert _fwd(lib, small) == -5
    assert _fwd(lib, small, ws=ctypes.c_void_p(0x20000), ws_bytes=need - 1) == -5
    assert _fwd(lib, small, ws=ctypes.c_void_p(0x20010), ws_bytes=need) == -4
    assert lib.m2rnn_fwd_workspace_bytes(ctypes.byref(_p(B=64, N=16))) == 0
    # empty calls are fine and launch nothing
    assert _fwd(lib, _p(T=0)) == 0
    assert _fwd(lib, _p(B=0)) == 0


def test_bwd_rejects_bad_arguments(lib):
    p = _p()
    need = lib.m2rnn_bwd_workspace_bytes(ctypes.byref(p), 0)
    need_ck = lib.m2rnn_bwd_workspace_bytes(ctypes.byref(p), 1)
    assert need > need_ck > 0
    assert need - need_ck >= lib.m2rnn_ckpt_bytes(ctypes.byref(p)) > 0
    ws = ctypes.c_void_p(0x20000)

    def bwd(p, ws=ws, nbytes=need, **over):
        a = dict(q=FAKE, k=FAKE, v=FAKE, gate=FAKE, W=FAKE, h0=None, alpha=None, beta=None, w_r=None,
                 ckpt=None, dy=FAKE, d_hT=None, dq=FAKE, dk=FAKE, dv=FAKE, dgate=FAKE, dW=FAKE, dh0=None)
        a.update(over)
        return lib.m2rnn_bwd(ctypes.byref(p), *a.values(), ws, nbytes, None, None)

    assert bwd(p, nbytes=need - 1) == -5
    assert bwd(p, ws=None) == -5
    assert bwd(p, ws=ctypes.c_void_p(0x20010)) == -4
    assert bwd(p, dy=None) == -1
    assert bwd(p, dW=None) == -1
    assert bwd(p, dq=ODD) == -4
    assert bwd(_p(V=8)) == -3
    # shared q/k heads need per-head partial sums in the workspace
    pm = _p(Nq=1, Nk=1)
    assert lib.m2rnn_bwd_workspace_bytes(ctypes.byref(pm), 0) > need


def test_decode_rejects_bad_arguments(lib):
    def dec(p, **over):
        a = dict(q=FAKE, k=FAKE, v=FAKE, gate=FAKE, W=FAKE, alpha=None, beta=None, w_r=None,
                 state=FAKE, y=FAKE, st=None, stream=None)
        a.update(over)
        return lib.m2rnn_decode_step(ctypes.byref(p), *a.values())

    assert dec(_p(), state=None) == -1
    assert dec(_p(K=8)) == -3
    assert dec(_p(), y=ODD) == -4
    assert dec(_p(B=0)) == 0
    assert dec(_p(T=-5, B=0)) == 0                    # T is ignored by the decode step


def test_ckpt_interval_query(lib):
    p = _p()
    c = lib.m2rnn_ckpt_interval(ctypes.byref(p))
    assert c >= 1
    assert lib.m2rnn_ckpt_interval(ctypes.byref(_p(ckpt_interval=4))) == 4
    assert lib.m2rnn_ckpt_bytes(ctypes.byref(_p(T=9, ckpt_interval=4))) == 2 * 4 * 3 * 32 * 32 * 4
    assert lib.m2rnn_ckpt_interval(ctypes.byref(_p(V=7))) == -3


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        binding.m2rnn_version()


def test_plans_for_small_states_with_many_units(lib):
    """V = 16 with more CTAs than SMs (the paper's layer shape, 84 heads x batch 4): the backward
    plan shortens the chunk so that several CTAs share an SM (and takes 32-row CTAs, three per SM,
    where that needs fewer waves); few units keep the long chunk."""
    many = _p(B=4, N=84, Nq=1, Nk=1, K=64, V=16, T=64)
    few = _p(B=1, N=4, Nq=1, Nk=1, K=64, V=16, T=64)
    c_many, c_few = lib.m2rnn_ckpt_interval(ctypes.byref(many)), lib.m2rnn_ckpt_interval(ctypes.byref(few))
    assert 2 <= c_many < c_few <= 16 and c_many % 2 == 0
    assert lib.m2rnn_bwd_row_slab(ctypes.byref(many)) == 32        # 672 CTAs at three per SM: two waves of the shorter kind
    some = _p(B=2, N=84, Nq=1, Nk=1, K=64, V=16, T=64)              # 168 units: one wave at two per SM
    assert lib.m2rnn_bwd_row_slab(ctypes.byref(some)) == 64        # a CTA keeps the whole state
    assert lib.m2rnn_bwd_row_slab(ctypes.byref(few)) == 16         # few units: spread the rows over the SMs
    # a caller may still ask for a longer chunk, up to what one CTA's shared memory holds
    assert lib.m2rnn_ckpt_interval(ctypes.byref(_p(B=4, N=84, Nq=1, Nk=1, K=64, V=16, T=64, ckpt_interval=12))) == 12
    assert lib.m2rnn_ckpt_interval(ctypes.byref(_p(B=4, N=84, Nq=1, Nk=1, K=64, V=16, T=64, ckpt_interval=18))) == -3


def test_gated_norm_rejects_bad_arguments(lib):
    f = lib.m2rnn_gated_norm_fwd
    assert f(-1, 1024, 1, FAKE, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -2
    assert f(4, 0, 1, FAKE, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -2
    assert f(4, 1020, 1, FAKE, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -3          # not a multiple of 8
    assert f(4, 16384, 1, FAKE, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -3         # longer than 8192
    assert f(4, 1024, 5, FAKE, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -3
    assert f(4, 1024, 1, None, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -1
    assert f(4, 1024, 1, ODD, FAKE, FAKE, 0.0, 1, FAKE, None, None) == -4
    assert f(0, 1024, 1, None, None, None, 0.0, 1, None, None, None) == 0           # an empty call needs no pointers
    b = lib.m2rnn_gated_norm_bwd
    need = lib.m2rnn_gated_norm_bwd_workspace_bytes(4096, 1024)
    assert need > 0 and lib.m2rnn_gated_norm_bwd_workspace_bytes(0, 1024) == 0
    args = [FAKE] * 4 + [1] + [FAKE] * 4
    assert b(4096, 1024, 1, *args, None, 0, None) == -5                              # no workspace
    assert b(4096, 1024, 1, *args, FAKE, need - 1, None) == -5                       # too small
    assert b(4096, 1024, 1, *args, ODD, need, None) == -4                            # workspace alignment
    assert b(4096, 1020, 1, *args, FAKE, need, None) == -3
    assert b(4096, 1024, 1, FAKE, FAKE, FAKE, None, 1, FAKE, FAKE, FAKE, FAKE, FAKE, need, None) == -1   # rstd missing
