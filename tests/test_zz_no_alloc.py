"""The allocation-free backward entry point (``m2rnn_bwd_static_scratch``).

Some users of the library run where device memory cannot be allocated on demand: inside a host
application that owns the allocator and passes in only input and output buffers, or in a service
that forbids allocation once it is up.  For them the backward pass keeps its scratch in a fixed
array inside the library.  These tests call that entry point through the C ABI and require the
same gradients as ``m2rnn_bwd`` (which takes a caller-allocated workspace) and as the fp64 oracle,
twice (or three times) in a row with different shapes, on the fp32 path and on the bf16
tensor-core path, so that whatever one call left in the shared array is shown not to leak into
the next.  The file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import ctypes

import pytest
import torch

from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import GATE_PSI, ScanConfig


def test_oversized_problem_is_refused_on_the_host():
    """Needs no GPU: the size check comes before the device is touched."""
    from paper_2603_14360_b200 import build
    build.build()
    lib = binding._lib()
    p = binding.Params(B=64, T=4096, N=32, Nq=32, Nk=32, K=128, V=128, io_dtype=0, gate_kind=1,
                       ckpt_interval=0, dh_clip=0.0)
    assert lib.m2rnn_bwd_workspace_bytes(ctypes.byref(p), 1) > binding.STATIC_SCRATCH_BYTES
    fake = ctypes.c_void_p(0x10000)          # aligned, never dereferenced
    rc = lib.m2rnn_bwd_static_scratch(ctypes.byref(p), *([fake] * 5), None, None, None, None, fake, fake, None,
                                      *([fake] * 5), None, None, None)
    assert rc == -5
    assert lib.m2rnn_bwd_static_scratch(None, *([fake] * 20)) == -1


def _alloc_outputs(g):
    B, N, K, V = g["h0"].shape
    return dict(dq=torch.empty_like(g["q"]), dk=torch.empty_like(g["k"]), dv=torch.empty_like(g["v"]),
                dgate=torch.empty_like(g["gate"]), dW=torch.empty((N, V, V), dtype=torch.float32, device="cuda"),
                dh0=torch.empty_like(g["h0"]))


FP32_CASES = [ScanConfig("na1", B=2, T=45, N=4, K=32, V=32, Nq=1, Nk=2, dtype="f32", gate_kind=GATE_PSI, seed=31),
              ScanConfig("na2", B=3, T=21, N=2, K=64, V=16, dtype="f32", seed=32)]
# bf16: the tensor-core kernels lay more partial sums out in the shared array -- per-row-slab shares
# of dv and dgate when a state's rows are split over CTAs (4 slabs in the first case), per-head
# shares of dq and dk when heads share them (both cases) -- and the two cases differ in every size,
# so the second call finds the first one's leftovers at other offsets
BF16_CASES = [ScanConfig("na3", B=1, T=33, N=4, K=64, V=16, Nq=1, Nk=1, seed=33),
              ScanConfig("na4", B=2, T=27, N=4, K=32, V=32, Nq=2, Nk=1, gate_kind=GATE_PSI, w_scale=0.5, seed=34)]


@pytest.mark.gpu
@pytest.mark.parametrize("cfgs", [FP32_CASES, BF16_CASES, BF16_CASES[::-1] + FP32_CASES[:1]], ids=["f32", "bf16", "mixed"])
def test_matches_workspace_entry_point_twice_in_a_row(oracle, cfgs):
    import parity
    for cfg in cfgs:
        d = inputs.make_inputs(cfg, backward=True, residual=True, d_hT=True)
        g = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in d.items()}
        kw = dict(gate_kind=cfg.gate_kind, alpha=g["alpha"], beta=g["beta"], w_r=g["w_r"])
        ref = binding.m2rnn_bwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], g["dy"], g["d_hT"], **kw)
        out = _alloc_outputs(g)                    # the caller's buffers; the call itself allocates nothing
        torch.cuda.synchronize()
        count = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]   # allocation events so far
        before = count()
        got = binding.m2rnn_bwd_static_scratch(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"], g["dy"],
                                               g["d_hT"], out=out, **kw)
        torch.cuda.synchronize()
        assert count() == before
        binding.check_device_status()
        want = parity.oracle_bwd(oracle, cfg, d)
        for name, r in ref.items():
            # same kernels, same order of operations as m2rnn_bwd: equal far inside the path's bound ...
            scale = r.abs().max().item()
            err = (got[name].double() - r.double()).abs().max().item()
            assert err <= 1e-4 * scale, (cfg.name, name, err, scale)
            # ... and the gradients themselves are right: against the fp64 oracle at the path's tolerance
            assert parity.rel_err(got[name], want[name]) <= parity.TOL[cfg.dtype], (cfg.name, name)
