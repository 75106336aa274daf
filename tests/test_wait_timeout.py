"""The failure-reporting path of the bounded device-side waits, exercised without making anything
fail: the library's self-test kernel waits (with the wait routine of the scan kernels and a limit
of a few thousand SM clocks) on a barrier that nothing completes, gives up, reports
M2RNN_ERR_TIMEOUT through the status word and returns; the context stays usable."""
import ctypes

import pytest
import torch

from paper_2603_14360_b200 import binding, inputs
from paper_2603_14360_b200.inputs import ScanConfig


def test_selftest_rejects_bad_arguments():
    from paper_2603_14360_b200 import build
    build.build()
    lib = binding._lib()
    fake = ctypes.c_void_p(0x10000)
    assert lib.m2rnn_wait_selftest(1000, None, None, None) == -1
    assert lib.m2rnn_wait_selftest(-1, fake, None, None) == -2
    assert lib.m2rnn_wait_selftest(10 ** 9, fake, None, None) == -2      # a self-test never waits that long


@pytest.mark.gpu
@pytest.mark.parametrize("limit", [0, 5000, 2_000_000])
def test_wait_runs_out_and_reports(limit):
    status, waited = binding.m2rnn_wait_selftest(limit)
    torch.cuda.synchronize()
    assert status == -7                                     # M2RNN_ERR_TIMEOUT
    # the wait lasted at least its limit and not much longer (the clock is read every 32nd poll, and
    # the polls sleep in between: a millisecond of slack at 2 GHz)
    assert waited >= limit and waited <= limit + 2_000_000, (limit, waited)
    # the kernel returned normally: the same context runs a scan right after, status word clean
    cfg = ScanConfig("after", B=1, T=8, N=1, K=16, V=16, seed=1)
    g = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inputs.make_inputs(cfg).items()}
    y, hT, _ = binding.m2rnn_fwd(g["q"], g["k"], g["v"], g["gate"], g["W"], g["h0"])
    binding.check_device_status()
    assert torch.isfinite(y.float()).all()


@pytest.mark.gpu
def test_status_word_raises_through_the_binding():
    """What a caller sees: the status word the scan calls share is raised by a timed-out wait and
    check_device_status() turns it into an exception, once."""
    w = binding.device_status_word()
    rc = binding._lib().m2rnn_wait_selftest(1000, ctypes.c_void_p(w.data_ptr()), None, binding._stream(None))
    assert rc == 0
    with pytest.raises(binding.M2RNNError) as e:
        binding.check_device_status()
    assert e.value.status == -7
    binding.check_device_status()                           # cleared
