"""B200-native M2RNN recurrent scan (forward, backward through time, decode step).

The compute lives in ``libm2rnn.so`` (hand-written sm_100a CUDA behind a C ABI,
declared in ``include/m2rnn.h``); :mod:`.binding` marshals torch tensors into it.
:mod:`.inputs` only generates seeded synthetic tensors and imports nothing else.
"""
__all__ = ["inputs"]
