"""B200-native forward (prefill + decode) of Ladder-Residual / standard transformers.

The compute lives in ``libladder.so`` (hand-written sm_100a CUDA behind a C ABI,
declared in ``include/ladder.h``); :mod:`.binding` marshals arguments to it and
:mod:`.synth` generates seeded synthetic models.  There is no CPU fallback.
"""
