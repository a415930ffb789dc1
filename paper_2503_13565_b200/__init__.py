"""B200-native MXFP4 weight-only linear layer (the draft-model hot path of ML-SpecQD).

The CUDA library is loaded on first use, not at import, so that the input
generators in :mod:`paper_2503_13565_b200.synth` can be used on a machine
without the built extension.  There is no CPU fallback: every operation raises
if ``libmxq.so`` is missing.
"""
