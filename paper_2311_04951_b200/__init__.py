"""Speculative-sampling verification path with KV caching on one B200 (sm_100a).

``binding`` mirrors the C ABI of ``include/ssd.h`` (hand-written CUDA kernels in ``csrc/``),
``engine`` strings the calls into generation loops, ``synth`` draws seeded synthetic inputs.
Importing the package loads nothing; the first call into ``binding`` loads the compiled
library and fails loudly if it is missing.
"""
