"""B200-native verify step for speculative decoding with a per-step draft length.

The package is a thin binding over a C-ABI CUDA library (``csrc/``):

* ``spec_verify_attn``   -- attention of the draft block against the paged KV cache
* ``spec_accept_sample`` -- fused accept / resample over the vocabulary
* ``gamma_tune_update``  -- the GammaTune controller, state kept on the device

``synth`` holds the seeded input generators; it does not need the CUDA library.
Everything else loads the library on first use and raises if it is missing.
"""
from __future__ import annotations

import importlib

_LAZY = ("binding", "synth", "build", "shard")


def __getattr__(name):
    if name in _LAZY:
        return importlib.import_module(f"{__name__}.{name}")
    binding = importlib.import_module(f"{__name__}.binding")
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
