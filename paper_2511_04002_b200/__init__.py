"""B200-native TS + TAB-Q codec (threshold splitting + token-wise adaptive bit quantisation).

The product is the C-ABI library built from ``csrc/`` (see ``include/tsq.h``); ``binding``
marshals torch tensors into its calls and nothing else.  There is no CPU fallback: every
call fails loudly if the CUDA library is missing.
"""
from . import synth  # noqa: F401  (seeded synthetic inputs; no codec arithmetic)

__all__ = ["synth", "binding", "build"]
