"""B200-native (sm_100a) int8 inference path of Q8BERT: quantised FC and embedding layers.

The arithmetic runs in hand-written CUDA kernels behind a C-ABI shared library
(``include/q8.h``); :mod:`.binding` marshals device pointers into it.  The library is loaded on
first use and loading fails loudly when it has not been built: there is no CPU fallback.
"""

__all__ = ["binding", "synth", "build", "encoder"]
