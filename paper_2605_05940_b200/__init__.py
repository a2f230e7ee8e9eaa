"""B200-native packed-sequence distillation loss step (Near-Policy Distillation).

The compute lives in a C-ABI shared library of hand-written sm_100a kernels
(``csrc/``, declared in ``include/npd.h``); ``binding`` marshals arguments to it.
Importing the package does not load the library; the first call does, and raises
if it has not been built.
"""

__all__ = ["binding", "synth_inputs"]
