"""B200-native hot path of TCA-Attention: score -> select -> compact -> sparse attention.

The compute lives in a C-ABI shared library of hand-written sm_100a kernels
(``csrc/``, declared in ``include/tca.h``); :mod:`.binding` marshals arguments to it and
:mod:`.inputs` draws the synthetic workloads.  Nothing here falls back to the CPU: if
the library is missing, loading it raises.
"""
__version__ = "0.1.0"
