"""B200-native SLiM compressed linear layer: Y = X (s Q)^T + (X R^T) L^T.

The compute path is the C-ABI CUDA library ``libslim.so`` (sources under
``csrc/``, interface in ``include/slim.h``); :mod:`.binding` marshals torch
tensors into it.  There is no CPU or library fallback: calls raise when the
library is missing.
"""
__all__ = ["binding", "inputs", "parity", "build"]
