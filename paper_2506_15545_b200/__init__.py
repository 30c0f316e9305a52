"""RAttention (sliding-window attention + residual linear attention) for B200.

The operator lives in a C-ABI CUDA library (``csrc/``); :mod:`.binding` marshals torch
tensors into it.  Importing the package does not load the library; the first call does,
and fails loudly when it is missing.
"""
