"""B200-native SKVQ hot path: sliding-window KV-cache quantization and decode attention.

The compute lives in a C-ABI CUDA library (``csrc/``, declared in ``include/skvq.h``);
``binding`` marshals torch tensors to it and ``workloads`` draws the synthetic inputs.
Nothing is loaded at import time; the CUDA library is opened on first use and a missing
library is an error, never a fallback.
"""
__all__ = ["binding", "workloads"]
