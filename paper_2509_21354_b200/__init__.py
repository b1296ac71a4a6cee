"""B200-native RNN-gated chunked KV cache: the decode hot path of KV-Efficient VLA.

The CUDA library (libkve.so, C ABI declared in include/kve.h) is loaded lazily by
`paper_2509_21354_b200.binding`; importing the package itself needs no GPU.
"""
__all__ = ["workloads", "binding", "build"]
