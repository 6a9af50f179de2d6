"""SparK hot path on B200: per-token key-channel pruning of the KV cache and decode attention with
on-the-fly recovery, as a C-ABI CUDA library (``libspark.so``) plus this thin binding.

Modules: ``binding`` (ctypes, same names as include/spark.h), ``cache`` (device buffers around the calls),
``inputs`` (seeded synthetic workloads), ``build`` (nvcc build).  Nothing here computes the method.
"""
__all__ = ["binding", "cache", "inputs", "build"]
