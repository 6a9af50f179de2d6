"""Seeded synthetic workloads and benchmark-cache builders shared by the tests and bench.py.

Not part of the library: ``inputs`` draws the tensors both the CPU oracle and the CUDA path consume,
``batches`` lays the benchmark configurations out as packed caches through the library's calls.
"""
