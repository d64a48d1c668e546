"""Seeded synthetic inputs and workload descriptions.

This package serves both the CUDA library's tests/benchmarks and the CPU
checker.  It holds no attention or cache arithmetic: only layer layouts
(plain data) and a counter-based value generator.
"""
