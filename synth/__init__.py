"""Seeded synthetic workload generator shared by the tests, the bench and the smoke run.

This package holds none of the method's arithmetic: it only produces bf16 Q/K/V
tensors that are a pure function of (seed, stream, sequence, layer, head, position,
channel), identical bit for bit on the CPU and on a CUDA device.
"""
from .generator import Workload, WORKLOADS, normal_table  # noqa: F401
