"""B200-native batched schedule evaluation for KV-cache-constrained LLM request scheduling.

``binding`` wraps the C-ABI of ``libkvsched.so`` (built from ``csrc/`` by ``build``); ``workloads``
generates the seeded synthetic backlogs.  The library is CUDA-only: nothing here computes a
schedule on the CPU.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]
