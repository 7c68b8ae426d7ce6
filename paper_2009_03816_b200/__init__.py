"""B200-native PSO-PS parameter synchronisation (CUDA library + thin binding).

Importing the package is cheap; the CUDA shared library is loaded on first use
of :mod:`paper_2009_03816_b200.binding` and its absence is an error, never a
fallback.
"""
__all__ = ["binding", "build", "replicas", "sharded", "workloads"]
