"""B200-native RanDeS hot path: superposition and retrieval of task deltas under
seed-defined random orthogonal transforms (layer shuffle, column sign flip).

``randes`` is the thin binding over the CUDA C-ABI library; ``workloads`` holds
the seeded synthetic weight sets.  Importing the package loads nothing; the
binding loads the compiled library on first use and raises if it is missing.
"""
__all__ = ["randes", "workloads"]
