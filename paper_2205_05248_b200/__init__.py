"""B200-native batched actor step for multi-agent reinforcement learning.

``paper_2205_05248_b200.binding`` is the thin ctypes layer over the C-ABI CUDA library
(``libmarl_actor.so``, built in-tree by ``paper_2205_05248_b200.build``); ``workloads`` holds the seeded
synthetic input recipes.  Importing the package loads nothing; the CUDA library is loaded on first use
and its absence is an error, never a fallback.
"""
__all__ = ["binding", "workloads", "build"]
