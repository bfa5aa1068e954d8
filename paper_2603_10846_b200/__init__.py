"""B200-native value-driven memory: batched two-phase retrieval and Q-value update.

``paper_2603_10846_b200.evk`` is the Python binding of the C-ABI library
(``libevk.so``, CUDA for sm_100a); ``paper_2603_10846_b200.synth`` draws the seeded
synthetic workloads.  Importing the package is cheap; the CUDA library is loaded
when ``evk`` is first imported and that import fails loudly if it is missing.
"""
__all__ = ["evk", "synth"]
