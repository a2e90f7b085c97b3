"""B200-native forward pass of a Parallel Track (PT) decoder stack.

``paper_2602_07306_b200.pt`` is the thin binding over the C-ABI library
(``libpt.so``, built from ``csrc/``); ``paper_2602_07306_b200.inputs`` draws the
seeded synthetic workloads.  Nothing here computes on the CPU: without the
compiled CUDA library every compute call raises.
"""
__all__ = ["inputs"]
