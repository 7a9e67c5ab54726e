"""Tropical convolution (max-plus, min-plus, compound, parallel) for NVIDIA B200.

``paper_2504_06881_b200.tconv`` is the thin binding over the C-ABI CUDA library;
``paper_2504_06881_b200.inputs`` draws seeded synthetic layers.  Nothing here
computes on the CPU: the binding raises if the CUDA library is missing.
"""
