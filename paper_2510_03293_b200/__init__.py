"""LASER (Load- and Score-based Expert Routing) hot path for NVIDIA B200.

``paper_2510_03293_b200.laser`` is the Python binding of the C-ABI CUDA library
(``liblaser.so``, built from ``csrc/``); ``paper_2510_03293_b200.synth`` generates the
seeded synthetic workloads.  There is no CPU implementation in this package: importing
``laser`` without the built library raises.
"""
__all__ = ["laser", "synth"]
