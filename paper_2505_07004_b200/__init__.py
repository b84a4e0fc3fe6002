"""libgq: B200-native construction of GuidedQuant's guided layer objective.

``paper_2505_07004_b200.api`` is the ctypes binding of the C-ABI CUDA library
(``include/gq.h``); ``paper_2505_07004_b200.synth`` draws seeded synthetic layers.
"""
__version__ = "0.1.0"
