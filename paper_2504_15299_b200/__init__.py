"""B200-native dual-routed MoE layer over matryoshka-weight-quantized (MWQ) experts.

``paper_2504_15299_b200.binding`` is the thin Python layer over the C-ABI library
(``libd2moe.so``, built from ``csrc/``); it is imported lazily so that the seeded input
generators in ``paper_2504_15299_b200.synth`` can be used on a machine without the library.
"""

__all__ = ["synth", "binding"]
