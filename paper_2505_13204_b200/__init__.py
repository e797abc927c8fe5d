"""B200-native draft-and-verify path of Alignment-Augmented Speculative Decoding.

``paper_2505_13204_b200.binding`` is the thin Python layer over the C-ABI library built
from ``csrc/``; ``paper_2505_13204_b200.synth`` draws the seeded synthetic workloads.
There is no CPU fallback: calling into the binding without the built CUDA library raises.
"""
