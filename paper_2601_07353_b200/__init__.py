"""B200-native hot path of Talon (confidence-aware, budget-driven speculative decoding).

``paper_2601_07353_b200.talon`` is the thin Python binding over the C-ABI library built
from ``csrc/``; ``paper_2601_07353_b200.synth`` generates the seeded synthetic inputs.
Nothing is imported eagerly so that the input generator can be used without the CUDA
library being built.
"""

__all__ = ["synth", "talon", "build"]
