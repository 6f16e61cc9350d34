"""UniQL inference hot path for B200: the C-ABI CUDA library and its thin Python binding.

`from paper_2512_03383_b200 import binding` loads libuniql.so and fails loudly when it is
missing; `synth` (pure numpy input generators) imports without it.
"""
__all__ = ["binding", "synth", "build"]
