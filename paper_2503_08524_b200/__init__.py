"""D3 (Position-Aware Depth Decay Decoding) on one B200: CUDA library + binding.

`inputs` (seeded synthetic data) imports without the CUDA library; `binding`
loads libd3.so and raises if it is missing or cannot be built.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
