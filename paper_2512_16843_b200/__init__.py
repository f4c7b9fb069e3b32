"""B200-native per-layer cache probe of LLMCache: C-ABI CUDA library + thin binding.

`binding` holds the entry points of include/llmcache.h; `synth` holds the seeded
synthetic workload generators (no arithmetic of the method lives there).
"""
from . import binding, synth  # noqa: F401
