"""B200-native DPPF consensus round: CUDA kernels behind a C ABI, plus this thin binding.

``inputs`` (seeded synthetic workloads) imports without a GPU.  The compute
entry points live in ``binding`` and load ``libdppf.so``; they raise if the
library has not been built -- there is no CPU fallback.
"""
__all__ = ["inputs", "binding", "build"]
