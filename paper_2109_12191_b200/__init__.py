"""B200-native DPSGD gradient-privatisation step (per-example weight gradients, norms,
clip, accumulate, noise, average) as a C-ABI CUDA library with a thin Python binding.

``synth`` (input generators) imports without the compiled library; everything in
``binding`` needs ``libdpstep.so`` and raises if it is missing.
"""
__all__ = ["synth", "binding", "build"]
