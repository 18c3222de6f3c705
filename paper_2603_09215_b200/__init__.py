"""B200-native SPAR-K decode: C-ABI CUDA library plus a thin ctypes binding.

``synth`` (seeded inputs) imports nothing from the CUDA side; ``binding`` loads the
compiled library and fails loudly when it is missing.
"""
