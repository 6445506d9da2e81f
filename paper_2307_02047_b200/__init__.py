"""B200-native CAME optimizer step (Algorithm 2 of "CAME: Confidence-guided Adaptive
Memory Efficient Optimization").

``synth`` holds the seeded synthetic workloads; ``binding`` is the ctypes layer over
the C-ABI CUDA library (imported lazily so that CPU-only tools can use ``synth``).
"""
__all__ = ["synth", "binding", "build"]
