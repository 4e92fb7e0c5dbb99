"""B200-native AWEQ calibration pass (arXiv 2311.01305).

``paper_2311_01305_b200.aweq`` is the thin Python binding of the C-ABI CUDA
library (it raises at import when the library is missing);
``paper_2311_01305_b200.synth`` draws the seeded synthetic inputs.
Nothing is imported eagerly so that the input generators can be used on a
machine without the CUDA library.
"""
__all__ = ["aweq", "synth", "build"]
