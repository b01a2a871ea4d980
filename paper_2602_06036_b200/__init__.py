"""B200-native DFlash draft-block / verify-accept path.

The CUDA library is loaded lazily by `paper_2602_06036_b200.binding`; importing the package (or
its `synth` input module) does not need a GPU or the built extension.
"""
__all__ = ["synth", "binding", "build"]
