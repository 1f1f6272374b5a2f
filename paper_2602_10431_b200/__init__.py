"""B200-native forward path of a QTALE token-adaptive quantised layer.

Sub-modules are imported on demand so that the input generators can be used
without the CUDA library being present:

  inputs      seeded synthetic inputs (no layer arithmetic)
  accounting  FLOP / byte model of the path
  api         thin binding over the C-ABI library (requires the built library)
"""
__all__ = ["inputs", "accounting", "api", "build"]
