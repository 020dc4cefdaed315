"""B200-native packed-wavefront decode step (FlowBlock hot path).

The CUDA library is loaded lazily by :mod:`paper_2607_17652_b200.binding`;
importing this package (for the seeded input generators) needs no GPU.
"""
__all__ = ["synth", "binding"]
