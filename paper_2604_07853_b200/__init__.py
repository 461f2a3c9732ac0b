"""B200-native block-scaled FP8 quantized forward (QaRL hot path).

The CUDA library is loaded lazily by :mod:`paper_2604_07853_b200.binding`; importing the
package (for example to reach the seeded input generators) loads nothing.
"""
__all__ = ["binding", "inputs"]
