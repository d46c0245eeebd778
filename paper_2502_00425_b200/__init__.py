"""B200-native W4A8 modality-specific static-quantized linear (MQuant hot path).

The CUDA library is loaded lazily by :mod:`paper_2502_00425_b200.binding`; importing
the package itself touches neither CUDA nor the shared library, so the seeded
input generators in :mod:`paper_2502_00425_b200.synth` can be used on any machine.
"""
__all__ = ["synth", "binding", "build"]
