"""B200-native V step of PV-Tuning: select -> re-encode -> dequantise.

The arithmetic lives in the CUDA library (``csrc/``, C ABI in ``include/pvt.h``);
``binding`` marshals arguments to it and ``synth`` draws seeded test layers.
"""
