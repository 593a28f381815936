"""CPU oracle of the Distribution Adaptive INT8 backward path (test infrastructure only).

`oracle.cpu` wraps the plain C++ restatement in ``dai8_oracle.cpp`` (statistics, discriminator,
clip update, quantizers, direct integer convolutions, de-quantization); `oracle.emodel` holds the
numeric model of the magnitude-weighted quantization error (Eq. 8-13) used to pin the clip rule.

Nothing in the CUDA library imports this package, and this package imports nothing from it.
"""
