"""dai8: Distribution Adaptive INT8 convolution backward for B200 (sm_100a).

The product is the C-ABI library built from ``csrc/`` (entry points declared in ``include/dai8.h``);
``paper_2102_04782_b200.api`` is the thin Python binding with the same names and
``paper_2102_04782_b200.synth`` the seeded synthetic workloads.  Importing the package loads
nothing; the shared library is opened on first use and its absence is an error, never a fallback.
"""
__all__ = ["api", "synth", "build"]
