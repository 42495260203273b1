"""GDWS convolution forward for NVIDIA B200 (sm_100a): C-ABI library + thin binding.

The compute lives in ``csrc/`` behind the C interface declared in ``include/gdws.h``;
``gdws`` (this package's binding) only marshals arguments.  ``inputs`` draws the
seeded synthetic layers.  Nothing here falls back to a CPU path.
"""
__version__ = "0.1.0"
