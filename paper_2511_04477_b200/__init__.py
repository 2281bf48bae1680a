"""SpQt hot path for NVIDIA B200 (sm_100a): activation-sparse, group-quantized GEMV.

The product is the C-ABI shared library built from ``csrc/`` (declared in
``include/spqt.h``); :mod:`paper_2511_04477_b200.binding` marshals arguments to
it and nothing else.  Importing the package does not load the library; the first
call does, and raises if it has not been built.  There is no CPU fallback.
"""

__all__ = ["binding", "inputs", "build"]
