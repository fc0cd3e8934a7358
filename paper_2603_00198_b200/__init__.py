"""libstr: token-reduced prefill of a hybrid Mamba-2 / attention layer stack on B200 (sm_100a).

The CUDA kernels live behind a C-ABI shared library (``csrc/``, declared in ``include/str.h``);
``binding`` marshals arguments to it.  Importing the package does not load the library, so the
host-side helpers (``inputs``) work on machines without a GPU.
"""
__all__ = ["inputs"]
