"""B200-native layout-lowered named-dimension einsum (Mesh-TensorFlow, arXiv 1811.02084).

The package is a thin binding over the CUDA library ``libmtf_b200.so`` (C ABI in ``include/mtf.h``).
Importing it loads the library and fails loudly when the library has not been built: there is no
CPU fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import (Epilogue, Layout, Mesh, MtfError, Named, Plan, desc, named)  # noqa: F401
