"""B200 (sm_100a) latent-KV decode attention for LoRC (arXiv 2410.03111).

The product is the C-ABI shared library declared in include/lorc.h; this package
holds its CUDA sources (csrc/), the build step (_build.py) and a ctypes binding
with the same entry-point names (binding.py).
"""
from . import _build  # noqa: F401


def load():
    """Import the binding (raises ImportError when liblorc.so has not been built)."""
    from . import binding
    return binding
