"""B200 (sm_100a) scheme evaluator for Arithmetic-Intensity-Aware Quantization.

`binding` loads libaiq.so (built in-tree by `build.build()`); importing it fails loudly
when the library is absent.  There is no CPU fallback.
"""
from . import build  # noqa: F401


def load():
    """Import and return the ctypes binding (raises ImportError if libaiq.so is missing)."""
    from . import binding
    return binding
