"""B200-native hot path of DiG's token mixer: chunkwise gated linear attention (forward and
backward) over 2-D patch grids in four scan orders, and the SREM 3x3 depthwise convolution.

``dig`` is the ctypes binding of the C-ABI CUDA library; ``inputs`` holds the seeded synthetic
workloads.  The binding is imported lazily so that ``inputs`` stays usable on a machine with
no CUDA toolchain.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "dig"]


def __getattr__(name):
    if name == "dig":
        import importlib
        return importlib.import_module(".dig", __name__)
    raise AttributeError(name)
