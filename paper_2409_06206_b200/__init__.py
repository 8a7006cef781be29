"""B200-native Group Shifted Window Attention (GSWA) layer: forward and training backward.

The CUDA library (`libgswa.so`, built from `csrc/`) is loaded lazily by
`binding`; importing the package itself needs no GPU.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
