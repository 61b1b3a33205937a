"""B200-native dynamic weight slicing (DS-Net++ inference hot path): Python binding of libdsn.

The package is a thin argument-marshalling layer over the C ABI declared in include/dsn.h.
There is no CPU or framework fallback: calling any compute entry point without the built
CUDA library raises ImportError.
"""
from .binding import *  # noqa: F401,F403
from .binding import (Context, DsnError, EXPORTS, LIB_PATH, Routing, GateDesc, LinearDesc, ConvDesc, LayerDesc, AttentionDesc, DepthwiseDesc, Stats,
                      load_library)
