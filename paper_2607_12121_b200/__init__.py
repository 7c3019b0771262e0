"""libflashdiff: region-selective denoising step of a diffusion transformer, B200-native.

The product is the C-ABI shared library built from ``csrc/``; this package is its thin
Python binding.  There is no CPU or PyTorch fallback: importing fails if the library is absent.
"""
from .binding import *  # noqa: F401,F403
from .binding import lib, Context, FdConfig, FdWeights, FlashDiffError, make_config, EXPORTS, LIB_PATH  # noqa: F401
