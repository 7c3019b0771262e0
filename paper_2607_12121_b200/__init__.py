"""libflashdiff: region-selective denoising step of a diffusion transformer, B200-native.

The product is the C-ABI shared library built from ``csrc/``; this package is its thin
Python binding.  There is no CPU or PyTorch fallback: importing fails if the library is absent.
"""
from .binding import *  # noqa: F401,F403
from .binding import (lib, Context, FdConfig, FdWeights, FdSamplerWeights, FdRSearch, FlashDiffError, make_config,  # noqa: F401
                      make_sampler_weights, EXPORTS, LIB_PATH)
