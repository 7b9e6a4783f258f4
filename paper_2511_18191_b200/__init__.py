"""B200 (sm_100a) speculative decoder for continuous patch autoregression: Python binding.

The product is the CUDA library behind include/tsfm.h; this package only loads it and
marshals arguments.  Importing it without the built library raises ImportError.
"""
from .binding import *  # noqa: F401,F403
from .binding import (  # noqa: F401
    SpecDecoder, TsfmError, EXPORTS, lib, pack_weights, tsfm_arch, tsfm_cfg, tsfm_stats, tsfm_variant, tsfm_weights,
)
