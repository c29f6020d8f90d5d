"""B200-native chunked causal attention (forward, LSE merge, backward) behind a C ABI.

`binding` mirrors the C entry points of include/hydra_attn.h; `runner.AttnStep` owns the device
buffers of one problem and calls them in order. Importing fails loudly if the CUDA library cannot
be loaded or built: there is no fallback path.
"""
from .binding import *  # noqa: F401,F403
from .binding import EXPORTS, LIBRARY_PATH, PAIR_DTYPE, HydraError, as_pairs  # noqa: F401
