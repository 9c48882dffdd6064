"""B200-native adaptive speculative-decoding iteration (AdaEAGLE): Python binding of the C ABI.

The product is the CUDA library `libada.so` (sources under csrc/, interface in include/ada.h).
This package only marshals arguments; PyTorch supplies device memory and streams.
Importing it does not need a GPU; creating an Engine does.
"""
from .binding import (ADA_ERRORS, AdaError, Config, Engine, ada_ldlp_eval_static, lib, exported_symbols)  # noqa: F401
