"""B200 (sm_100a) Superposed Decoding: thin Python binding over the C-ABI library libspd.so.

Every step of the decoding path runs inside the CUDA library; this package only marshals
arguments (torch is used for device memory and streams).  Importing it does not load the
library; the first use does, and fails loudly if the library is missing and cannot be built.
"""
from .binding import (SpdConfig, SpdError, SpdContext, build_ngram_tables, pack_weights, load_library,
                      DBG, status_name, spd_batch_generate, spd_batch_step)

__all__ = ["SpdConfig", "SpdError", "SpdContext", "build_ngram_tables", "pack_weights", "load_library", "DBG",
           "status_name", "spd_batch_generate", "spd_batch_step"]
