"""B200-native batched N-gram speculation step (arXiv 2411.03786): Python binding of the C ABI.

Every step runs in the CUDA library ``libngram_spec.so`` (hand-written sm_100a kernels).  This
package only marshals arguments: torch tensors supply device memory and the stream.  There is
no CPU path; importing works without a GPU (so the build can be checked), but creating a
``SpecContext`` without an sm_100 device raises.
"""
from .binding import (FLAG_DEDUP, FLAG_KEY_NEXT_TOKEN, FLAG_MODEL_FILL, FLAG_PARTIAL_TAIL, STATUS_CAPACITY, STATUS_GROUPS, STATUS_INDEX, STATUS_TIMEOUT,
                      STATUS_TOKEN_RANGE, SpecContext, SpecError, declared_symbols, flag_reserve, load_library, unpack_keys,
                      verify_lmhead_argmax_noalloc)

__all__ = ["SpecContext", "SpecError", "load_library", "unpack_keys", "declared_symbols", "flag_reserve", "verify_lmhead_argmax_noalloc", "FLAG_DEDUP", "FLAG_MODEL_FILL", "FLAG_KEY_NEXT_TOKEN", "FLAG_PARTIAL_TAIL",
           "STATUS_TOKEN_RANGE", "STATUS_CAPACITY", "STATUS_TIMEOUT", "STATUS_GROUPS", "STATUS_INDEX"]
