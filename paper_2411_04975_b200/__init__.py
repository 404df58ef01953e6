"""B200-native batched SuffixDecoding draft generation (arXiv 2411.04975).

`SuffixStore` is a thin binding of the C ABI declared in include/suffixspec.h;
every step of the path runs in the CUDA library.  Importing this package does
not load the library; the first use does, and fails loudly if it is missing.
"""
from .binding import (FLAG_GLOBAL_ONLY, FLAG_LINEAR, FLAG_REQUEST_ONLY, STATUS_BAD_SLOT, STATUS_BAD_TOKEN,  # noqa: F401
                      STATUS_GLOBAL_FULL, STATUS_POOL_FULL, SuffixSpecError, SuffixStore, library, sd_build,
                      sd_append, sd_speculate, sd_speculate_noalloc, sd_free)
