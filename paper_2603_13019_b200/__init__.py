"""B200-native batched elastic scheduling round of ARL-Tangram (arxiv 2603.13019).

The product is the CUDA library `libtangram.so` (C ABI in include/tangram.h); this package
is its thin Python binding: argument marshalling only, every step runs in the kernels.
"""
from .binding import (  # noqa: F401
    POOL_CPU, POOL_GPU, POOL_API, UNIT_GANG,
    STATUS_OK, STATUS_BAD_ACTION, STATUS_UNSORTED, STATUS_WORKSPACE,
    TangramError, PoolDesc, Round, round_create, load_library, to_device,
)
