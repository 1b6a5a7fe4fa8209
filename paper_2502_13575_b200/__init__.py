"""Tree-decode attention over prefix-shared paged KV for B200 (sm_100a).

The product is `libets_b200.so` (C ABI in include/ets.h); this package is its thin ctypes
binding.  Importing it loads the library and fails if the library is missing.
"""
from .binding import (  # noqa: F401
    EtsContext,
    EtsError,
    ets_config,
    ets_pool_bytes,
    ets_version,
    make_config,
    lib,
    ETS_OK,
    ETS_ERR_INVALID_ARG,
    ETS_ERR_BAD_TREE,
    ETS_ERR_POOL_EXHAUSTED,
    ETS_ERR_UNSUPPORTED,
    ETS_ERR_STATE,
    ETS_ERR_CUDA,
    ETS_ERR_DEVICE_TIMEOUT,
    ETS_OPT_CHUNK_PAGES,
    ETS_OPT_KERNEL,
    ETS_OPT_TIMING,
)
