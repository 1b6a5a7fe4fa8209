"""Tree-decode attention over prefix-shared paged KV for B200 (sm_100a).

The product is `libets_b200.so` (C ABI in include/ets.h); this package is its thin ctypes
binding.  The binding is loaded on first use of any of its names and raises ImportError if the
library has not been built (`python -m paper_2502_13575_b200.build`); there is no fallback.
"""
import importlib

_BINDING_NAMES = (
    "EtsContext", "EtsError", "ets_config", "ets_pool_bytes", "ets_select", "ets_version", "ets_probe_stream_read", "ets_probe_empty_launch", "make_config", "lib",
    "ETS_OK", "ETS_ERR_INVALID_ARG", "ETS_ERR_BAD_TREE", "ETS_ERR_POOL_EXHAUSTED", "ETS_ERR_UNSUPPORTED",
    "ETS_ERR_STATE", "ETS_ERR_CUDA", "ETS_ERR_DEVICE_TIMEOUT",
    "ETS_OPT_CHUNK_PAGES", "ETS_OPT_KERNEL", "ETS_OPT_TIMING", "ETS_OPT_WIDE", "ETS_OPT_HOST_PIPELINE", "ETS_OPT_PATH_ITEMS", "ETS_OPT_OVERLAP_APPEND", "ETS_OPT_PACKED_INPUTS",
    "ETS_OPT_LAUNCH_CHAIN", "ETS_OPT_TEST_FIRST_WAIT_POLLS",
)


def __getattr__(name):
    if name in _BINDING_NAMES:
        binding = importlib.import_module(".binding", __name__)   # loads the shared library
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
