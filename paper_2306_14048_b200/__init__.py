"""B200 (sm_100a) implementation of the H2O KV-cache eviction hot path behind a C ABI.

The product is ``libh2o_b200.so`` (see ``include/h2o.h``); this package is the thin
Python binding used by the tests and the benchmark.
"""
from .binding import (  # noqa: F401
    EXPORTED,
    H2O_BF16,
    H2O_BF16_KV4,
    H2O_ERR_CUDA,
    H2O_ERR_INVALID_ARG,
    H2O_ERR_STATE,
    H2O_ERR_TIMEOUT,
    H2O_ERR_UNSUPPORTED,
    H2O_ERR_WORKSPACE,
    H2O_F32,
    H2O_OK,
    H2OCache,
    H2OError,
    h2o_cache_workspace_bytes,
    h2o_config_t,
    h2o_prefill_scratch_bytes,
    lib,
    make_config,
)
