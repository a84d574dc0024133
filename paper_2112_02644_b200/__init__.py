"""SMTM semantic-memory hot path on NVIDIA B200: Python binding of the C-ABI CUDA library.

The library (``libsmtm.so``, built from ``csrc/`` by ``build.py``) does all the
work; this package only marshals arguments.  There is no CPU fallback: calls
fail if the library is missing or no sm_100 device is present.
"""
from .binding import (  # noqa: F401
    BF16, F16, F32, FLAG_FORGET_FT, FLAG_MAPS_READY, NCHW, NHWC, CTR_EXITS, CTR_LOOKUPS, CTR_NEAR, MAX_LAYERS, PROF_CENTERS, PROF_FINISH_DENSE, PROF_KERNELS, PROF_PLAN, PROF_REFRESH, PROF_SCORE, PROF_SCORE_TC, PROF_TABLES, Batch, Cache, SmtmError,
    Fmap, ROUTE_COUNT, ROUTE_DENSE, ROUTE_FUSED, ROUTE_PIPELINED, ROUTE_PIPELINED_DENSE, ROUTE_PLAIN, declared_symbols, library_path, load_library, smtm_batch_reset, smtm_cache_create, smtm_cache_destroy,
    smtm_cache_get_centers, smtm_cache_get_counters, smtm_cache_export, smtm_cache_get_launches, smtm_cache_get_members, smtm_cache_get_routes, smtm_cache_import,
    smtm_cache_clear_status, smtm_cache_selftest_wait, smtm_cache_get_profile, smtm_cache_get_profile_device, smtm_cache_get_profile_timeline, smtm_cache_get_tables, smtm_cache_profile, smtm_cache_resize, smtm_cache_status, smtm_cache_update, smtm_cache_update_resize, smtm_cache_warmup, smtm_encode,
    smtm_lookup_exit, smtm_lookup_exit_begin, smtm_lookup_exit_static, smtm_status_string, smtm_step_host,
)
