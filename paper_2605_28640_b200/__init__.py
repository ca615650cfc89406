"""Query-aware sparse decode attention over exponentially decaying KV memory,
as hand-written CUDA for B200 behind a small C ABI (see ``include/rq.h``)."""
from .binding import (  # noqa: F401
    RQ_BF16, RQ_ERR_CAPACITY, RQ_ERR_CUDA, RQ_ERR_INVALID_ARG, RQ_ERR_TIMEOUT, RQ_ERR_UNSUPPORTED, RQ_F32,
    RQ_OK, Cache, RqError, rq_attend_pages, rq_attend_pages_noalloc, rq_build_cache, rq_cache, rq_cache_init, rq_cache_len, rq_decode_step_launches,
    rq_cache_reset, rq_config, rq_decode_step, rq_decode_step_host, rq_decode_step_profiled, rq_device_status, rq_moba_prefill, rq_moba_scratch_bytes, rq_probe_read, rq_select_pages, rq_snapkv_compact, rq_snapkv_scratch_bytes, rq_snapkv_select,
    rq_sizes, rq_status_string, rq_version)
