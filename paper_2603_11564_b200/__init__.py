"""B200-native DapQ eviction scorer: thin Python binding over libdapq.so.

The functions mirror the C ABI in include/dapq.h one to one.  Importing this package
does not load the shared library; the first call (or load_library()) does, and raises
ImportError if it has not been built - there is no CPU or PyTorch fallback.
"""
from .binding import (DAPQ_BF16, DAPQ_ERR_CUDA, DAPQ_ERR_INVALID_ARG, DAPQ_ERR_TIMEOUT,  # noqa: F401
                      DAPQ_ERR_UNSUPPORTED, DAPQ_ERR_WORKSPACE, DAPQ_F32, DAPQ_FLAG_CUDA_CORE_SCORER, DAPQ_FLAG_ROPE_INTERLEAVED, DAPQ_FLAG_Q_BF16,
                      DAPQ_FLAG_Q_LO_SWEEP1, DAPQ_FLAG_Q_LO_SWEEP2, DAPQ_OK, DAPQ_POOL_AVG,
                      DAPQ_POOL_MAX, DAPQ_POOL_NONE, EXPORTS, DapqError, dapq_cache_view,
                      dapq_compact_kv, dapq_create, dapq_destroy, dapq_evict, dapq_evict_host, dapq_evict_layers, dapq_evict_layers_host,
                      dapq_last_error, dapq_launch_count, dapq_set_wait_limit, dapq_rope_inv_freq_llama3, dapq_poll_status, dapq_profile, dapq_profile_read, PROF_KINDS, dapq_rope_pseudo_q,
                      dapq_recall, dapq_score, dapq_score_static, dapq_shape, dapq_topk_select, load_library,
                      DAPQ_STATIC_SCRATCH_BYTES)
