"""B200-native example retrieval for IC-Cache: a bf16 embedding slab in HBM, exhaustive cosine
scoring and fused top-k, behind the C ABI of include/ic_cache.h."""
from .binding import (  # noqa: F401
    ICCache, ICCacheError, load_library,
    ic_cache_create, ic_cache_create_ex, ic_cache_insert, ic_cache_insert_host, ic_cache_query,
    ic_cache_query_host, ic_cache_query_static, ic_cache_query_min_score, ic_cache_destroy, ic_cache_plan, ic_cache_last_error,
    ic_cache_workspace_bytes,
    IC_OK, IC_ERR_INVALID, IC_ERR_NOMEM, IC_ERR_FULL, IC_ERR_CUDA, IC_ERR_UNSUPPORTED, IC_ERR_TIMEOUT,
    IC_BF16, IC_F32, IC_PATH_AUTO, IC_PATH_GENERIC, IC_PATH_SCAN, IC_PATH_UMMA, IC_MAX_K, IC_MAX_DIM,
)
