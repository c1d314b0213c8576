"""worldkv-b200: the WorldKV hot path (compression, chunk pool, retrieval, memory attention) as hand-written
CUDA for sm_100a behind a C ABI (include/wk.h), with a thin ctypes binding."""
from .binding import (WorldKV, WkError, SCORE_WHOLE_KEY, SCORE_PER_HEAD, retrieve_noalloc, load_library, status_string, wk_config, wk_dense_seg, EXPORTED_SYMBOLS,  # noqa: F401
                      WK_OK, WK_ERR_ARG, WK_ERR_SHAPE, WK_ERR_POOL_FULL, WK_ERR_BAD_SLOT, WK_ERR_CUDA, WK_ERR_TIMEOUT,
                      WK_ERR_NONFINITE, WK_ERR_UNBOUND, WK_ERR_NO_DEVICE, WK_DEV_BAD_SLOT, WK_DEV_TIMEOUT,
                      WK_DEV_NONFINITE)
