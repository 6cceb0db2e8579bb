"""FlashForward renderer chunk attention for B200: Python binding over the C-ABI CUDA library."""
from . import binding  # noqa: F401
from .binding import (FF_ATTN_AUTO, FF_ATTN_SIMT, FF_ATTN_TCGEN05, FF_ATTN_TCGEN05_PAIR, FF_BF16, FF_DEVICE_NONE, FF_ERR_CUDA,  # noqa: F401
                      FF_ERR_INVALID_ARG, FF_ERR_OOM, FF_ERR_STATE, FF_ERR_TIMEOUT, FF_ERR_UNSUPPORTED, FF_F32, FF_OK,
                      Cache, FFError, ff_cache_query_bytes, ff_euler_step, ff_plan_sigma, make_config, make_io)
