"""B200-native verify-and-judge step of AutoJudge speculative decoding (C-ABI library + binding)."""
from .binding import (  # noqa: F401
    AJ_BF16, AJ_F32, AJ_W_VD, AJ_W_DV, AJ_FLAG_FORCE_SIMT, AJ_FLAG_TIME_KERNELS, AJ_FLAG_ONE_SM, AJ_FLAG_NO_EXTRA_ROW,
    AJ_OK, AJ_ERR_INVALID_ARG, AJ_ERR_UNSUPPORTED, AJ_ERR_WORKSPACE, AJ_ERR_CUDA, AJ_ERR_TIMEOUT, AJ_ERR_NOT_SM100,
    AjError, Handle, lib, status_string, version, verify_static, AJ_STATIC_MAX_ROWS, pair_schedule, shard_exchange_bytes, shard_exchange_alloc, shard_exchange_free, shard_range, ipc_export, ipc_import, ipc_close, lr_fit, lr_release,
)
