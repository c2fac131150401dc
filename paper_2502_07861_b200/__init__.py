"""BalanceKV hot path on B200: C-ABI CUDA library plus a thin ctypes binding."""
from .binding import (  # noqa: E402,F401
    BalanceKVError,
    Config,
    Context,
    EXPORTS,
    LIB_PATH,
    decode_attn_static,
    decode_attn_static_status,
    load,
    plan_calls,
)
