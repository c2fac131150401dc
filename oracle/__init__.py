"""CPU oracle for BalanceKV -- test infrastructure only.

Only tests, the smoke check and the bench's CPU baseline may import this package;
the CUDA library and its Python binding never do.
"""
from .binding import (  # noqa: F401
    OracleParams,
    OracleStream,
    build,
    compress_streams,
    merged_estimate,
    num_threads,
    philox4x32_10,
    softmax_balance,
    two_instance_estimate,
    walk_constant,
    walk_uniform,
    weighted_attention,
    weighted_sums,
)
from .bucketing import NO_BUCKET, BucketedOracle, value_bucket  # noqa: F401,E402
from .preserving import PreservingOracle, anticorrelated  # noqa: F401,E402
